// The O(B*T) kernels: per-token reward, GAE reverse scan, and the loss finalisation
// (value loss, dvalues, deterministic reduction of both losses).
#pragma once
#include "common.cuh"
#include "kernels_generic.cuh"

namespace rlhf {

// ---------------------------------------------------------------- step 2: per-token reward
// r = -beta * (lp_old - lp_ref), plus the clipped sequence score at the last valid token (t == len-1).
__device__ __forceinline__ float reward_token(float lp_old, float lp_ref, float score, int t, int len,
                                              float beta, float clip)
{
    float r = -beta * (lp_old - lp_ref);
    if (t == len - 1) r += fminf(fmaxf(score, -clip), clip);
    return r;
}

// lp_old and lp_ref carry no __restrict__: `out` may be one of them (each element is read before it is written,
// by the same thread).
__global__ void __launch_bounds__(256) kl_reward_kernel(const float* lp_old, const float* lp_ref,
                                                        const float* __restrict__ score,
                                                        const int* __restrict__ lengths, int B, int T,
                                                        float beta, float clip, float* out)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const long long total = (long long)B * T;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int b = (int)(i / T), t = (int)(i % T);
        int len = clamp_len(__ldg(lengths + b), T);
        float r = 0.f;
        if (t < len) r = reward_token(lp_old[i], lp_ref[i], __ldg(score + b), t, len, beta, clip);
        out[i] = r;
    }
}

// ---------------------------------------------------------------- step 3: GAE
// One warp per sequence.  The recurrence A_t = delta_t + q A_{t+1} (q = gamma*lambda) is an affine
// map of A_{t+1}; each lane composes the maps of its contiguous chunk of the valid range, a
// 5-step shuffle suffix scan composes the chunks, and each lane then replays its chunk from the
// now-known incoming value.  delta_t = r_t + gamma V_{t+1} - V_t with V_len = 0.
constexpr int kGaeWarpsPerBlock = 4;

// GAE of one sequence by one warp: r, v, a_out, g_out point at the sequence's T entries, n valid.
__device__ __forceinline__ void gae_warp(const float* r, const float* v, int n, int T, float gamma, float lambda,
                                         float* a_out, float* g_out, int lane)
{
    const float q = gamma * lambda;
    const int chunk = (n + 31) / 32;
    const int lo = min(n, lane * chunk), hi = min(n, lo + chunk);

    // chunk map: A_lo = P + c * A_hi
    float P = 0.f, c = 1.f;
    {
        float v_next = hi < n ? v[hi] : 0.f;
        for (int t = hi - 1; t >= lo; --t) {
            float vt = v[t];
            float delta = r[t] + gamma * v_next - vt;
            P = fmaf(q, P, delta);
            c *= q;
            v_next = vt;
        }
    }
    // suffix scan over lanes: (P,c) of lane l becomes the map of chunks l..31
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        float P2 = __shfl_down_sync(0xffffffffu, P, o);
        float c2 = __shfl_down_sync(0xffffffffu, c, o);
        if (lane + o < 32) { P = fmaf(c, P2, P); c *= c2; }
    }
    float a = __shfl_down_sync(0xffffffffu, P, 1);     // A at this lane's hi = A_lo of the next chunk
    if (lane == 31) a = 0.f;
    {
        float v_next = hi < n ? v[hi] : 0.f;
        for (int t = hi - 1; t >= lo; --t) {
            float vt = v[t];
            float delta = r[t] + gamma * v_next - vt;
            a = fmaf(q, a, delta);
            a_out[t] = a;
            g_out[t] = a + vt;
            v_next = vt;
        }
    }
    for (int t = n + lane; t < T; t += 32) { a_out[t] = 0.f; g_out[t] = 0.f; }
}

__global__ void __launch_bounds__(kGaeWarpsPerBlock * 32) gae_kernel(const float* __restrict__ rewards,
                                                                     const float* __restrict__ values,
                                                                     const int* __restrict__ lengths,
                                                                     int B, int T, float gamma, float lambda,
                                                                     float* __restrict__ adv,
                                                                     float* __restrict__ ret)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kGaeWarpsPerBlock + (threadIdx.x >> 5);
    if (b >= B) return;
    const int n = clamp_len(__ldg(lengths + b), T);
    gae_warp(rewards + (long long)b * T, values + (long long)b * T, n, T, gamma, lambda,
             adv + (long long)b * T, ret + (long long)b * T, lane);
}

// ---------------------------------------------------------------- steps 2+3 in one launch
// One warp per sequence: the rewards are written first (same formula as kl_reward_kernel), then the
// warp runs the GAE scan over what it has just written.  Results are bit-identical to the two kernels.
__global__ void __launch_bounds__(kGaeWarpsPerBlock * 32) reward_gae_kernel(const float* __restrict__ lp_old,
                                                                            const float* __restrict__ lp_ref,
                                                                            const float* __restrict__ score,
                                                                            const float* __restrict__ values,
                                                                            const int* __restrict__ lengths,
                                                                            int B, int T, float beta, float clip,
                                                                            float gamma, float lambda,
                                                                            float* rewards, float* __restrict__ adv,
                                                                            float* __restrict__ ret)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kGaeWarpsPerBlock + (threadIdx.x >> 5);
    if (b >= B) return;
    const int n = clamp_len(__ldg(lengths + b), T);
    const long long off = (long long)b * T;
    const float sc = __ldg(score + b);
    for (int t = lane; t < T; t += 32)
        rewards[off + t] = t < n ? reward_token(lp_old[off + t], lp_ref[off + t], sc, t, n, beta, clip) : 0.f;
    __syncwarp();
    gae_warp(rewards + off, values + off, n, T, gamma, lambda, adv + off, ret + off, lane);
}

// ---------------------------------------------------------------- optional: advantage whitening
// (A - mean) / sqrt(var + eps) over the valid tokens of the whole batch, population variance, in two launches.
// The first reduces sum and sum of squares in double precision in a fixed order (each block a contiguous range of
// tokens with a fixed tree; the last block to finish adds the block partials in index order) and leaves mean and
// 1/sqrt(var + eps) in the workspace; the second applies them.  No floating-point atomics: bit-stable.
constexpr int kWhitenThreads = 256;
constexpr int kWhitenMaxBlocks = 256;

struct WhitenArgs {
    const float* adv;
    const int* lengths;
    int B, T;
    float eps;
    float* out;
    unsigned* ticket;           // workspace word 1, zero between calls
    double* partials;           // workspace: [kWhitenMaxBlocks][2]
    float* mean_rstd;           // workspace: 2 floats
};

__global__ void __launch_bounds__(kWhitenThreads) whiten_stats_kernel(WhitenArgs p)
{
    __shared__ double s_red[2][kWhitenThreads / 32];
    __shared__ long long s_n[kWhitenThreads / 32];
    __shared__ bool s_last;
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const long long total = (long long)p.B * p.T;
    const long long per_block = (total + gridDim.x - 1) / gridDim.x;
    const long long begin = per_block * blockIdx.x, end = min(total, begin + per_block);
    double s1 = 0.0, s2 = 0.0;
    for (long long i = begin + threadIdx.x; i < end; i += blockDim.x) {
        const int b = (int)(i / p.T), t = (int)(i % p.T);
        if (t < clamp_len(__ldg(p.lengths + b), p.T)) {
            const double a = (double)p.adv[i];
            s1 += a;
            s2 += a * a;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_red[0][warp] = s1; s_red[1][warp] = s2; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, c = 0.0;
        for (int w = 0; w < kWhitenThreads / 32; ++w) { a += s_red[0][w]; c += s_red[1][w]; }
        p.partials[2 * blockIdx.x] = a;
        p.partials[2 * blockIdx.x + 1] = c;
        __threadfence();
        s_last = (atomicAdd(p.ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    // the last block: number of valid tokens, then mean and 1/sqrt(var + eps)
    long long n = 0;
    for (int b = threadIdx.x; b < p.B; b += blockDim.x) n += clamp_len(__ldg(p.lengths + b), p.T);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    if (lane == 0) s_n[warp] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        long long N = 0;
        for (int w = 0; w < kWhitenThreads / 32; ++w) N += s_n[w];
        double a = 0.0, c = 0.0;
        for (unsigned k = 0; k < gridDim.x; ++k) {
            a += ((volatile double*)p.partials)[2 * k];
            c += ((volatile double*)p.partials)[2 * k + 1];
        }
        float mean = 0.f, rstd = 0.f;
        if (N > 0) {
            const double m = a / (double)N;
            double var = c / (double)N - m * m;
            if (var < 0.0) var = 0.0;
            const double d = var + (double)p.eps;
            mean = (float)m;
            rstd = d > 0.0 ? (float)(1.0 / sqrt(d)) : 0.f;
        }
        p.mean_rstd[0] = mean;
        p.mean_rstd[1] = rstd;
        *p.ticket = 0u;
    }
}

__global__ void __launch_bounds__(256) whiten_apply_kernel(WhitenArgs p)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const float mean = p.mean_rstd[0], rstd = p.mean_rstd[1];
    const long long total = (long long)p.B * p.T;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(i / p.T), t = (int)(i % p.T);
        float w = 0.f;
        if (t < clamp_len(__ldg(p.lengths + b), p.T)) w = (p.adv[i] - mean) * rstd;
        p.out[i] = w;
    }
}

// ---------------------------------------------------------------- monitors of the policy step
// approx_kl = mean over valid tokens of (rho - 1) - log rho, clip_frac = share of valid tokens whose gradient the
// clip switches off (clipped term strictly larger), rho = exp(lp_new - lp_old); from the O(B*T) arrays alone.
// Same fixed-order reduction as the whitening statistics.
struct StatsArgs {
    const float* lp_new;
    const float* lp_old;
    const float* adv;
    const int* lengths;
    int B, T;
    float clip_eps;
    float* out;                 // device float[2]: approx_kl, clip_frac
    unsigned* ticket;
    double* partials;           // workspace: [kWhitenMaxBlocks][2]
};

__global__ void __launch_bounds__(kWhitenThreads) ppo_stats_kernel(StatsArgs p)
{
    __shared__ double s_red[2][kWhitenThreads / 32];
    __shared__ long long s_n[kWhitenThreads / 32];
    __shared__ bool s_last;
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const long long total = (long long)p.B * p.T;
    const long long per_block = (total + gridDim.x - 1) / gridDim.x;
    const long long begin = per_block * blockIdx.x, end = min(total, begin + per_block);
    double s1 = 0.0, s2 = 0.0;
    for (long long i = begin + threadIdx.x; i < end; i += blockDim.x) {
        const int b = (int)(i / p.T), t = (int)(i % p.T);
        if (t < clamp_len(__ldg(p.lengths + b), p.T)) {
            const float d = p.lp_new[i] - p.lp_old[i];
            const float rho = expf(d);
            s1 += (double)((rho - 1.f) - d);
            const float A = p.adv[i];
            const float unclipped = -A * rho;
            const float clipped = -A * fminf(fmaxf(rho, 1.f - p.clip_eps), 1.f + p.clip_eps);
            if (clipped > unclipped) s2 += 1.0;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_red[0][warp] = s1; s_red[1][warp] = s2; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, c = 0.0;
        for (int w = 0; w < kWhitenThreads / 32; ++w) { a += s_red[0][w]; c += s_red[1][w]; }
        p.partials[2 * blockIdx.x] = a;
        p.partials[2 * blockIdx.x + 1] = c;
        __threadfence();
        s_last = (atomicAdd(p.ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    long long n = 0;
    for (int b = threadIdx.x; b < p.B; b += blockDim.x) n += clamp_len(__ldg(p.lengths + b), p.T);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    if (lane == 0) s_n[warp] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        long long N = 0;
        for (int w = 0; w < kWhitenThreads / 32; ++w) N += s_n[w];
        double a = 0.0, c = 0.0;
        for (unsigned k = 0; k < gridDim.x; ++k) {
            a += ((volatile double*)p.partials)[2 * k];
            c += ((volatile double*)p.partials)[2 * k + 1];
        }
        p.out[0] = N > 0 ? (float)(a / (double)N) : 0.f;
        p.out[1] = N > 0 ? (float)(c / (double)N) : 0.f;
        *p.ticket = 0u;
    }
}

// ---------------------------------------------------------------- step 4: finalisation
// Value loss and dvalues per token, then both losses summed in a fixed order: each block reduces a
// contiguous range of tokens with a fixed tree, the last block to finish (a ticket in the workspace)
// adds the block partials in index order.  No floating-point atomics, so the result is bit-stable.
constexpr int kFinalThreads = 256;
constexpr int kFinalMaxBlocks = 256;

struct FinalArgs {
    const int* lengths;
    int B, T;
    const float* values_new;
    const float* values_old;
    const float* returns;
    const float* row_loss;      // per-token policy loss terms written by the row kernel (valid tokens)
    float value_clip, grad_scale;
    float* out_dvalues;
    float* out_lp_new;          // optional: zeroed at padded tokens here
    float* out_loss_pg;
    float* out_loss_vf;
    unsigned* status;
    unsigned* ticket;           // workspace word, zero between calls
    double* partials;           // workspace: [kFinalMaxBlocks][2]
};

__global__ void __launch_bounds__(kFinalThreads) ppo_finalize_kernel(FinalArgs p)
{
    __shared__ long long s_cnt[33];
    __shared__ double s_red[2][kFinalThreads / 32];
    __shared__ bool s_last;
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, nullptr);
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;

    const long long total = (long long)p.B * p.T;
    const long long per_block = (total + gridDim.x - 1) / gridDim.x;
    const long long begin = per_block * blockIdx.x, end = min(total, begin + per_block);
    double sum_pg = 0.0, sum_vf = 0.0;
    for (long long i = begin + threadIdx.x; i < end; i += blockDim.x) {
        int b = (int)(i / p.T), t = (int)(i % p.T);
        float dv = 0.f;
        if (t < clamp_len(__ldg(p.lengths + b), p.T)) {
            float v = p.values_new[i], vo = p.values_old[i], G = p.returns[i];
            float vc = vo + fminf(fmaxf(v - vo, -p.value_clip), p.value_clip);
            float e1 = (v - G) * (v - G), e2 = (vc - G) * (vc - G);
            if (e1 >= e2) { sum_vf += 0.5 * (double)e1; dv = (v - G) * scale_over_N; }
            else sum_vf += 0.5 * (double)e2;
            sum_pg += (double)p.row_loss[i];
        } else if (p.out_lp_new) {
            p.out_lp_new[i] = 0.f;
        }
        p.out_dvalues[i] = dv;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sum_pg += __shfl_xor_sync(0xffffffffu, sum_pg, o);
        sum_vf += __shfl_xor_sync(0xffffffffu, sum_vf, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_red[0][warp] = sum_pg; s_red[1][warp] = sum_vf; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, c = 0.0;
        for (int w = 0; w < kFinalThreads / 32; ++w) { a += s_red[0][w]; c += s_red[1][w]; }
        p.partials[2 * blockIdx.x] = a;
        p.partials[2 * blockIdx.x + 1] = c;
        __threadfence();
        unsigned prev = atomicAdd(p.ticket, 1u);
        s_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (s_last && threadIdx.x == 0) {
        __threadfence();
        double a = 0.0, c = 0.0;
        for (unsigned k = 0; k < gridDim.x; ++k) {
            a += ((volatile double*)p.partials)[2 * k];
            c += ((volatile double*)p.partials)[2 * k + 1];
        }
        *p.out_loss_pg = N > 0 ? (float)(a / (double)N) : 0.f;
        *p.out_loss_vf = N > 0 ? (float)(c / (double)N) : 0.f;
        *p.ticket = 0u;
    }
}

// ---------------------------------------------------------------- step 4: finalisation inside a row kernel
// The same work as ppo_finalize_kernel, done by the row kernel's own blocks: each block takes a
// contiguous slice of the B*T tokens for the value loss (at its start, while its first row is still
// in flight) and sums the policy-loss terms of the rows it processes in the order it processes them
// (the row assignment is static); the last block to finish adds the block partials in index order.
// The value-loss part: one thread's share of the block's slice; writes dvalues (and zeroes lp_new at
// padding) and returns the thread's partial sum of loss terms.
// zero_pad_terms: also writes 0 to the per-token policy loss terms (row_loss) of the padded tokens.
__device__ inline double value_loss_slice(const RowArgs& p, long long N, int tid, int nthreads, bool zero_pad_terms = false)
{
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const long long total = (long long)p.B * p.T;
    const long long per_block = (total + gridDim.x - 1) / gridDim.x;
    const long long begin = per_block * blockIdx.x, end = min(total, begin + per_block);
    double sum_vf = 0.0;
    for (long long i = begin + tid; i < end; i += nthreads) {
        int b = (int)(i / p.T), t = (int)(i % p.T);
        float dv = 0.f;
        if (t < clamp_len(__ldg(p.lengths + b), p.T)) {
            float v = p.values_new[i], vo = p.values_old[i], G = p.returns[i];
            float vc = vo + fminf(fmaxf(v - vo, -p.value_clip), p.value_clip);
            float e1 = (v - G) * (v - G), e2 = (vc - G) * (vc - G);
            if (e1 >= e2) { sum_vf += 0.5 * (double)e1; dv = (v - G) * scale_over_N; }
            else sum_vf += 0.5 * (double)e2;
        } else {
            if (p.out_lp_new) p.out_lp_new[i] = 0.f;
            if (zero_pad_terms) p.row_loss[i] = 0.f;
        }
        p.out_dvalues[i] = dv;
    }
    return sum_vf;
}

// Sum of one double per consumer thread over NW warps (fixed shuffle tree, then warps in index order).
// Uses named barrier 1 with NW*32 threads; s_dbl holds 32 doubles.  Thread 0 gets the total.
template <int NW>
__device__ inline double consumer_sum_double(double v, double* s_dbl, int warp, int lane)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) s_dbl[warp] = v;
    asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
    double tot = 0.0;
    if (warp == 0 && lane == 0)
        for (int w = 0; w < NW; ++w) tot += s_dbl[w];
    return tot;
}

// Called by consumer thread 0 of every block when the block has finished its rows: publishes the
// block's two partial sums; the last block to arrive adds all of them in index order and writes the
// two losses.
__device__ inline void publish_block_losses(const RowArgs& p, long long N, double sum_pg, double sum_vf)
{
    p.partials[2 * blockIdx.x] = sum_pg;
    p.partials[2 * blockIdx.x + 1] = sum_vf;
    __threadfence();
    const unsigned prev = atomicAdd(p.ticket, 1u);
    if (prev == gridDim.x - 1) {
        __threadfence();
        double a = 0.0, c = 0.0;
        for (unsigned k = 0; k < gridDim.x; ++k) {
            a += ((volatile double*)p.partials)[2 * k];
            c += ((volatile double*)p.partials)[2 * k + 1];
        }
        *p.out_loss_pg = N > 0 ? (float)(a / (double)N) : 0.f;
        *p.out_loss_vf = N > 0 ? (float)(c / (double)N) : 0.f;
        *p.ticket = 0u;
    }
}

}  // namespace rlhf
