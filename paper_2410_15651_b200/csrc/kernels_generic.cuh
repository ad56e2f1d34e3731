// Row kernels for any layout: element-wise global loads and stores, no alignment requirement.
// They serve rows that the 16-byte fast path cannot take (odd V, odd strides, odd base address).
// One block walks the valid rows k = blockIdx.x, blockIdx.x + gridDim.x, ...; each row is read
// from global memory (twice in the loss kernel: once for the partition sum, once for the gradient,
// the second read coming from L2).
#pragma once
#include "common.cuh"

namespace rlhf {

struct RowArgs {
    const uint16_t* logits;     // bf16 bit patterns
    long long stride_b, stride_t;
    const long long* ids;
    long long ids_stride_b;
    const int* lengths;
    int B, T, V;
    unsigned* status;           // workspace word 0
    unsigned long long wait_limit_ns;   // bound of every wait on a shared-memory barrier (row kernels with a producer)
    // step 1
    float* out_lp;
    // step 4
    const float* lp_old;
    const float* adv;
    float clip_eps, grad_scale;
    uint16_t* dlogits;
    long long dl_stride_b, dl_stride_t;
    float* row_loss;            // workspace: per-token policy loss term
    float* out_lp_new;          // optional
    // step 4, finalisation fused into the row kernel (fused != 0): value loss, dvalues and both scalar losses
    int fused;
    const float* values_new;
    const float* values_old;
    const float* returns;
    float value_clip;
    float* out_dvalues;
    float* out_loss_pg;
    float* out_loss_vf;
    unsigned* ticket;           // workspace word 1, zero between calls
    double* partials;           // workspace: [gridDim.x][2] block partial sums (policy, value)
};

constexpr int kGenericThreads = 256;

// Block-wide merge of per-thread partial sums; every thread returns the total.
__device__ inline Acc block_merge(Acc a, Acc* smem /* >= 32 */)
{
    a = acc_warp_reduce(a);
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();                 // smem free from the previous row
    if (lane == 0) smem[warp] = a;
    __syncthreads();
    Acc r = smem[0];
    for (int w = 1; w < nw; ++w) r = acc_merge(r, smem[w]);
    return r;
}

// kF16: logits and gradient are IEEE binary16 instead of bf16.
template <bool kLoss, bool kF16 = false>
__global__ void __launch_bounds__(kGenericThreads) row_generic_kernel(RowArgs p)
{
    __shared__ Acc s_acc[32];
    __shared__ long long s_cnt[33];
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;

    Cursor cur{0, 0};
    for (long long k = blockIdx.x; k < N; k += gridDim.x) {
        int b, t;
        if (!cursor_seek_valid(cur, k, p.lengths, p.B, p.T, b, t)) break;
        const long long flat = (long long)b * p.T + t;
        long long y = __ldg(p.ids + (long long)b * p.ids_stride_b + t);
        const bool bad_id = (y < 0 || y >= p.V);
        if (bad_id) { y = 0; if (threadIdx.x == 0) atomicOr(p.status, kErrIdRange); }
        const uint16_t* row = p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t;

        // every thread reads z_y before the block barrier, i.e. before any in-place write of this row
        const float zy = El<kF16>::widen(row[y]);
        Acc a = acc_empty();
        for (int v = threadIdx.x; v < p.V; v += blockDim.x)
            acc_add(a, El<kF16>::widen(row[v]), v == (int)y);
        a = block_merge(a, s_acc);
        RowResult r = row_finish(a, zy);

        if (!kLoss) {
            if (threadIdx.x == 0) p.out_lp[flat] = bad_id ? 0.f : r.lp;
            continue;
        }
        float loss = 0.f, g = 0.f;
        if (!bad_id) ppo_token(r.lp, p.lp_old[flat], p.adv[flat], p.clip_eps, scale_over_N, loss, g);
        if (threadIdx.x == 0) {
            p.row_loss[flat] = loss;
            if (p.out_lp_new) p.out_lp_new[flat] = bad_id ? 0.f : r.lp;
        }
        uint16_t* drow = p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t;
        if (g == 0.f) {
            for (int v = threadIdx.x; v < p.V; v += blockDim.x) drow[v] = 0;
        } else {
            // |g| * p_v = 2^(x_v - lse2 + log2|g|); the sign is applied to the packed result
            const float c2 = log2f(fabsf(g)) - r.lse2;
            const uint16_t sign = g > 0.f ? 0x8000u : 0u;
            for (int v = threadIdx.x; v < p.V; v += blockDim.x) {
                float z = El<kF16>::widen(row[v]);                    // read before the in-place write
                float d = ex2(fmaf(z, kLog2e, c2));
                uint16_t h = (uint16_t)(El<kF16>::pack2(d, 0.f) & 0xffffu) ^ sign;
                if (v == (int)y) h = (uint16_t)(El<kF16>::pack2(g * r.one_m_py, 0.f) & 0xffffu);
                drow[v] = h;
            }
        }
    }

    if (kLoss) {
        // zero rows for padded tokens
        const long long n_pad = (long long)p.B * p.T - N;
        Cursor pc{0, 0};
        for (long long k = blockIdx.x; k < n_pad; k += gridDim.x) {
            int b, t;
            if (!cursor_seek_padded(pc, k, p.lengths, p.B, p.T, b, t)) break;
            uint16_t* drow = p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t;
            for (int v = threadIdx.x; v < p.V; v += blockDim.x) drow[v] = 0;
        }
    } else {
        // log-prob 0 at padded tokens
        const long long total = (long long)p.B * p.T;
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
             i += (long long)gridDim.x * blockDim.x) {
            int b = (int)(i / p.T), t = (int)(i % p.T);
            if (t >= clamp_len(__ldg(p.lengths + b), p.T)) p.out_lp[i] = 0.f;
        }
    }
}

}  // namespace rlhf
