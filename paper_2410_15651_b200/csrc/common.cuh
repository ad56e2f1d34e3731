// Shared device helpers for the token-level PPO kernels (sm_100a).
//
// Softmax arithmetic is done in base 2: x = z * log2(e), partition sums are kept as
// (M, s) with  sum_v 2^(x_v) = s * 2^M,  so that one ex2 per element is the only special-function
// work.  The generated token's own term is kept apart (ey) so that 1 - p_y = s / (s + ey) is
// formed without cancellation when the distribution is peaked.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace rlhf {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kFloorM = -1.0e38f;        // reference exponent of an empty partial sum
constexpr float kRebase = 64.0f;           // raise the reference when a term would exceed 2^64

// status flags kept in word 0 of the workspace (values of rlhf_status_t)
constexpr unsigned kErrIdRange = 16u;
constexpr unsigned kErrLengthRange = 32u;
constexpr unsigned kErrTimeout = 64u;

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic stream
// serialisation allowed: its blocks may become resident while the kernel before it in the stream is
// still draining, set up their shared memory and barriers, and then wait here, before their first
// access to global memory, until that kernel has completed and its writes are visible.  Under a plain
// launch, or behind work that is not a kernel, the wait returns at once.
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream begin its own set-up as soon as this kernel's blocks leave room.
__device__ __forceinline__ void pdl_release_next_grid() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }

__device__ __forceinline__ float2 unpack_bf16x2(uint32_t w) { return make_float2(bf16_lo(w), bf16_hi(w)); }

// The 16-bit element type of the logits and of their gradient: bf16 (kF16 = false) or IEEE binary16 (true).
// Widening is exact; narrowing rounds to nearest even (and, for binary16, overflows to infinity above 65504).
template <bool kF16>
struct El {
    static constexpr uint32_t kNegInf = kF16 ? 0xfc00u : 0xff80u;       // bit pattern of -inf
    static constexpr uint32_t kNegInf2 = kNegInf | (kNegInf << 16);     // two of them
    __device__ __forceinline__ static float widen(uint32_t bits16)
    {
        if (!kF16) return __uint_as_float(bits16 << 16);
        float f;
        asm("{\n\t.reg .b16 h;\n\tcvt.u16.u32 h, %1;\n\tcvt.f32.f16 %0, h;\n\t}" : "=f"(f) : "r"(bits16));
        return f;
    }
    __device__ __forceinline__ static float2 unpack2(uint32_t w)
    {
        if (!kF16) return make_float2(bf16_lo(w), bf16_hi(w));
        float2 r;
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}"
            : "=f"(r.x), "=f"(r.y) : "r"(w));
        return r;
    }
    __device__ __forceinline__ static uint32_t pack2(float lo, float hi)
    {
        uint32_t r;
        if (!kF16) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        else asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
};

// Partial partition sum in the base-2 domain.
struct Acc {
    float M;     // reference exponent
    float s;     // sum over all entries but the generated token of 2^(x - M)
    float ey;    // 2^(x_y - M) if this partial sum has seen the generated token, else 0
};

__device__ __forceinline__ Acc acc_empty() { return Acc{kFloorM, 0.f, 0.f}; }

__device__ __forceinline__ void acc_rebase(Acc& a, float newM)
{
    float sc = ex2(a.M - newM);
    a.s *= sc;
    a.ey *= sc;
    a.M = newM;
}

// One element, any order; used by the scalar kernels.
__device__ __forceinline__ void acc_add(Acc& a, float z, bool is_label)
{
    float x = z * kLog2e;
    if (x - a.M > kRebase) acc_rebase(a, x);
    float e = ex2(x - a.M);
    if (is_label) a.ey = e; else a.s += e;
}

__device__ __forceinline__ Acc acc_merge(const Acc& a, const Acc& b)
{
    Acc r;
    r.M = fmaxf(a.M, b.M);
    float sa = ex2(a.M - r.M), sb = ex2(b.M - r.M);
    r.s = a.s * sa + b.s * sb;
    r.ey = a.ey * sa + b.ey * sb;
    return r;
}

__device__ __forceinline__ Acc acc_warp_reduce(Acc a)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Acc b;
        b.M = __shfl_xor_sync(0xffffffffu, a.M, o);
        b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
        b.ey = __shfl_xor_sync(0xffffffffu, a.ey, o);
        a = acc_merge(a, b);
    }
    return a;
}

// What one row needs after its partition sum is known.
struct RowResult {
    float lse2;      // log2 sum_v 2^(x_v)
    float lp;        // z_y - ln sum_v e^(z_v)
    float one_m_py;  // 1 - p_y
};

__device__ __forceinline__ RowResult row_finish(const Acc& a, float zy)
{
    RowResult r;
    float tot = a.s + a.ey;
    r.lse2 = a.M + log2f(tot);
    r.lp = zy - r.lse2 * kLn2;
    r.one_m_py = a.s / tot;
    return r;
}

__device__ __forceinline__ float lg2(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Same as row_finish with the hardware lg2/rcp (relative error about 2^-22): a short dependent
// chain, for kernels in which a whole block waits on these scalars once per row.
__device__ __forceinline__ RowResult row_finish_fast(const Acc& a, float zy)
{
    RowResult r;
    float tot = a.s + a.ey;
    r.lse2 = a.M + lg2(tot);
    r.lp = fmaf(-r.lse2, kLn2, zy);
    r.one_m_py = __fdividef(a.s, tot);
    return r;
}

// Clipped-surrogate terms of one token: loss and g = d(grad_scale * loss / N) / d lp_new.
template <bool kFast = false>
__device__ __forceinline__ void ppo_token(float lp_new, float lp_old, float A, float clip_eps,
                                          float scale_over_N, float& loss, float& g)
{
    float rho = kFast ? ex2((lp_new - lp_old) * kLog2e) : expf(lp_new - lp_old);
    float unclipped = -A * rho;
    float clipped = -A * fminf(fmaxf(rho, 1.f - clip_eps), 1.f + clip_eps);
    if (unclipped >= clipped) { loss = unclipped; g = unclipped * scale_over_N; }
    else { loss = clipped; g = 0.f; }
}

// Walks the flattened list of valid (or padded) tokens in increasing order.  item k of the valid
// list is the k-th (b,t) with t < len_b in row-major order; of the padded list, the k-th with
// t >= len_b.  Lengths are clamped to [0,T].
struct Cursor {
    int b;
    long long acc;   // number of listed tokens in sequences before b
};

__device__ __forceinline__ int clamp_len(int len, int T) { return len < 0 ? 0 : (len > T ? T : len); }

__device__ __forceinline__ bool cursor_seek_valid(Cursor& c, long long k, const int* __restrict__ lengths,
                                                  int B, int T, int& b, int& t)
{
    while (c.b < B) {
        int len = clamp_len(__ldg(lengths + c.b), T);
        if (k < c.acc + len) { b = c.b; t = (int)(k - c.acc); return true; }
        c.acc += len;
        ++c.b;
    }
    return false;
}

__device__ __forceinline__ bool cursor_seek_padded(Cursor& c, long long k, const int* __restrict__ lengths,
                                                   int B, int T, int& b, int& t)
{
    while (c.b < B) {
        int len = clamp_len(__ldg(lengths + c.b), T);
        int pad = T - len;
        if (k < c.acc + pad) { b = c.b; t = len + (int)(k - c.acc); return true; }
        c.acc += pad;
        ++c.b;
    }
    return false;
}

// Which padded rows a block zero-fills.  Valid rows are dealt round-robin, so the first N % G blocks have
// one valid row more than the others; a valid row moves twice the bytes of a padded one (read + write
// against write only), so the other blocks first receive up to two padded rows each, and what is left is
// dealt evenly.  Block i takes the contiguous range [start, start + count) of the padded-token list.
struct PadShare {
    long long start, count;
};

__host__ __device__ inline PadShare pad_share(long long N, long long n_pad, long long G, long long i)
{
    const long long r = N % G;                  // blocks [0, r) hold the extra valid row
    const long long lows = G - r;               // >= 1
    const long long level = n_pad < 2 * lows ? n_pad : 2 * lows;
    const long long rest = n_pad - level;
    const long long lq = level / lows, lr = level % lows, eq = rest / G, er = rest % G;
    const long long j = i - r;                  // position among the lows (if >= 0)
    PadShare s;
    s.count = (j >= 0 ? lq + (j < lr ? 1 : 0) : 0) + eq + (i < er ? 1 : 0);
    s.start = (j > 0 ? j * lq + (j < lr ? j : lr) : 0) + i * eq + (i < er ? i : er);
    return s;
}

// Sum of clamped lengths over the batch, by the whole block; flags out-of-range lengths.
// `scratch` is 33 long longs of shared memory.  Every thread returns the total.
__device__ inline long long block_count_valid(const int* __restrict__ lengths, int B, int T,
                                              long long* scratch, unsigned* status)
{
    long long n = 0;
    bool bad = false;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        int len = __ldg(lengths + b);
        bad |= (len < 0 || len > T);
        n += clamp_len(len, T);
    }
    if (bad && status) atomicOr(status, kErrLengthRange);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    if (lane == 0) scratch[warp] = n;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < nw; ++w) tot += scratch[w];
        scratch[32] = tot;
    }
    __syncthreads();
    return scratch[32];
}

}  // namespace rlhf
