// Loss row kernel with a ring of shared-memory chunks, for 16-byte aligned rows outside the range of
// the kernel that keeps a row's exponentials on chip (sm_100a): rows shorter than 16 KB, and rows beyond
// what a cluster of four blocks holds; also the PTX wrappers and per-vector arithmetic that the other row
// kernels share.
//
// Each persistent block owns a ring of 4/8/32 KB slots.  One elected producer thread streams the
// block's rows into the ring with bulk asynchronous copies (cp.async.bulk, completion counted on an
// mbarrier per slot); NW consumer warps work on the slots as they land and release them through a
// second mbarrier per slot.
//
//   short rows (< 16 KB)     blocks of 8 consumer warps, up to 7 per SM; the row stays in the ring
//                            ("resident") between the partition-sum pass and the gradient pass.
//   rows beyond a cluster    streamed twice by one block of 16 consumer warps per SM; the second read
//                            is served by L2.
//   Padded rows are zero-filled by bulk stores from a zeroed shared buffer, issued by the producer
//   thread between its loads.
//
// Work assignment is static: block i takes valid rows i, i+G, i+2G, ... (and padded rows likewise),
// so results never depend on timing.  Every wait on an mbarrier is bounded; if one runs out the
// thread flags RLHF_ERR_TIMEOUT, stops waiting and lets the block drain.
#pragma once
#include "common.cuh"
#include "kernels_generic.cuh"
#include "kernels_small.cuh"

namespace rlhf {

constexpr int kZeroBytes = 4096;                       // zeroed buffer that feeds the bulk zero-fill
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default bound of a barrier wait: 2 s

struct RingArgs {
    RowArgs row;
    int n_slots;          // ring size in chunks
    int chunks_per_row;   // ceil(row_bytes / chunk_bytes)
    int resident;         // loss kernel: the row stays in the ring between the two passes
    unsigned row_bytes;   // 2*V, a multiple of 16
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false (after flagging the status word) if the phase did not complete in time.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, unsigned* status, unsigned long long limit_ns)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) {
            atomicOr(status, kErrTimeout);
            return false;
        }
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, unsigned* status, bool& aborted,
                                          unsigned long long limit_ns)
{
    if (aborted) return;
    if (mbar_try_wait(bar, parity)) return;
    if (!mbar_wait_slow(bar, parity, status, limit_ns)) aborted = true;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void store_v4(void* p, const uint4& q)
{
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(q.x), "r"(q.y), "r"(q.z), "r"(q.w)
                 : "memory");
}

// One block of one warp that waits, with the bounded wait every pipelined kernel of the library uses, on a
// shared-memory barrier at which nobody ever arrives: the wait runs out after `limit_ns`, the status word gets
// RLHF_ERR_TIMEOUT and the kernel returns.  It exists so that the give-up path can be exercised without a fault.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(unsigned* status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long s_bar;
    const uint32_t bar = smem_u32(&s_bar);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    __syncwarp();
    bool aborted = false;
    mbar_wait(bar, 0u, status, aborted, limit_ns);
    // (aborted is true here on every thread; nothing else to release)
}

// ---------------------------------------------------------------- 8 logits at a time
template <bool kF16 = false>
__device__ __forceinline__ void unpack8(const uint4& q, float (&z)[8])
{
    const float2 a = El<kF16>::unpack2(q.x), b = El<kF16>::unpack2(q.y), c = El<kF16>::unpack2(q.z), d = El<kF16>::unpack2(q.w);
    z[0] = a.x; z[1] = a.y;
    z[2] = b.x; z[3] = b.y;
    z[4] = c.x; z[5] = c.y;
    z[6] = d.x; z[7] = d.y;
}

// Adds 8 entries none of which is the generated token.  The exponentials are formed against the
// thread's current reference first; only if their sum is out of range (first vector of a thread, or
// a logit more than 64 binades above the reference) is the reference raised and the vector redone.
template <bool kF16 = false>
__device__ __forceinline__ void acc_add_vec(Acc& a, const uint4& q)
{
    float z[8], e[8];
    unpack8<kF16>(q, z);
    float negM = -a.M;
#pragma unroll
    for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(z[i], kLog2e, negM));
    float vs = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
    if (!(vs <= 1.8446744e19f)) {
        float vm = kFloorM;
#pragma unroll
        for (int i = 0; i < 8; ++i) vm = fmaxf(vm, z[i] * kLog2e);
        acc_rebase(a, vm);
        negM = -a.M;
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(z[i], kLog2e, negM));
        vs = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
    }
    a.s += vs;
}

// The vector that holds the generated token (entry j): its term goes to a.ey; returns z_y.
template <bool kF16 = false>
__device__ __forceinline__ float acc_add_vec_label(Acc& a, const uint4& q, int j)
{
    float z[8];
    unpack8<kF16>(q, z);
    float zy = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        acc_add(a, z[i], i == j);
        if (i == j) zy = z[i];
    }
    return zy;
}

// A vector of which only entries jlo <= j < jhi belong to the row (the first or last vector of a row that
// does not start or end on a 16-byte boundary); entry jlabel, if in range, is the generated token.
template <bool kF16 = false>
__device__ __forceinline__ float acc_add_vec_range(Acc& a, const uint4& q, int jlo, int jhi, int jlabel)
{
    float z[8];
    unpack8<kF16>(q, z);
    float zy = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i >= jlo && i < jhi) {
            acc_add(a, z[i], i == jlabel);
            if (i == jlabel) zy = z[i];
        }
    }
    return zy;
}

// Entries of a vector outside [jlo, jhi) replaced by -inf: they then add nothing to a partition sum.
// For the first or last vector of a row that does not start or end on a 16-byte boundary.
template <bool kF16 = false>
__device__ __forceinline__ uint4 mask_vec_outside(const uint4& q, int jlo, int jhi)
{
    uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i < jlo || i >= jhi)
            w[i >> 1] = (i & 1) ? ((w[i >> 1] & 0x0000ffffu) | (El<kF16>::kNegInf << 16)) : ((w[i >> 1] & 0xffff0000u) | El<kF16>::kNegInf);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// dlogits for 8 entries: sign * 2^(x + c2), packed to bf16.  The scaling runs two entries at a time on
// the packed fp32x2 FMA of sm_100; the exponentials stay on the special-function unit.
template <bool kF16 = false>
__device__ __forceinline__ uint4 grad_vec(const uint4& q, float c2, uint32_t sign2)
{
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 x = __ffma2_rn(El<kF16>::unpack2(w[k]), splat2(kLog2e), splat2(c2));
        o[k] = El<kF16>::pack2(ex2(x.x), ex2(x.y)) ^ sign2;
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

template <int U, bool kF16 = false>
__device__ __forceinline__ void grad_vecs(const uint4 (&q)[U], uint4 (&o)[U], float c2, uint32_t sign2)
{
#pragma unroll
    for (int u = 0; u < U; ++u) o[u] = grad_vec<kF16>(q[u], c2, sign2);
}

template <bool kF16 = false>
__device__ __forceinline__ void patch_label(uint4& o, int j, float value)
{
    const uint32_t h = El<kF16>::pack2(value, 0.f) & 0xffffu;
    const int ws = j >> 1;
    uint32_t w = ws == 0 ? o.x : (ws == 1 ? o.y : (ws == 2 ? o.z : o.w));
    w = (j & 1) ? ((w & 0x0000ffffu) | (h << 16)) : ((w & 0xffff0000u) | h);
    o.x = ws == 0 ? w : o.x;
    o.y = ws == 1 ? w : o.y;
    o.z = ws == 2 ? w : o.z;
    o.w = ws == 3 ? w : o.w;
}

// ---------------------------------------------------------------- block-wide merge of partial sums
// What the owner of the generated token's vector publishes for the row.
struct LabelInfo {
    float zy;    // the generated token's logit
    float ey;    // 2^(x_y - M) against the owner thread's final reference
    float M;     // that reference
    float pad;
};

// Merges the per-thread partial sums of NW consumer warps.  Each warp first agrees on a common
// reference (max by shuffles), rescales once and adds; lane 0 publishes (M, s); after the consumer
// barrier the same is done across warps with one partial per lane.  The generated token's own term
// comes from the LabelInfo its owner thread wrote before the barrier.  Every thread returns the total.
template <int NW>
__device__ __forceinline__ Acc consumer_reduce(const Acc& a, float2* s_part, const LabelInfo* s_lab,
                                               int warp, int lane)
{
    float M = a.M;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float s = a.s * ex2(a.M - M);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) s_part[warp] = make_float2(M, s);
    asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
    const float2 pw = lane < NW ? s_part[lane] : make_float2(kFloorM, 0.f);
    float Mt = pw.x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Mt = fmaxf(Mt, __shfl_xor_sync(0xffffffffu, Mt, o));
    float st = pw.y * ex2(pw.x - Mt);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st += __shfl_xor_sync(0xffffffffu, st, o);
    const LabelInfo li = *s_lab;
    Acc tot;
    tot.M = fmaxf(Mt, li.M);
    tot.s = st * ex2(Mt - tot.M);
    tot.ey = li.ey * ex2(li.M - tot.M);
    return tot;
}

// Barrier over the NW consumer warps (named barrier 1) that also tells every thread whether `flag` was
// set in any of them.
template <int NW>
__device__ __forceinline__ bool consumer_barrier_or(bool flag)
{
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(any) : "r"((uint32_t)flag), "n"(NW * 32) : "memory");
    return any != 0;
}

// Sum of the NW warp sums published in `s_sum` (16-byte aligned), added by every thread in the same fixed tree.
template <int NW>
__device__ __forceinline__ float sum_warp_sums(const float* s_sum)
{
    // (the array is read in whole float4s: it holds a multiple of 4 floats, of which the first NW are used)
    float v[(NW + 3) / 4 * 4];
#pragma unroll
    for (int w4 = 0; w4 < (NW + 3) / 4; ++w4) {
        const float4 t4 = ((const float4*)s_sum)[w4];
        v[4 * w4] = t4.x; v[4 * w4 + 1] = t4.y; v[4 * w4 + 2] = t4.z; v[4 * w4 + 3] = t4.w;
    }
#pragma unroll
    for (int st = 1; st < NW; st <<= 1)
#pragma unroll
        for (int w = 0; w + st < NW; w += 2 * st) v[w] += v[w + st];
    return v[0];
}

// ---------------------------------------------------------------- the kernel
// Sum of the exponentials of U vectors against one reference exponent (no range check): scaling and
// accumulation two entries at a time (packed fp32x2), one ex2 per entry.
template <int U, bool kF16 = false>
__device__ __forceinline__ float exp_sum_vecs(const uint4 (&q)[U], float negM)
{
    float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 x = __ffma2_rn(El<kF16>::unpack2(w[k]), splat2(kLog2e), splat2(negM));
            acc[k & 1] = __fadd2_rn(acc[k & 1], make_float2(ex2(x.x), ex2(x.y)));
        }
    }
    return (acc[0].x + acc[0].y) + (acc[1].x + acc[1].y);
}

template <bool kF16 = false>
__device__ __forceinline__ float max8_scaled(const uint4& q)
{
    float z[8];
    unpack8<kF16>(q, z);
    float m = fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7])));
    return fmaxf(m * kLog2e, kFloorM);
}

// Dynamic shared memory: [n_slots * chunk][full barriers n_slots * 8][empty barriers n_slots * 8][zero buffer].
// NW consumer warps + 1 producer warp; a chunk is NW*32*U 16-byte vectors.
template <int NW, int U>
__global__ void __launch_bounds__(NW * 32 + 32, NW == 16 ? 1 : 3) row_ring_kernel(RingArgs ra)
{
    constexpr int kCons = NW * 32;
    constexpr int kThreads = kCons + 32;
    constexpr uint32_t kChunkVecs = (uint32_t)kCons * U;
    constexpr uint32_t kChunk = kChunkVecs * 16u;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ float2 s_part[2][32];
    __shared__ __align__(16) float s_sum[2][NW];
    __shared__ LabelInfo s_lab[2];
    __shared__ double s_dbl[32];

    const RowArgs& p = ra.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = ra.n_slots, chunks = ra.chunks_per_row;
    const uint32_t slots_addr = smem_u32(smem);
    const uint32_t full_addr = slots_addr + (uint32_t)S * kChunk;
    const uint32_t empty_addr = full_addr + (uint32_t)S * 8u;
    unsigned char* zero_buf = smem + (size_t)S * kChunk + (size_t)S * 16;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_addr + 8u * s, 1);
            mbar_init(empty_addr + 8u * s, NW);
        }
        fence_mbar_init();
    }
    for (int i = tid; i < kZeroBytes / 16; i += kThreads) ((uint4*)zero_buf)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    __syncthreads();
    pdl_wait_prior_grid();                       // nothing above touches global memory
    pdl_release_next_grid();

    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const long long G = gridDim.x;

    bool aborted = false;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        if (lane != 0) return;
        const long long n_pad = (long long)p.B * p.T - N;
        const long long rows_mine = N > blockIdx.x ? (N - blockIdx.x + G - 1) / G : 0;
        const PadShare pads = pad_share(N, n_pad, G, blockIdx.x);
        const long long pads_mine = pads.count;
        Cursor cur{0, 0}, pcur{0, 0};
        long long pads_done = 0;
        auto zero_fill_next = [&]() {
            int b, t;
            if (!cursor_seek_padded(pcur, pads.start + pads_done, p.lengths, p.B, p.T, b, t)) return;
            unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t);
            for (uint32_t off = 0; off < ra.row_bytes; off += kZeroBytes)
                bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kZeroBytes, ra.row_bytes - off));
            bulk_commit();
        };
        int slot = 0;
        uint32_t phase = 0;
        const int loads_per_row = (!ra.resident) ? 2 * chunks : chunks;
        long long i = 0;
        for (long long k = blockIdx.x; k < N && !aborted; k += G, ++i) {
            int b, t;
            if (!cursor_seek_valid(cur, k, p.lengths, p.B, p.T, b, t)) break;
            const unsigned char* row = (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t);
            for (int j = 0; j < loads_per_row; ++j) {
                const int c = j >= chunks ? j - chunks : j;
                mbar_wait(empty_addr + 8u * slot, phase ^ 1u, p.status, aborted, p.wait_limit_ns);
                if (aborted) break;
                const uint32_t off = (uint32_t)c * kChunk;
                const uint32_t bytes = min(kChunk, ra.row_bytes - off);
                mbar_arrive_expect_tx(full_addr + 8u * slot, bytes);
                bulk_load(slots_addr + (uint32_t)slot * kChunk, row + off, bytes, full_addr + 8u * slot);
                if (++slot == S) { slot = 0; phase ^= 1u; }
            }
            {
                const long long target = ((i + 1) * pads_mine) / rows_mine;
                while (pads_done < target) { zero_fill_next(); ++pads_done; }
            }
        }
        while (pads_done < pads_mine) { zero_fill_next(); ++pads_done; }
        bulk_wait_all();
        return;
    }

    // ---------------------------------------------------------------- consumers
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const uint32_t nvec = ra.row_bytes / 16u;
    const int full_chunks = (int)(nvec / kChunkVecs);          // chunks in which every vector exists
    double sum_pg = 0.0, sum_vf = 0.0;                         // block partial sums (thread 0)
    if (p.fused) sum_vf = consumer_sum_double<NW>(value_loss_slice(p, N, tid, kCons), s_dbl, warp, lane);

    Cursor cur{0, 0};
    int slot = 0;
    uint32_t phase = 0;
    int par = 0;

    // scalars of the row about to be processed (loaded one row ahead)
    int nb = 0, nt = 0;
    long long ny = 0;
    float n_lp_old = 0.f, n_adv = 0.f;
    auto fetch_row = [&](long long k) {
        if (k < N && cursor_seek_valid(cur, k, p.lengths, p.B, p.T, nb, nt)) {
            ny = __ldg(p.ids + (long long)nb * p.ids_stride_b + nt);
            const long long f = (long long)nb * p.T + nt;
            n_lp_old = __ldg(p.lp_old + f);
            n_adv = __ldg(p.adv + f);
        }
    };
    fetch_row(blockIdx.x);

    for (long long k = blockIdx.x; k < N; k += G, par ^= 1) {
        const int b = nb, t = nt;
        long long y = ny;
        const float lp_old = n_lp_old, adv = n_adv;
        const long long flat = (long long)b * p.T + t;
        const bool bad_id = (y < 0 || y >= p.V);
        if (bad_id) { y = 0; if (tid == 0) atomicOr(p.status, kErrIdRange); }
        const uint32_t yvec = (uint32_t)(y >> 3);
        const int yj = (int)(y & 7);
        const int ychunk = (int)(yvec / kChunkVecs);

        const int slot0 = slot;
        const uint32_t phase0 = phase;

        // ---- pass 1: partition sum
        // Every thread starts from the same reference exponent (the scaled maximum of the row's first vector), so
        // that the block's partial sums add up without rescaling unless some thread had to raise its reference.
        Acc a = acc_empty();
        float zy = 0.f;
        float Mref = kFloorM;
        const bool owner = (yvec % kCons) == (uint32_t)tid;      // this thread sums the generated token's vector
        for (int c = 0; c < chunks; ++c) {
            mbar_wait(full_addr + 8u * slot, phase, p.status, aborted, p.wait_limit_ns);
            const uint4* src = (const uint4*)(smem + (size_t)slot * kChunk) + tid;
            if (c == 0) {
                Mref = max8_scaled(*(const uint4*)(smem + (size_t)slot * kChunk));
                if (Mref > kFloorM) a.M = Mref;
            }
            if (c < full_chunks && c != ychunk) {
                // common case: every vector exists and none holds the generated token
                uint4 q[U];
#pragma unroll
                for (int u = 0; u < U; ++u) q[u] = src[u * kCons];
                const float vs = exp_sum_vecs<U>(q, -a.M);
                if (vs <= 1.8446744e19f) {
                    a.s += vs;
                } else {
                    // a logit far above the reference (or a non-finite sum): redo with range handling
#pragma unroll
                    for (int u = 0; u < U; ++u) acc_add_vec(a, q[u]);
                }
            } else {
                const uint32_t v0 = (uint32_t)c * kChunkVecs + tid;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t v = v0 + u * kCons;
                    if (v < nvec) {
                        const uint4 q = src[u * kCons];
                        if (v == yvec) zy = acc_add_vec_label(a, q, yj);
                        else acc_add_vec(a, q);
                    }
                }
            }
            if (!ra.resident) {
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_addr + 8u * slot);
            }
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
        if (owner) s_lab[par] = LabelInfo{zy, a.ey, a.M, 0.f};
        float ws = a.s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
        if (lane == 0) s_sum[par][warp] = ws;
        Acc tot;
        if (!consumer_barrier_or<NW>(a.M != Mref)) {
            tot.M = Mref;
            tot.s = sum_warp_sums<NW>(s_sum[par]);
            tot.ey = s_lab[par].ey;
        } else {
            tot = consumer_reduce<NW>(a, s_part[par], &s_lab[par], warp, lane);
        }
        const RowResult r = row_finish(tot, s_lab[par].zy);

        // scalars of the next row, in flight while this row is finished
        fetch_row(k + G);

        float loss = 0.f, g = 0.f;
        if (!bad_id) ppo_token(r.lp, lp_old, adv, p.clip_eps, scale_over_N, loss, g);
        if (tid == 0) {
            if (p.fused) sum_pg += (double)loss; else p.row_loss[flat] = loss;
            if (p.out_lp_new) p.out_lp_new[flat] = bad_id ? 0.f : r.lp;
        }

        // ---- pass 2: dlogits
        if (ra.resident) { slot = slot0; phase = phase0; }
        unsigned char* dst = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t) +
                             (size_t)tid * 16;
        const float c2 = log2f(fabsf(g)) - r.lse2;
        const uint32_t sign2 = g > 0.f ? 0x80008000u : 0u;
        const float dy = g * r.one_m_py;
        for (int c = 0; c < chunks; ++c, dst += kChunk) {
            if (!ra.resident) mbar_wait(full_addr + 8u * slot, phase, p.status, aborted, p.wait_limit_ns);
            const uint4* src = (const uint4*)(smem + (size_t)slot * kChunk) + tid;
            if (c < full_chunks && c != ychunk && g != 0.f) {
                uint4 q[U];
#pragma unroll
                for (int u = 0; u < U; ++u) q[u] = src[u * kCons];
                uint4 o[U];
                grad_vecs<U>(q, o, c2, sign2);
#pragma unroll
                for (int u = 0; u < U; ++u) store_v4(dst + (size_t)u * kCons * 16, o[u]);
            } else {
                const uint32_t v0 = (uint32_t)c * kChunkVecs + tid;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t v = v0 + u * kCons;
                    if (v < nvec) {
                        uint4 o = make_uint4(0, 0, 0, 0);
                        if (g != 0.f) {
                            o = grad_vec(src[u * kCons], c2, sign2);
                            if (v == yvec) patch_label(o, yj, dy);
                        }
                        store_v4(dst + (size_t)u * kCons * 16, o);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_addr + 8u * slot);
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
    }
    if (p.fused && tid == 0) publish_block_losses(p, N, sum_pg, sum_vf);
}

// ---------------------------------------------------------------- host-side plan
struct RingPlan {
    int NW = 0;                // consumer warps per block (8 or 16); 0 = not applicable
    int U = 0;                 // 16-byte vectors per consumer thread per chunk (1 or 2)
    int n_slots = 0;
    int chunks_per_row = 0;
    int resident = 0;
    int blocks_per_sm = 0;
    size_t smem_bytes = 0;
};

inline size_t ring_smem_bytes(int NW, int U, int n_slots)
{
    return (size_t)n_slots * ((size_t)NW * 32 * 16 * U) + (size_t)n_slots * 16 + kZeroBytes;
}

// Chooses block shape, chunk size, ring depth and blocks per SM for rows of `row_bytes`.
// sm_smem: shared memory per SM; block_smem_max: opt-in maximum per block.  The system reserves
// 1 KB per resident block.
inline RingPlan plan_ring(unsigned row_bytes, int sm_smem, int block_smem_max)
{
    constexpr size_t kStatic = 1280;                   // static shared memory of the kernel, rounded up
    constexpr size_t kReserved = 1024;
    if (row_bytes < 32768) {
        // short rows: blocks of 8 consumer warps, as many per SM as can hold a row each (at most 7 by
        // thread count); among chunk sizes that reach that count take the preferred one; the ring then
        // grows into what is left.
        constexpr int NW = 8;
        constexpr int kMaxBlocksByThreads = 2048 / (NW * 32 + 32);
        RingPlan best;
        const int order[2] = {row_bytes >= 16384 ? 2 : 1, row_bytes >= 16384 ? 1 : 2};
        for (int U : order) {
            const size_t chunk = (size_t)NW * 32 * 16 * U;
            const int chunks = (int)((row_bytes + chunk - 1) / chunk);
            const size_t need = ring_smem_bytes(NW, U, chunks) + kStatic;
            if (need > (size_t)block_smem_max) continue;
            int k = (int)std::min<size_t>(kMaxBlocksByThreads, (size_t)sm_smem / (need + kReserved));
            if (k < 1 || k <= best.blocks_per_sm) continue;
            const size_t per_block = std::min<size_t>((size_t)sm_smem / k - kReserved, (size_t)block_smem_max) - kStatic;
            int S = chunks;
            while (ring_smem_bytes(NW, U, S + 1) <= per_block) ++S;
            best = RingPlan{NW, U, S, chunks, 1, k, ring_smem_bytes(NW, U, S)};
        }
        if (best.NW) return best;
    }
    // rows larger than shared memory are streamed twice.  One block of 16 consumer warps per SM
    // keeps the number of rows in flight at the number of SMs, so that the second read of a row
    // (a few tens of microseconds after the first) is still served by L2.
    const int NW = 16, U = 4;
    const size_t chunk = (size_t)NW * 32 * 16 * U;
    const int chunks = (int)((row_bytes + chunk - 1) / chunk);
    int S = 2;
    while (ring_smem_bytes(NW, U, S + 1) + kStatic <= (size_t)block_smem_max) ++S;
    return RingPlan{NW, U, S, chunks, 0, 1, ring_smem_bytes(NW, U, S)};
}

}  // namespace rlhf
