// Loss forward/backward with the row's exponentials kept on chip between the two passes, for 16-byte
// aligned rows of 16 KB and more; rows that do not fit one block twice are shared by a thread-block
// cluster of up to 4 blocks.
// (kernels_cring.cuh holds the variant that passes the row through a ring of chunks, which takes some row
// lengths with fewer blocks; the helpers below serve both.)
//
// A row's gradient needs every softmax term twice: once in the partition sum and once, scaled by the
// token's g / sum, as the gradient entry itself.  Recomputing the exponential in the second pass costs two
// ex2 per logit, which makes the special-function unit (16 results per clock per SM) the limiter
// whenever the SM clock drops under the power cap.  Here every consumer
// thread keeps the exponentials of its share of the row after the first pass -- those of its first
// kRegVecs vectors in registers, those of the following ones in tensor memory (the 256 KB per SM that
// otherwise hold tensor-core accumulators; each warp stores and loads its own 32 lanes x 128 columns with
// tcgen05.st / tcgen05.ld) -- so the second pass is one packed multiply and one conversion per pair of
// logits: one ex2 per logit in total, and no second read of the row from shared memory.
//
// Rows up to about 105 KB are held by one block, in two row buffers (three where they fit, which keeps more
// loads in flight): while row i is reduced (pass 1) and turned into dlogits (pass 2) out of one buffer, the
// bulk copies of the next rows into the others are already in flight, so that DRAM sees each row read once
// and written once and, but for a block's first row, the consumers find their row in shared memory.
// Longer rows are cut into kCluster contiguous slices, one per block of a cluster: every block runs the
// pipeline on its slice (its own producer thread, its own two slice buffers), and once per row the blocks
// exchange their partial partition sums through distributed shared memory (one asynchronous 16-byte store
// per peer, which completes on the peer's mbarrier), after which every block holds the same row total and
// finishes its slice on its own.
//
// Work distribution.  A block that holds whole rows (kCluster == 1) takes its rows from a counter in the
// workspace, one at a time, in row-major order of all B*T rows: a padded row is zero-filled on the spot by
// the producer thread, a valid row goes through the pipeline.  (The SMs do not see the same memory
// bandwidth and latency, so a static deal leaves the slowest block 10 to 20% behind the median.)  Results
// do not depend on which block gets which row: a row's outputs are a function of the row alone, and the
// policy loss is not summed per block: every row's term goes to the per-token area of the workspace, and
// the block that finishes last adds all of them in a fixed order.  Clusters take their rows statically
// (cluster c the valid rows c, c + G, ...): their rows are long and uniform.
//
// Pipeline of one block: a producer thread loads slice i+1 into the other buffer while the consumers work
// on slice i (it also requests each row's token id, old log-prob and advantage two rows ahead, so that it
// never waits for them); the consumers write the bf16 gradient over the logits in the buffer and hand it
// back; the producer drains it to global memory with one bulk store and refills it.  Waits are bounded
// (RowArgs::wait_limit_ns); if one runs out the thread flags RLHF_ERR_TIMEOUT, stops waiting and lets the
// block drain.  The tensor-memory columns are released by the warp that took them, after all consumers
// have passed a block barrier at the end of the kernel.
#pragma once
#include "kernels_ring.cuh"

namespace rlhf {

constexpr long long kTailPads = 2;      // padded rows of a cluster that are zero-filled after its last load

// What the producer publishes for each row before it arms the row's "landed" barrier.
struct RowInfo {
    long long flat;         // b*T + t
    long long dl_offset;    // element offset of the dlogits row
    int y;                  // generated token (0 if it was out of range)
    int bad_id;
    float lp_old;
    float adv;
    unsigned mis;           // bytes between the 16-byte boundary below the row's first logit and that logit
    unsigned pad;
};

// Block-wide total of the partial sums, as consumer_reduce but with log2(NW) cross-warp steps.
template <int NW>
__device__ __forceinline__ Acc creg_reduce(const Acc& a, float2* s_part, const LabelInfo* s_lab, int warp, int lane)
{
    float M = a.M;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float s = a.s * ex2(a.M - M);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) s_part[warp] = make_float2(M, s);
    asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
    constexpr int kTop = NW > 16 ? 16 : (NW > 8 ? 8 : 4);
    const float2 pw = lane < NW ? s_part[lane] : make_float2(kFloorM, 0.f);
    float Mt = pw.x;
#pragma unroll
    for (int o = kTop; o > 0; o >>= 1) Mt = fmaxf(Mt, __shfl_xor_sync(0xffffffffu, Mt, o));
    float st = pw.y * ex2(pw.x - Mt);
#pragma unroll
    for (int o = kTop; o > 0; o >>= 1) st += __shfl_xor_sync(0xffffffffu, st, o);
    // lanes >= 2*kTop did not take part; everyone takes lane 0's result
    Mt = __shfl_sync(0xffffffffu, Mt, 0);
    st = __shfl_sync(0xffffffffu, st, 0);
    const LabelInfo li = *s_lab;
    Acc tot;
    tot.M = fmaxf(Mt, li.M);
    tot.s = st * ex2(Mt - tot.M);
    tot.ey = li.ey * ex2(li.M - tot.M);
    return tot;
}


#ifndef RLHF_CREG_REGVECS_ONLY
#define RLHF_CREG_REGVECS_ONLY 8
#endif
constexpr int kRegVecsOnly = RLHF_CREG_REGVECS_ONLY;        // vectors per consumer thread when the registers hold all of a thread's exponentials
constexpr int kRegVecsTmem = 4;        // vectors per consumer thread kept in registers when the rest goes to tensor memory
constexpr int kTmemVecs = 16;          // at most so many vectors per consumer thread in tensor memory
constexpr int kCregZeroBytes = 16384;  // zeroed buffer that feeds the bulk zero-fill of padded rows
#ifndef RLHF_CREG_PIECE
#define RLHF_CREG_PIECE 16384
#endif

struct CregArgs {
    RowArgs row;
    unsigned row_bytes;      // 2*V, a multiple of 16
    unsigned slice_vecs;     // vectors per block of a cluster: ceil(row vectors / cluster size)
    unsigned buf_stride;     // bytes between the two slice buffers: a whole number of vectors per consumer thread
    unsigned tmem_cols;      // tensor-memory columns to take: 0, or a power of two from 32 to 512
    int n_buf;               // slice buffers per block: 2 or 3
    unsigned* row_counter;   // workspace word, zero between calls: next row to hand out (kCluster == 1)
};

// A slice buffer holds the same number of vectors for every consumer thread; the vectors past the end of the
// slice are set to -inf once and never written again, so that the loops over a thread's vectors need no
// per-thread bound.
inline size_t creg_buf_stride(unsigned slice_vecs, int consumer_warps)
{
    const size_t per_round = (size_t)consumer_warps * 32;
    return (slice_vecs + per_round - 1) / per_round * per_round * 16;
}
constexpr int kCregMaxBufs = 3;
inline size_t creg_smem_bytes(unsigned slice_vecs, int consumer_warps, int n_buf)
{
    return (size_t)n_buf * creg_buf_stride(slice_vecs, consumer_warps) + kCregZeroBytes + 64;
}
// Columns of tensor memory that a block needs for slices of `slice_vecs` vectors: each warp stores 8 columns per
// vector beyond the first kRegVecsTmem; warps w, w+4, w+8, ... share 32 lanes and take consecutive column ranges.
inline unsigned creg_tmem_cols(unsigned slice_vecs, int consumer_warps)
{
    const unsigned per_round = (unsigned)consumer_warps * 32;
    const unsigned nj = (slice_vecs + per_round - 1) / per_round;
    if (nj <= (unsigned)kRegVecsOnly) return 0;
    const unsigned need = (nj - kRegVecsTmem) * 8 * (((unsigned)consumer_warps + 3) / 4);
    unsigned cols = 32;
    while (cols < need) cols *= 2;
    return cols;
}

// ---------------------------------------------------------------- cluster helpers
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address, in the cluster's shared window, of this block's shared address `addr` in block `rank`.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// 16 bytes into a peer's shared memory; the peer's mbarrier receives 16 transaction bytes when they are visible.
__device__ __forceinline__ void remote_store_v4(uint32_t remote_addr, const float4& v, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The same barrier for code in which the warps are no longer whole (the producer warp has one live lane).
__device__ __forceinline__ void cluster_sync_unaligned()
{
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a phase that peers of the cluster complete.
__device__ __noinline__ bool mbar_wait_cluster_slow(uint32_t bar, uint32_t parity, unsigned* status,
                                                    unsigned long long limit_ns)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) {
            atomicOr(status, kErrTimeout);
            return false;
        }
    }
}

// Entry j of a vector replaced by -inf.
template <bool kF16>
__device__ __forceinline__ uint4 mask_vec_entry(const uint4& q, int j)
{
    uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i == j)
            w[i >> 1] = (i & 1) ? ((w[i >> 1] & 0x0000ffffu) | (El<kF16>::kNegInf << 16)) : ((w[i >> 1] & 0xffff0000u) | El<kF16>::kNegInf);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// ---------------------------------------------------------------- tensor memory as a scratch pad
// One warp takes `cols` columns (a power of two >= 32) for the block and writes their base address to shared memory.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 8 values per thread: lane (of the warp's 32) x 8 consecutive columns.  Whole warp.
__device__ __forceinline__ void tmem_store8(uint32_t taddr, const float2 (&v)[4])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(__float_as_uint(v[0].x)), "r"(__float_as_uint(v[0].y)), "r"(__float_as_uint(v[1].x)),
                   "r"(__float_as_uint(v[1].y)), "r"(__float_as_uint(v[2].x)), "r"(__float_as_uint(v[2].y)),
                   "r"(__float_as_uint(v[3].x)), "r"(__float_as_uint(v[3].y)) : "memory");
}
__device__ __forceinline__ void tmem_load8(uint32_t taddr, float2 (&v)[4])
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int h = 0; h < 4; ++h) v[h] = make_float2(__uint_as_float(r[2 * h]), __uint_as_float(r[2 * h + 1]));
}
__device__ __forceinline__ void tmem_wait_stores() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_loads() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- the kernel
// kTmem: a thread's vectors beyond the first kRegVecsTmem keep their exponentials in tensor memory; otherwise a
// thread has at most kRegVecsOnly vectors and registers hold all of them.  kF16: logits and gradient are IEEE
// binary16 instead of bf16.  kAny (single blocks only): rows, of logits and dlogits alike and with the same offset
// from a 16-byte boundary, may start at any even address and have any length; the aligned span around a row is
// loaded, the entries of its first and last vector that belong to neighbouring rows are turned into -inf in the
// buffer before the first pass, and only the row's own bytes are stored: whole vectors by bulk store, the ragged
// ends by 2-byte stores.
template <int NW, int kCluster, bool kTmem, bool kF16, bool kAny = false>
__global__ void __launch_bounds__(NW * 32 + 32, 1) loss_creg_kernel(CregArgs ca)
{
    static_assert(!kAny || kCluster == 1, "rows off 16-byte boundaries are not split over a cluster");
    constexpr int kRegVecs = kTmem ? kRegVecsTmem : kRegVecsOnly;
    constexpr int kCons = NW * 32;
    constexpr int kThreads = kCons + 32;
    constexpr uint32_t kPiece = RLHF_CREG_PIECE;  // size of one bulk copy
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ float2 s_part[2][32];
    __shared__ __align__(16) float s_sum[2][(NW + 3) / 4 * 4];
    __shared__ LabelInfo s_lab[2];
    __shared__ RowInfo s_row[kCregMaxBufs];
    __shared__ double s_dbl[32];
    __shared__ double s_loss[2];
    __shared__ int s_last;
    __shared__ __align__(16) float4 s_xchg[2][kCluster];     // per row parity: (M, s, ey, zy) of every block of the cluster
    __shared__ __align__(8) unsigned long long s_xbar[2];
    static_assert(kCregMaxBufs * 16 <= 64, "the mbarriers of the buffers take the 64 bytes after the zero buffer");
    __shared__ uint32_t s_tmem_base;

    const RowArgs& p = ca.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NB = ca.n_buf;
    const uint32_t crank = kCluster > 1 ? cluster_ctarank() : 0u;
    const long long cid = blockIdx.x / kCluster;             // this block's cluster
    const long long G = gridDim.x / kCluster;                // clusters in the grid
    const uint32_t row_vecs = kAny ? ca.slice_vecs : ca.row_bytes / 16u;   // kAny: the longest aligned span around a row
    const uint32_t v0 = min(row_vecs, crank * ca.slice_vecs);      // this block's slice of every row: vectors [v0, v0+nvec)
    const uint32_t nvec = min(row_vecs - v0, ca.slice_vecs);
    const uint32_t slice_off = v0 * 16u, slice_bytes = nvec * 16u;

    const uint32_t buf_addr = smem_u32(smem);
    unsigned char* zero_buf = smem + (size_t)NB * ca.buf_stride;
    const uint32_t bar_addr = smem_u32(zero_buf + kCregZeroBytes);
    auto landed = [&](int buf) { return bar_addr + 8u * buf; };
    auto computed = [&](int buf) { return bar_addr + 8u * (kCregMaxBufs + buf); };
    const uint32_t xbar_addr = smem_u32(s_xbar);

    if (tid == 0) {
        for (int b = 0; b < NB; ++b) {
            mbar_init(landed(b), 1);
            mbar_init(computed(b), NW);
        }
        mbar_init(xbar_addr, 1);
        mbar_init(xbar_addr + 8u, 1);
        fence_mbar_init();
    }
    if (kTmem && warp == 0) tmem_alloc(smem_u32(&s_tmem_base), ca.tmem_cols);
    for (int i = tid; i < kCregZeroBytes / 16; i += kThreads) ((uint4*)zero_buf)[i] = make_uint4(0, 0, 0, 0);
    // the vectors of every buffer past the end of the slice: -inf, a term of 0 in every sum
    for (int b = 0; b < NB; ++b)
        for (uint32_t v = nvec + tid; v < ca.buf_stride / 16u; v += kThreads)
            ((uint4*)(smem + (size_t)b * ca.buf_stride))[v] = make_uint4(El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2);
    fence_async_smem();
    if (kTmem) tmem_fence_before_sync();
    __syncthreads();
    if (kTmem) tmem_fence_after_sync();
    if (kCluster > 1) cluster_sync_all();        // every peer's barriers exist before anyone signals them
    pdl_wait_prior_grid();                       // nothing above touches global memory
    pdl_release_next_grid();

    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const int n_mine = N > cid ? (int)((N - cid + G - 1) / G) : 0;   // rows of this cluster: cid, cid + G, ...

    bool aborted = false;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            const long long total_rows = (long long)p.B * p.T;
            const long long n_pad = total_rows - N;
            const PadShare pads = kCluster > 1 ? pad_share(N, n_pad, G, cid) : PadShare{0, 0};   // static deal: padded rows of the cluster
            const long long pads_mine = pads.count;
            const long long pads_early = pads_mine > kTailPads ? pads_mine - kTailPads : 0;
            Cursor cur{0, 0}, pcur{0, 0};
            long long pads_done = 0;
            auto zero_fill_row = [&](int b, int t) {
                unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t) + slice_off;
                uint32_t lo = 0, hi = slice_bytes;                   // [lo,hi): the part of the row made of whole 16-byte vectors
                if (kAny) {
                    const uint32_t mis = (uint32_t)((uintptr_t)drow & 15u);
                    lo = min(ca.row_bytes, (16u - mis) & 15u);
                    hi = max(lo, ca.row_bytes - ((mis + ca.row_bytes) & 15u));
                    for (uint32_t o = 0; o < lo; o += 2) *(uint16_t*)(drow + o) = 0;
                    for (uint32_t o = hi; o < ca.row_bytes; o += 2) *(uint16_t*)(drow + o) = 0;
                }
                for (uint32_t off = lo; off < hi; off += kCregZeroBytes)
                    bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kCregZeroBytes, hi - off));
                bulk_commit();
            };
            auto zero_fill_next = [&]() {
                int b, t;
                if (!cursor_seek_padded(pcur, pads.start + pads_done, p.lengths, p.B, p.T, b, t)) return;
                zero_fill_row(b, t);
            };
            // Hands buffer i % NB, holding the finished gradient of this block's i-th slice, to the bulk-store
            // engine and waits until it has been read out of shared memory.
            auto drain = [&](int i) {
                const int buf = i % NB;
                mbar_wait(computed(buf), (uint32_t)(i / NB) & 1u, p.status, aborted, p.wait_limit_ns);
                if (aborted) return;
                const uint32_t srcb = buf_addr + (uint32_t)buf * ca.buf_stride;
                unsigned char* drow = (unsigned char*)(p.dlogits + s_row[buf].dl_offset) + slice_off;
                uint32_t mis = 0, lo = 0, hi = slice_bytes;          // row = span bytes [mis, mis + row_bytes); whole vectors [lo,hi)
                if (kAny) {
                    mis = (uint32_t)((uintptr_t)drow & 15u);
                    lo = (mis + 15u) & ~15u;
                    hi = (mis + ca.row_bytes) & ~15u;
                    if (hi < lo) hi = lo;
                    const unsigned char* sb = smem + (size_t)buf * ca.buf_stride;
                    for (uint32_t o = mis; o < min(lo, mis + ca.row_bytes); o += 2) *(uint16_t*)(drow - mis + o) = *(const uint16_t*)(sb + o);
                    for (uint32_t o = max(hi, mis); o < mis + ca.row_bytes; o += 2) *(uint16_t*)(drow - mis + o) = *(const uint16_t*)(sb + o);
                    fence_async_smem();                              // these reads, before the buffer is refilled by bulk copies
                }
                for (uint32_t off = lo; off < hi; off += kPiece)
                    bulk_store(drow - mis + off, srcb + off, min(kPiece, hi - off));
                bulk_commit();
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            };
            // The scalars of a row (token id, old log-prob, advantage) are requested two rows ahead of their use.
            struct Ahead {
                int b, t;
                long long y;
                float lp_old, adv;
                bool ok;
            };
            long long k_ahead = cid;
            // dynamic deal: the next row of the row-major list of all rows, requested one call ahead of its use
            long long r_next = 0;
            if (kCluster == 1) r_next = (long long)atomicAdd(ca.row_counter, 1u);
            auto fetch = [&]() {
                Ahead a;
                a.ok = false;
                if (kCluster == 1) {
                    while (r_next < total_rows) {
                        const long long r = r_next;
                        r_next = (long long)atomicAdd(ca.row_counter, 1u);
                        a.b = (int)(r / p.T);
                        a.t = (int)(r % p.T);
                        if (a.t < clamp_len(__ldg(p.lengths + a.b), p.T)) { a.ok = true; break; }
                        zero_fill_row(a.b, a.t);                       // a padded row: nothing to read
                    }
                } else {
                    a.ok = k_ahead < N && cursor_seek_valid(cur, k_ahead, p.lengths, p.B, p.T, a.b, a.t);
                    k_ahead += G;
                }
                if (a.ok) {
                    const long long f = (long long)a.b * p.T + a.t;
                    a.y = __ldg(p.ids + (long long)a.b * p.ids_stride_b + a.t);
                    a.lp_old = __ldg(p.lp_old + f);
                    a.adv = __ldg(p.adv + f);
                }
                return a;
            };
            Ahead a0 = fetch(), a1 = fetch();
            int i = 0;
            for (; !aborted; ++i) {
                const Ahead a = a0;
                a0 = a1;
                a1 = fetch();
                if (!a.ok) break;
                const unsigned char* row = (const unsigned char*)(p.logits + (long long)a.b * p.stride_b + (long long)a.t * p.stride_t) + slice_off;
                RowInfo ri;
                ri.flat = (long long)a.b * p.T + a.t;
                ri.dl_offset = (long long)a.b * p.dl_stride_b + (long long)a.t * p.dl_stride_t;
                ri.bad_id = (a.y < 0 || a.y >= p.V) ? 1 : 0;
                ri.y = ri.bad_id ? 0 : (int)a.y;
                ri.lp_old = a.lp_old;
                ri.adv = a.adv;
                ri.mis = kAny ? (unsigned)((uintptr_t)row & 15u) : 0u;
                ri.pad = 0;
                if (ri.bad_id && crank == 0) atomicOr(p.status, kErrIdRange);
                const int buf = i % NB;
                if (i >= NB) drain(i - NB);                              // the buffer's previous slice goes out first
                if (aborted) break;
                s_row[buf] = ri;
                const uint32_t dst = buf_addr + (uint32_t)buf * ca.buf_stride;
                // kAny: the aligned span around the row (it stays inside the 16-byte blocks that hold the row's ends)
                const uint32_t load_bytes = kAny ? ((ri.mis + ca.row_bytes + 15u) & ~15u) : slice_bytes;
                mbar_arrive_expect_tx(landed(buf), load_bytes);          // release: publishes s_row[buf]
                for (uint32_t off = 0; off < load_bytes; off += kPiece)
                    bulk_load(dst + off, row - ri.mis + off, min(kPiece, load_bytes - off), landed(buf));
                if (kCluster > 1) {
                    const long long target = ((long long)(i + 1) * pads_early) / n_mine;
                    while (pads_done < target) { zero_fill_next(); ++pads_done; }
                }
            }
            while (pads_done < pads_mine) { zero_fill_next(); ++pads_done; }
            // no more rows: the consumers are told through the next buffer's row info
            if (!aborted) {
                const int buf = i % NB;
                if (i >= NB) drain(i - NB);
                if (!aborted) {
                    s_row[buf].flat = -1;
                    mbar_arrive_expect_tx(landed(buf), 0);
                }
            }
            for (int j = i + 1 >= NB ? i + 1 - NB : 0; j < i && !aborted; ++j) drain(j);
            bulk_wait_all();
            if (kCluster > 1) cluster_sync_unaligned();                 // no block leaves while a peer may still write to it
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const int cnt = (uint32_t)tid < nvec ? (int)((nvec - tid + kCons - 1) / kCons) : 0;   // this thread's vectors
    const int nj = (int)((nvec + kCons - 1) / kCons);              // vectors per thread, the -inf tail included
    const int nt = kTmem && nj > kRegVecs ? nj - kRegVecs : 0;     // of which in tensor memory (<= kTmemVecs)
    // this warp's window of tensor memory: its 32 lanes, 8 columns per vector
    const uint32_t tmem_addr = kTmem ? s_tmem_base + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)(warp >> 2) * (uint32_t)(nt * 8) : 0u;
    // the block's share of the value loss (thread 0 keeps the sum); it also zeroes the per-token policy terms of the
    // padded tokens, so that the final sum can run over all B*T entries
    {
        const double vf = consumer_sum_double<NW>(value_loss_slice(p, N, tid, kCons, true), s_dbl, warp, lane);
        if (tid == 0) s_loss[1] = vf;
    }

    for (int i = 0;; ++i) {
        const int buf = i % NB, par = i & 1;
        const uint32_t use = (uint32_t)(i >> 1) & 1u;                // of the exchange barrier, which alternates by row
        mbar_wait(landed(buf), (uint32_t)(i / NB) & 1u, p.status, aborted, p.wait_limit_ns);
        aborted = __any_sync(0xffffffffu, aborted);                 // a warp gives up as a whole
        RowInfo ri = s_row[buf];
        if (aborted) { ri.y = 0; ri.bad_id = 1; ri.flat = 0; }      // stale row info: touch nothing
        if (ri.flat < 0) break;                                      // the producer has no more rows (the same for every thread)
        unsigned char* rowbuf = smem + (size_t)buf * ca.buf_stride;
        const uint4* src = (const uint4*)rowbuf + tid;

        // kAny: eoff entries of the buffer's first vector precede the row; they, the entries after the row's end in its
        // last vector and the vector after that (left from a longer span) are not the row's: their owners make them -inf
        const uint32_t eoff = kAny ? (ri.mis >> 1) : 0u;
        if (kAny) {
            const uint32_t end = eoff + (uint32_t)p.V;               // entry index, in the buffer, of the row's end
            const uint32_t last = (end - 1) >> 3, past = last + 1;   // vector of the last entry, and the one after it
            uint4* vecs = (uint4*)rowbuf;
            if (eoff != 0 && tid == 0) vecs[0] = mask_vec_outside<kF16>(vecs[0], (int)eoff, 8);
            if ((end & 7u) != 0 && (last % kCons) == (uint32_t)tid) vecs[last] = mask_vec_outside<kF16>(vecs[last], 0, (int)(end & 7u));
            if (past < nvec && (past % kCons) == (uint32_t)tid)
                vecs[past] = make_uint4(El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2);
        }
        // where the generated token sits: vector ylocal of this slice (if < nvec), entry yj
        const uint32_t ylocal = ((eoff + (uint32_t)ri.y) >> 3) - v0;
        const int yj = (int)((eoff + (uint32_t)ri.y) & 7u);
        const bool label_here = ylocal < nvec;
        const bool owner = label_here && (ylocal % kCons) == (uint32_t)tid;
        const int jy = owner ? (int)(ylocal / kCons) : -1;

        // The reference exponent: the scaled maximum of the slice's first vector, which every thread reads; the
        // generated token's entry is left out of it, because its owner is replacing that entry in the buffer.
        float Mref = kFloorM;
        if (nvec > 0) {
            uint4 q0 = *(const uint4*)rowbuf;
            if (kAny) q0 = mask_vec_outside<kF16>(q0, (int)eoff, 8);
            if (label_here && ylocal == 0) q0 = mask_vec_entry<kF16>(q0, yj);
            Mref = max8_scaled<kF16>(q0);
        }
        // The owner takes the generated token's logit out of the row (it becomes -inf, a term of 0), so that
        // the sums below are sums over the other entries and 1 - p_y comes without cancellation.
        float zy = 0.f, xy = kFloorM;
        if (owner) {
            uint16_t* slot = (uint16_t*)rowbuf + ((size_t)ylocal * 8 + yj);
            zy = El<kF16>::widen(*slot);
            *slot = (uint16_t)El<kF16>::kNegInf;
            xy = fmaxf(zy * kLog2e, kFloorM);
        }

        // ---- pass 1: the exponentials of this thread's vectors against the reference; the first kRegVecs
        // vectors' stay in registers, the others' go to tensor memory
        float2 e[kRegVecs][4];
        auto fill = [&](float negM) -> float {
            float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < kRegVecs; ++j) {
                if (j < nj) {
                    const uint4 q = src[(size_t)j * kCons];
                    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const float2 x = __ffma2_rn(El<kF16>::unpack2(w[h]), splat2(kLog2e), splat2(negM));
                        e[j][h] = make_float2(ex2(x.x), ex2(x.y));
                    }
                    acc0 = __fadd2_rn(acc0, e[j][0]);
                    acc1 = __fadd2_rn(acc1, e[j][1]);
                    acc0 = __fadd2_rn(acc0, e[j][2]);
                    acc1 = __fadd2_rn(acc1, e[j][3]);
                } else {
#pragma unroll
                    for (int h = 0; h < 4; ++h) e[j][h] = make_float2(0.f, 0.f);
                }
            }
#pragma unroll 2
            for (int j = 0; kTmem && j < nt; ++j) {
                const uint4 q = src[(size_t)(kRegVecs + j) * kCons];
                const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                float2 et[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float2 x = __ffma2_rn(El<kF16>::unpack2(w[h]), splat2(kLog2e), splat2(negM));
                    et[h] = make_float2(ex2(x.x), ex2(x.y));
                }
                tmem_store8(tmem_addr + (uint32_t)j * 8u, et);
                acc0 = __fadd2_rn(acc0, et[0]);
                acc1 = __fadd2_rn(acc1, et[1]);
                acc0 = __fadd2_rn(acc0, et[2]);
                acc1 = __fadd2_rn(acc1, et[3]);
            }
            return (acc0.x + acc0.y) + (acc1.x + acc1.y);
        };
        float M = Mref, vs = 0.f;
#pragma unroll 1
        for (int attempt = 0;; ++attempt) {
            vs = fill(-M);
            // in range: every term at most 2^64 against the reference, the generated token's included
            const bool in_range = vs <= 1.8446744e19f && M > kFloorM && !(xy - M > kRebase);
            const bool redo = attempt == 0 && !in_range && (cnt > 0 || owner);
            // the tensor-memory stores are warp-wide: if any lane has to redo its share, the whole warp does
            if (!__any_sync(0xffffffffu, redo)) break;
            if (redo) {
                // a reference of this thread's own: its largest scaled entry
                float m = xy;
                for (int j = 0; j < nj; ++j) m = fmaxf(m, max8_scaled<kF16>(src[(size_t)j * kCons]));
                M = m;
            }
        }
        if (cnt == 0 && !owner) { M = Mref; vs = 0.f; }
        const bool diverged = M != Mref;

        if (label_here ? owner : tid == 0)
            s_lab[par] = label_here ? LabelInfo{zy, ex2(fmaf(zy, kLog2e, -M)), M, 0.f} : LabelInfo{0.f, 0.f, kFloorM, 0.f};
        float ws = vs;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
        if (lane == 0) s_sum[par][warp] = ws;
        Acc tot;
        if (!consumer_barrier_or<NW>(diverged || aborted)) {
            tot.M = Mref;
            tot.s = sum_warp_sums<NW>(s_sum[par]);
            tot.ey = s_lab[par].ey;
        } else {
            // a wait that ran out somewhere in the block ends the block's work here, for all its threads alike
            if (consumer_barrier_or<NW>(aborted)) { aborted = true; break; }
            tot = creg_reduce<NW>(Acc{M, vs, 0.f}, s_part[par], &s_lab[par], warp, lane);
        }
        float zy_row = s_lab[par].zy;

        if (kCluster > 1) {
            // every block of the cluster sends its slice's (M, s, ey, zy) to every block, itself included
            if (tid == 0) {
                mbar_arrive_expect_tx(xbar_addr + 8u * par, 16u * kCluster);
                const float4 mine = make_float4(tot.M, tot.s, tot.ey, zy_row);
                const uint32_t slot = smem_u32(&s_xchg[par][crank]);
#pragma unroll
                for (int r = 0; r < kCluster; ++r)
                    remote_store_v4(map_to_rank(slot, (uint32_t)r), mine, map_to_rank(xbar_addr + 8u * par, (uint32_t)r));
            }
            if (!aborted && !mbar_try_wait_cluster(xbar_addr + 8u * par, use))
                if (!mbar_wait_cluster_slow(xbar_addr + 8u * par, use, p.status, p.wait_limit_ns)) aborted = true;
            aborted = __any_sync(0xffffffffu, aborted);
            float Mx = kFloorM;
#pragma unroll
            for (int r = 0; r < kCluster; ++r) Mx = fmaxf(Mx, s_xchg[par][r].x);
            float sx = 0.f, eyx = 0.f, zx = 0.f;
#pragma unroll
            for (int r = 0; r < kCluster; ++r) {                   // in rank order: the same total in every block
                const float4 part = s_xchg[par][r];
                const float sc = ex2(part.x - Mx);
                sx = fmaf(part.y, sc, sx);
                eyx = fmaf(part.z, sc, eyx);
                zx += part.w;
            }
            tot = Acc{Mx, sx, eyx};
            zy_row = zx;
        }
        const RowResult r = row_finish_fast(tot, zy_row);

        float loss = 0.f, g = 0.f;
        if (!ri.bad_id) ppo_token<true>(r.lp, ri.lp_old, ri.adv, p.clip_eps, scale_over_N, loss, g);
        if (tid == 0 && crank == 0 && !aborted) {
            p.row_loss[ri.flat] = loss;
            if (p.out_lp_new) p.out_lp_new[ri.flat] = ri.bad_id ? 0.f : r.lp;
        }

        // ---- pass 2: gradient = exponential * (-g / sum), written over the logits in the buffer
        uint4* dst = (uint4*)rowbuf + tid;
        if (g == 0.f) {
            for (int j = 0; j < cnt; ++j) dst[(size_t)j * kCons] = make_uint4(0, 0, 0, 0);
        } else {
            const float mag = ex2(M + (lg2(fabsf(g)) - r.lse2));       // |g| 2^M / sum, M this thread's reference
            const float2 sc2 = splat2(g > 0.f ? -mag : mag);
            const float dy = g * r.one_m_py;
            auto emit = [&](const float2 (&ev)[4], int j) {
                uint32_t o[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float2 d = __fmul2_rn(ev[h], sc2);
                    o[h] = El<kF16>::pack2(d.x, d.y);
                }
                uint4 ov = make_uint4(o[0], o[1], o[2], o[3]);
                if (j == jy) patch_label<kF16>(ov, yj, dy);
                if (j < cnt) dst[(size_t)j * kCons] = ov;
            };
            if (kTmem) tmem_wait_stores();
#pragma unroll
            for (int j = 0; j < kRegVecs; ++j)
                if (j < nj) emit(e[j], j);
            for (int j = 0; kTmem && j < nt; ++j) {
                float2 et[4];
                tmem_load8(tmem_addr + (uint32_t)j * 8u, et);
                tmem_wait_loads();
                emit(et, kRegVecs + j);
            }
        }
        fence_async_smem();                                         // this thread's writes, before the bulk store reads them
        __syncwarp();
        if (lane == 0) mbar_arrive(computed(buf));
    }
    // The two losses.  Every block leaves its share of the value loss in the workspace; the block that finishes last
    // adds the per-token policy terms of the whole batch (all its consumer threads, fixed shares, fixed tree) and the
    // blocks' value-loss shares in block order.
    if (p.fused) {
        if (tid == 0) {
            p.partials[2 * blockIdx.x] = 0.0;
            p.partials[2 * blockIdx.x + 1] = s_loss[1];
            __threadfence();
            s_last = atomicAdd(p.ticket, 1u) == gridDim.x - 1 ? 1 : 0;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kCons) : "memory");
        if (s_last) {
            __threadfence();
            const long long total = (long long)p.B * p.T;
            double acc = 0.0;
            for (long long q = tid; q < total; q += kCons) acc += (double)__ldcg(p.row_loss + q);
            const double pg = consumer_sum_double<NW>(acc, s_dbl, warp, lane);
            if (tid == 0) {
                double c = 0.0;
                for (unsigned k = 0; k < gridDim.x; ++k) c += ((volatile double*)p.partials)[2 * k + 1];
                *p.out_loss_pg = N > 0 ? (float)(pg / (double)N) : 0.f;
                *p.out_loss_vf = N > 0 ? (float)(c / (double)N) : 0.f;
                *p.ticket = 0u;
                if (kCluster == 1) *ca.row_counter = 0u;
            }
        }
    }
    // the tensor-memory columns go back once every consumer is done with them
    if (kTmem) {
        tmem_fence_before_sync();
        asm volatile("bar.sync 1, %0;" ::"n"(kCons) : "memory");
        if (warp == 0) tmem_dealloc(s_tmem_base, ca.tmem_cols);
    }
    if (kCluster > 1) cluster_sync_unaligned();                     // no block leaves while a peer may still write to it
}

}  // namespace rlhf
