// Loss forward/backward with the exponentials kept on chip between the passes (registers and tensor memory, as
// in kernels_creg.cuh) and the row passing through a ring of 16 KB chunks instead of whole-slice buffers.  A
// block's slice is then bounded by the ring (eight chunks of a slice in flight beside five that prefetch the
// next one: 128 KB) rather than by half of shared memory (105 KB), so that rows of 105-128 KB need no cluster
// and rows of 210-256 KB (V = 128256) a cluster of two blocks instead of three: every SM of the device has a
// block (clusters of three leave 13 of 148 SMs idle), and the per-row block reduction and cluster exchange are
// paid once per 128 KB instead of once per 85 KB.  The host picks this kernel where it needs fewer blocks per
// row than the whole-slice kernel, and for rows beyond that kernel's largest cluster.
//
// Ring: R slots of 16 KB (two vectors per consumer thread).  Chunk c of the block's i-th slice is global
// chunk g = i*C + c and lives in slot g % R.  Per slot a "full" mbarrier (bulk load landed) and a "done"
// mbarrier (the consumers have replaced the chunk's logits by its gradient).  The producer thread drains
// done chunks to global memory with bulk stores and reloads their slots, in chunk order; it keeps up to
// three stores in flight and waits for a slot's store to have read shared memory only when it reloads that
// slot.  The consumers read chunk after chunk in pass 1 (waiting for each to land), meet once (block
// reduction, cluster exchange), and write chunk after chunk in pass 2, handing each chunk back as soon as a
// warp is done with it.  The chunks of a slice stay in their slots from pass 1 to pass 2.
//
// Rows are dealt as in kernels_creg.cuh: single blocks take them from the counter in the workspace (a padded
// row is zero-filled on the spot), clusters statically.  Waits are bounded; the tensor-memory columns are
// released by the warp that took them.
#pragma once
#include <type_traits>

#include "kernels_creg.cuh"

namespace rlhf {

constexpr int kCringU = 2;                    // vectors per consumer thread and chunk
constexpr int kCringZeroBytes = 8192;         // zeroed buffer that feeds the bulk zero-fill of padded rows
constexpr int kCringMaxSlots = 13;
constexpr int kCringRows = 8;                 // row infos in flight (a power of two)

struct CringArgs {
    RowArgs row;
    unsigned row_bytes;      // 2*V, a multiple of 16
    unsigned slice_vecs;     // vectors per block of a cluster: ceil(row vectors / cluster size)
    unsigned tmem_cols;      // tensor-memory columns to take: a power of two from 32 to 512
    int n_slots;             // R
    int chunks;              // chunks of the longest slice, at most R - 1
    unsigned* row_counter;   // workspace word, zero between calls: next row to hand out (kCluster == 1)
};

inline size_t cring_chunk_bytes(int consumer_warps) { return (size_t)consumer_warps * 32 * 16 * kCringU; }
inline size_t cring_smem_bytes(int consumer_warps, int n_slots)
{
    return (size_t)n_slots * cring_chunk_bytes(consumer_warps) + kCringZeroBytes + 256;
}

__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits until at most n (0..3) of this thread's bulk-store groups have not yet read their shared-memory source.
__device__ __forceinline__ void bulk_wait_read_upto(uint32_t n)
{
    if (n == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    else if (n == 1) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
    else if (n == 2) asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory");
    else asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
}

template <int NW, int kCluster, bool kF16>
__global__ void __launch_bounds__(NW * 32 + 32, 1) loss_cring_kernel(CringArgs ca)
{
    constexpr int kRegVecs = kRegVecsTmem;                   // the first two chunks' exponentials stay in registers
    static_assert(kRegVecs == 2 * kCringU, "two chunks in registers");
    constexpr int kCons = NW * 32;
    constexpr int kThreads = kCons + 32;
    constexpr uint32_t kChunk = (uint32_t)kCons * 16u * kCringU;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ float2 s_part[2][32];
    __shared__ __align__(16) float s_sum[2][(NW + 3) / 4 * 4];
    __shared__ LabelInfo s_lab[2];
    __shared__ RowInfo s_row[kCringRows];
    __shared__ double s_dbl[32];
    __shared__ double s_loss[2];
    __shared__ int s_last;
    __shared__ __align__(16) float4 s_xchg[2][kCluster];     // per row parity: (M, s, ey, zy) of every block of the cluster
    __shared__ __align__(8) unsigned long long s_xbar[2];
    __shared__ uint32_t s_tmem_base;

    const RowArgs& p = ca.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = ca.n_slots;
    const uint32_t crank = kCluster > 1 ? cluster_ctarank() : 0u;
    const long long cid = blockIdx.x / kCluster;             // this block's cluster
    const long long G = gridDim.x / kCluster;                // clusters in the grid
    const uint32_t row_vecs = ca.row_bytes / 16u;
    const uint32_t v0 = min(row_vecs, crank * ca.slice_vecs);      // this block's slice of every row: vectors [v0, v0+nvec)
    const uint32_t nvec = min(row_vecs - v0, ca.slice_vecs);
    const uint32_t slice_off = v0 * 16u, slice_bytes = nvec * 16u;
    const int C = (int)((slice_bytes + kChunk - 1) / kChunk);      // chunks of this block's slice (at most ca.chunks)

    const uint32_t ring_addr = smem_u32(smem);
    unsigned char* zero_buf = smem + (size_t)R * kChunk;
    const uint32_t bar_addr = smem_u32(zero_buf + kCringZeroBytes);
    auto full = [&](int s) { return bar_addr + 8u * s; };
    auto done = [&](int s) { return bar_addr + 8u * (kCringMaxSlots + s); };
    const uint32_t xbar_addr = smem_u32(s_xbar);
    static_assert(2 * kCringMaxSlots * 8 <= 256, "the slots' mbarriers take the 256 bytes after the zero buffer");

    if (tid == 0) {
        for (int s = 0; s < R; ++s) {
            mbar_init(full(s), 1);
            mbar_init(done(s), NW);
        }
        mbar_init(xbar_addr, 1);
        mbar_init(xbar_addr + 8u, 1);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem_base), ca.tmem_cols);
    for (int i = tid; i < kCringZeroBytes / 16; i += kThreads) ((uint4*)zero_buf)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    if (kCluster > 1) cluster_sync_all();        // every peer's barriers exist before anyone signals them
    pdl_wait_prior_grid();                       // nothing above touches global memory
    pdl_release_next_grid();

    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const int n_mine = N > cid ? (int)((N - cid + G - 1) / G) : 0;   // rows of this cluster: cid, cid + G, ...
    const uint32_t last_bytes = slice_bytes - (uint32_t)(C - 1) * kChunk;   // of a slice's last chunk (C = ceil(slice/chunk))

    bool aborted = false;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        if (lane == 0 && nvec > 0) {
            const long long total_rows = (long long)p.B * p.T;
            const long long n_pad = total_rows - N;
            const PadShare pads = kCluster > 1 ? pad_share(N, n_pad, G, cid) : PadShare{0, 0};   // static deal: padded rows of the cluster
            const long long pads_mine = pads.count;
            const long long pads_early = pads_mine > kTailPads ? pads_mine - kTailPads : 0;
            Cursor cur{0, 0}, pcur{0, 0};
            long long pads_done = 0;
            uint32_t seq = 0;                 // bulk-store groups committed so far
            uint32_t sseq[4] = {0, 0, 0, 0};  // seq of the store of chunk d, at d & 3, for the last four chunks stored
            auto zero_fill_row = [&](int b, int t) {
                unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t) + slice_off;
                for (uint32_t off = 0; off < slice_bytes; off += kCringZeroBytes)
                    bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kCringZeroBytes, slice_bytes - off));
                bulk_commit();
                ++seq;
            };
            auto zero_fill_next = [&]() {
                int b, t;
                if (!cursor_seek_padded(pcur, pads.start + pads_done, p.lengths, p.B, p.T, b, t)) return;
                zero_fill_row(b, t);
            };
            // drain side: chunk d_row*C + d_c in slot d_slot, phase d_ph of that slot's barriers
            long long d_idx = 0;
            int d_row = 0, d_c = 0, d_slot = 0;
            uint32_t d_ph = 0;
            auto store_next = [&]() {
                unsigned char* dst = (unsigned char*)(p.dlogits + s_row[d_row & (kCringRows - 1)].dl_offset) + slice_off + (size_t)d_c * kChunk;
                bulk_store(dst, ring_addr + (uint32_t)d_slot * kChunk, d_c == C - 1 ? last_bytes : kChunk);
                bulk_commit();
                sseq[d_idx & 3] = ++seq;
                ++d_idx;
                if (++d_c == C) { d_c = 0; ++d_row; }
                if (++d_slot == R) { d_slot = 0; d_ph ^= 1u; }
            };
            // Makes the slot of global chunk g reusable: chunk g - R has been stored and the store has read the slot.
            auto ensure_free = [&](long long g) {
                const long long need = g - R;
                if (need < 0) return;
                while (d_idx <= need && !aborted) {
                    mbar_wait(done(d_slot), d_ph, p.status, aborted, p.wait_limit_ns);
                    if (!aborted) store_next();
                }
                if (aborted) return;
                // chunks that are done already go out too, so that their stores overlap this one's
                while (d_idx <= need + 2 && d_idx < g && mbar_test(done(d_slot), d_ph)) store_next();
                bulk_wait_read_upto(min(seq - sseq[need & 3], 3u));
            };
            // The rows: single blocks take the next row of the row-major list of all rows from a counter (a padded row
            // is zero-filled on the spot); clusters take valid rows cid, cid + G, ...  A row's scalars (token id, old
            // log-prob, advantage) are requested two rows ahead of their use.
            struct Ahead {
                int b, t;
                long long y;
                float lp_old, adv;
                bool ok;
            };
            long long k_ahead = cid;
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
            // load side
            long long g = 0;
            int l_slot = 0;
            int i = 0;
            for (; !aborted; ++i) {
                const Ahead a = a0;
                a0 = a1;
                a1 = fetch();
                if (!a.ok) break;
                const int b = a.b, t = a.t;
                const long long flat = (long long)b * p.T + t;
                RowInfo ri;
                ri.flat = flat;
                ri.dl_offset = (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t;
                ri.bad_id = (a.y < 0 || a.y >= p.V) ? 1 : 0;
                ri.y = ri.bad_id ? 0 : (int)a.y;
                ri.lp_old = a.lp_old;
                ri.adv = a.adv;
                ri.mis = 0;
                ri.pad = 0;
                if (ri.bad_id && crank == 0) atomicOr(p.status, kErrIdRange);
                const unsigned char* row = (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t) + slice_off;
                for (int c = 0; c < C && !aborted; ++c, ++g) {
                    ensure_free(g);
                    if (aborted) break;
                    if (c == 0) s_row[i & (kCringRows - 1)] = ri;       // published by the arrival below
                    const uint32_t bytes = c == C - 1 ? last_bytes : kChunk;
                    mbar_arrive_expect_tx(full(l_slot), bytes);
                    bulk_load(ring_addr + (uint32_t)l_slot * kChunk, row + (size_t)c * kChunk, bytes, full(l_slot));
                    if (++l_slot == R) l_slot = 0;
                }
                if (kCluster > 1) {
                    const long long target = ((long long)(i + 1) * pads_early) / n_mine;
                    while (pads_done < target) { zero_fill_next(); ++pads_done; }
                }
            }
            while (pads_done < pads_mine) { zero_fill_next(); ++pads_done; }
            // no more rows: the consumers are told through the next row's info
            if (!aborted) {
                ensure_free(g);
                if (!aborted) {
                    s_row[i & (kCringRows - 1)].flat = -1;
                    mbar_arrive_expect_tx(full(l_slot), 0);
                }
            }
            while (d_idx < g && !aborted) {
                mbar_wait(done(d_slot), d_ph, p.status, aborted, p.wait_limit_ns);
                if (!aborted) store_next();
            }
            bulk_wait_all();
        }
        if (kCluster > 1) cluster_sync_unaligned();                     // no block leaves while a peer may still write to it
        return;
    }

    // ---------------------------------------------------------------- consumers
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const int nj = 2 * C;                                          // vectors per thread, the ones past the slice's end included
    const int nt = nj - kRegVecs;                                  // of which in tensor memory
    const uint32_t tmem_addr = s_tmem_base + (((uint32_t)(warp & 3) * 32u) << 16) + (uint32_t)(warp >> 2) * (uint32_t)(nt * 8);
    {
        const double vf = consumer_sum_double<NW>(value_loss_slice(p, N, tid, kCons, true), s_dbl, warp, lane);
        if (tid == 0) s_loss[1] = vf;
    }
    const uint4 neg4 = make_uint4(El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2, El<kF16>::kNegInf2);
    // this thread's vector j of a slice (vector j*kCons + tid): inside the slice?
    auto valid = [&](int j) { return (uint32_t)j * kCons + (uint32_t)tid < nvec; };

    int s0 = 0;                     // slot of the current slice's first chunk, and the phase of that slot's barriers
    uint32_t ph0 = 0;
    if (nvec > 0)
    for (int i = 0;; ++i) {
        const int par = i & 1;
        const uint32_t use = (uint32_t)(i >> 1) & 1u;                // of the exchange barrier, which alternates by row
        auto slot_of = [&](int c) { const int s = s0 + c; return s >= R ? s - R : s; };
        auto phase_of = [&](int c) { return s0 + c >= R ? ph0 ^ 1u : ph0; };
        mbar_wait(full(s0), ph0, p.status, aborted, p.wait_limit_ns);
        aborted = __any_sync(0xffffffffu, aborted);                 // a warp gives up as a whole
        RowInfo ri = s_row[i & (kCringRows - 1)];
        if (aborted) { ri.y = 0; ri.bad_id = 1; ri.flat = 0; }      // stale row info: touch nothing
        if (ri.flat < 0) break;                                      // the producer has no more rows (the same for every thread)

        // where the generated token sits: vector ylocal of this slice (if < nvec), entry yj
        const uint32_t ylocal = ((uint32_t)ri.y >> 3) - v0;
        const int yj = ri.y & 7;
        const bool label_here = ylocal < nvec;
        const bool owner = label_here && (ylocal % kCons) == (uint32_t)tid;
        const int jy = owner ? (int)(ylocal / kCons) : -1;

        // The reference exponent: the scaled maximum of the slice's first vector, which every thread reads,
        // without the generated token's entry.
        float Mref;
        {
            uint4 q0 = *(const uint4*)(smem + (size_t)s0 * kChunk);
            if (label_here && ylocal == 0) q0 = mask_vec_entry<kF16>(q0, yj);
            Mref = max8_scaled<kF16>(q0);
        }
        // This thread's vector j, the generated token's entry taken out (it becomes -inf, a term of 0), so that
        // the sums below are sums over the other entries and 1 - p_y comes without cancellation.
        // Only a slice's last chunk has vectors past the slice's end (a slice has at least three chunks): `last` says
        // whether the chunk at hand is that one.
        float zy = 0.f;
        auto vec = [&](auto last, int j, const unsigned char* chunk, int u) -> uint4 {
            uint4 q = ((const uint4*)chunk)[u * kCons + tid];
            if (decltype(last)::value && !valid(j)) q = neg4;
            if (j == jy) {
                const uint32_t w = yj < 2 ? q.x : (yj < 4 ? q.y : (yj < 6 ? q.z : q.w));
                zy = El<kF16>::widen((uint16_t)((yj & 1) ? (w >> 16) : (w & 0xffffu)));
                q = mask_vec_entry<kF16>(q, yj);
            }
            return q;
        };
        auto exps = [&](const uint4& q, float negM, float2 (&ev)[4]) {
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const float2 x = __ffma2_rn(El<kF16>::unpack2(w[h]), splat2(kLog2e), splat2(negM));
                ev[h] = make_float2(ex2(x.x), ex2(x.y));
            }
        };

        // ---- pass 1: the exponentials of this thread's vectors against the reference, chunk by chunk as the
        // chunks land; the first two chunks' stay in registers, the others' go to tensor memory
        float2 e[kRegVecs][4];
        auto fill = [&](float negM) -> float {
            float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                mbar_wait(full(slot_of(c)), phase_of(c), p.status, aborted, p.wait_limit_ns);
                const unsigned char* chunk = smem + (size_t)slot_of(c) * kChunk;
#pragma unroll
                for (int u = 0; u < kCringU; ++u) {
                    const int j = c * kCringU + u;
                    exps(vec(std::false_type{}, j, chunk, u), negM, e[j]);
                    acc0 = __fadd2_rn(acc0, e[j][0]);
                    acc1 = __fadd2_rn(acc1, e[j][1]);
                    acc0 = __fadd2_rn(acc0, e[j][2]);
                    acc1 = __fadd2_rn(acc1, e[j][3]);
                }
            }
            auto to_tmem = [&](auto last, int c) {
                mbar_wait(full(slot_of(c)), phase_of(c), p.status, aborted, p.wait_limit_ns);
                const unsigned char* chunk = smem + (size_t)slot_of(c) * kChunk;
#pragma unroll
                for (int u = 0; u < kCringU; ++u) {
                    const int j = c * kCringU + u;
                    float2 et[4];
                    exps(vec(last, j, chunk, u), negM, et);
                    tmem_store8(tmem_addr + (uint32_t)(j - kRegVecs) * 8u, et);
                    acc0 = __fadd2_rn(acc0, et[0]);
                    acc1 = __fadd2_rn(acc1, et[1]);
                    acc0 = __fadd2_rn(acc0, et[2]);
                    acc1 = __fadd2_rn(acc1, et[3]);
                }
            };
            for (int c = 2; c < C - 1; ++c) to_tmem(std::false_type{}, c);
            to_tmem(std::true_type{}, C - 1);
            return (acc0.x + acc0.y) + (acc1.x + acc1.y);
        };
        float M = Mref, vs = 0.f, xy = kFloorM;
#pragma unroll 1
        for (int attempt = 0;; ++attempt) {
            vs = fill(-M);
            if (owner) xy = fmaxf(zy * kLog2e, kFloorM);
            // in range: every term at most 2^64 against the reference, the generated token's included
            const bool in_range = vs <= 1.8446744e19f && M > kFloorM && !(xy - M > kRebase);
            const bool redo = attempt == 0 && !in_range && (valid(0) || owner);
            // the tensor-memory stores are warp-wide: if any lane has to redo its share, the whole warp does
            if (!__any_sync(0xffffffffu, redo)) break;
            if (redo) {
                // a reference of this thread's own: its largest scaled entry (all chunks have landed)
                float m = xy;
                for (int c = 0; c < C; ++c)
                    for (int u = 0; u < kCringU; ++u)
                        if (valid(c * kCringU + u))
                            m = fmaxf(m, max8_scaled<kF16>(((const uint4*)(smem + (size_t)slot_of(c) * kChunk))[u * kCons + tid]));
                M = m;
            }
        }
        aborted = __any_sync(0xffffffffu, aborted);
        if (!valid(0) && !owner) { M = Mref; vs = 0.f; }
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
            if (!mbar_try_wait_cluster(xbar_addr + 8u * par, use))
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

        // ---- pass 2: gradient = exponential * (-g / sum), written over the logits chunk by chunk; every chunk
        // goes back to the producer as soon as this warp is done with it
        auto release = [&](int c) {
            fence_async_smem();                                     // this thread's writes, before the bulk store reads them
            __syncwarp();
            if (lane == 0) mbar_arrive(done(slot_of(c)));
        };
        if (g == 0.f) {
            for (int c = 0; c < C; ++c) {
                uint4* chunk = (uint4*)(smem + (size_t)slot_of(c) * kChunk);
#pragma unroll
                for (int u = 0; u < kCringU; ++u)
                    if (c < C - 1 || valid(c * kCringU + u)) chunk[u * kCons + tid] = make_uint4(0, 0, 0, 0);
                release(c);
            }
        } else {
            const float mag = ex2(M + (lg2(fabsf(g)) - r.lse2));       // |g| 2^M / sum, M this thread's reference
            const float2 sc2 = splat2(g > 0.f ? -mag : mag);
            const float dy = g * r.one_m_py;
            auto emit = [&](auto last, const float2 (&ev)[4], int j, uint4* chunk, int u) {
                uint32_t o[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float2 d = __fmul2_rn(ev[h], sc2);
                    o[h] = El<kF16>::pack2(d.x, d.y);
                }
                uint4 ov = make_uint4(o[0], o[1], o[2], o[3]);
                if (j == jy) patch_label<kF16>(ov, yj, dy);
                if (!decltype(last)::value || valid(j)) chunk[u * kCons + tid] = ov;
            };
            tmem_wait_stores();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint4* chunk = (uint4*)(smem + (size_t)slot_of(c) * kChunk);
#pragma unroll
                for (int u = 0; u < kCringU; ++u) emit(std::false_type{}, e[c * kCringU + u], c * kCringU + u, chunk, u);
                release(c);
            }
            auto from_tmem = [&](auto last, int c) {
                uint4* chunk = (uint4*)(smem + (size_t)slot_of(c) * kChunk);
#pragma unroll
                for (int u = 0; u < kCringU; ++u) {
                    const int j = c * kCringU + u;
                    float2 et[4];
                    tmem_load8(tmem_addr + (uint32_t)(j - kRegVecs) * 8u, et);
                    tmem_wait_loads();
                    emit(last, et, j, chunk, u);
                }
                release(c);
            };
            for (int c = 2; c < C - 1; ++c) from_tmem(std::false_type{}, c);
            from_tmem(std::true_type{}, C - 1);
        }
        s0 += C;
        if (s0 >= R) { s0 -= R; ph0 ^= 1u; }
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
    tmem_fence_before_sync();
    asm volatile("bar.sync 1, %0;" ::"n"(kCons) : "memory");
    if (warp == 0) tmem_dealloc(s_tmem_base, ca.tmem_cols);
    if (kCluster > 1) cluster_sync_unaligned();                     // no block leaves while a peer may still write to it
}

}  // namespace rlhf
