// Loss forward/backward for rows of which two fit in shared memory (16 KB <= row <= ~111 KB,
// i.e. vocabularies from 8K to 56K entries in bf16) -- the OPT- and Llama-2-shaped cases.
//
// One persistent block per SM: NW consumer warps work on one row at a time, a producer thread keeps
// the other row buffer filling.  While row i is reduced (pass 1) and turned into dlogits (pass 2)
// out of buffer i&1, the bulk copies of row i+1 into the other buffer are already in flight, having
// been issued when that buffer was released a whole row-time earlier; so, except for the very
// first row of a block, consumers never wait for HBM, and DRAM sees each row read once and written
// once.  Pass 2 writes the bf16 gradient over the logits in the shared-memory buffer; the producer
// thread then drains the buffer to global memory with bulk stores and refills it with the row after
// next as soon as the drain has read it, so that the block's stores and loads keep flowing while
// the consumers are already reducing the other buffer.  Synchronisation is per row, not per chunk:
// two "landed" mbarriers per buffer (a 4-vector head part so that the first row can start early, and
// the rest) and one "computed" mbarrier that hands the finished buffer back to the producer.
// The producer also looks up each row's scalars (token id, old log-prob, advantage) and hands them
// to the consumers through shared memory, so that the consumers' per-row work is the reduction and
// a short scalar chain only.  Inside a row every thread runs straight-line blocks of 4 vectors
// (32 logits) with no per-vector branch: all threads sum against one reference exponent, the sums
// are range-checked once per row (a thread whose check fails redoes its share carefully), and only
// the block that holds the generated token takes the careful path.
#pragma once
#include "kernels_ring.cuh"

namespace rlhf {

constexpr long long kTailPads = 2;      // padded rows of a block that are zero-filled after its last load

struct DbufArgs {
    RowArgs row;
    unsigned row_bytes;     // 2*V, multiple of 16
    unsigned row_stride;    // row_bytes rounded up to 128: distance between the two buffers
};

// What the producer publishes for each row before it arms the row's first "landed" barrier.
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

inline size_t dbuf_row_stride(unsigned row_bytes, bool any_alignment)
{
    return ((size_t)row_bytes + (any_alignment ? 16 : 0) + 127) & ~(size_t)127;
}

inline size_t dbuf_smem_bytes(unsigned row_bytes, bool any_alignment = false)
{
    const size_t stride = dbuf_row_stride(row_bytes, any_alignment);
    return 2 * stride + kZeroBytes + 64;       // + 6 mbarriers
}

// Block-wide total of the partial sums, as consumer_reduce but with log2(NW) cross-warp steps.
template <int NW>
__device__ __forceinline__ Acc dbuf_reduce(const Acc& a, float2* s_part, const LabelInfo* s_lab, int warp, int lane)
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

// kAny: rows (of logits and dlogits alike, with the same offset from a 16-byte boundary) may start at any
// even address and have any length.  The aligned span around the row is loaded; entries of its first and
// last vector outside the row are skipped in pass 1 and never stored: the whole vectors inside the row go
// out by bulk store, the ragged ends by 2-byte stores.
// kF16: logits and gradient are IEEE binary16 instead of bf16.
template <int NW, bool kAny, bool kF16 = false>
__global__ void __launch_bounds__(NW * 32 + 32, 1) loss_dbuf_kernel(DbufArgs da)
{
    constexpr int kCons = NW * 32;
    constexpr int kThreads = kCons + 32;
    constexpr uint32_t kPiece = 16384;           // size of one bulk copy
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ float2 s_part[2][32];
    __shared__ __align__(16) float s_sum[2][NW];
    __shared__ LabelInfo s_lab[2];
    __shared__ RowInfo s_row[2];
    __shared__ double s_dbl[32];

    const RowArgs& p = da.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t buf_addr = smem_u32(smem);
    unsigned char* zero_buf = smem + 2 * (size_t)da.row_stride;
    const uint32_t bar_addr = smem_u32(zero_buf + kZeroBytes);
    // barriers: landed[buf][part] at bar_addr + 8*(2*buf+part), computed[buf] at bar_addr + 32 + 8*buf
    auto landed = [&](int buf, int part) { return bar_addr + 8u * (2 * buf + part); };
    auto computed = [&](int buf) { return bar_addr + 32u + 8u * buf; };

    const uint32_t nvec = da.row_bytes / 16u;
    // head part: the first 4 vectors of every thread, if the row has at least twice that
    const uint32_t head_vecs = nvec >= 8u * kCons ? 4u * kCons : nvec;
    const uint32_t head_bytes = head_vecs * 16u;

    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(bar_addr + 8u * i, 1);
        mbar_init(computed(0), NW);
        mbar_init(computed(1), NW);
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
        // the last padded rows are kept back until the block's last valid row has been requested: their
        // stores then keep the memory pipe busy while that row is still being reduced
        const long long pads_early = pads_mine > kTailPads ? pads_mine - kTailPads : 0;
        Cursor cur{0, 0}, pcur{0, 0};
        long long pads_done = 0;
        auto zero_fill_next = [&]() {
            int b, t;
            if (!cursor_seek_padded(pcur, pads.start + pads_done, p.lengths, p.B, p.T, b, t)) return;
            unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t);
            uint32_t lo = 0, hi = da.row_bytes;                  // [lo,hi): the part of the row made of whole 16-byte vectors
            if (kAny) {
                const uint32_t mis = (uint32_t)((uintptr_t)drow & 15u);
                lo = min(da.row_bytes, (16u - mis) & 15u);
                hi = max(lo, da.row_bytes - ((mis + da.row_bytes) & 15u));
                for (uint32_t o = 0; o < lo; o += 2) *(uint16_t*)(drow + o) = 0;
                for (uint32_t o = hi; o < da.row_bytes; o += 2) *(uint16_t*)(drow + o) = 0;
            }
            for (uint32_t off = lo; off < hi; off += kZeroBytes)
                bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kZeroBytes, hi - off));
            bulk_commit();
        };
        // Hands buffer (i&1), holding the finished gradient of this block's i-th row, to the bulk-store
        // engine and waits until it has been read out of shared memory.
        unsigned char *drow0 = nullptr, *drow1 = nullptr;       // global rows the two buffers drain to
        auto drain = [&](long long i) {
            const int buf = (int)(i & 1);
            mbar_wait(computed(buf), (uint32_t)(i >> 1) & 1u, p.status, aborted, p.wait_limit_ns);
            if (aborted) return;
            const uint32_t srcb = buf_addr + (uint32_t)buf * da.row_stride;
            unsigned char* drow = buf ? drow1 : drow0;               // the row's first entry in global memory
            uint32_t mis = 0, lo = 0, hi = da.row_bytes;             // row = span bytes [mis, mis+row_bytes); whole vectors [lo,hi)
            if (kAny) {
                mis = (uint32_t)((uintptr_t)drow & 15u);
                lo = (mis + 15u) & ~15u;
                hi = (mis + da.row_bytes) & ~15u;
                if (hi < lo) hi = lo;
                const unsigned char* sb = smem + (size_t)buf * da.row_stride;
                for (uint32_t o = mis; o < min(lo, mis + da.row_bytes); o += 2) *(uint16_t*)(drow - mis + o) = *(const uint16_t*)(sb + o);
                for (uint32_t o = max(hi, mis); o < mis + da.row_bytes; o += 2) *(uint16_t*)(drow - mis + o) = *(const uint16_t*)(sb + o);
                fence_async_smem();                                  // these reads, before the buffer is refilled by bulk copies
            }
            for (uint32_t off = lo; off < hi; off += kPiece)
                bulk_store(drow - mis + off, srcb + off, min(kPiece, hi - off));
            bulk_commit();
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        };
        long long i = 0;
        for (long long k = blockIdx.x; k < N && !aborted; k += G, ++i) {
            int b, t;
            if (!cursor_seek_valid(cur, k, p.lengths, p.B, p.T, b, t)) break;
            const unsigned char* row = (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t);
            RowInfo ri;
            ri.flat = (long long)b * p.T + t;
            ri.dl_offset = (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t;
            const long long y = __ldg(p.ids + (long long)b * p.ids_stride_b + t);
            ri.bad_id = (y < 0 || y >= p.V) ? 1 : 0;
            ri.y = ri.bad_id ? 0 : (int)y;
            ri.lp_old = __ldg(p.lp_old + ri.flat);
            ri.adv = __ldg(p.adv + ri.flat);
            if (ri.bad_id) atomicOr(p.status, kErrIdRange);
            const int buf = (int)(i & 1);
            if (i >= 2) drain(i - 2);                                // the buffer's previous row goes out first
            if (aborted) break;
            if (buf) drow1 = (unsigned char*)(p.dlogits + ri.dl_offset);
            else drow0 = (unsigned char*)(p.dlogits + ri.dl_offset);
            ri.mis = kAny ? (unsigned)((uintptr_t)row & 15u) : 0u;
            ri.pad = 0;
            s_row[buf] = ri;
            const uint32_t dst = buf_addr + (uint32_t)buf * da.row_stride;
            if (kAny) {
                // the aligned span around the row, as one part
                const uint32_t span = (ri.mis + da.row_bytes + 15u) & ~15u;
                mbar_arrive_expect_tx(landed(buf, 0), span);         // release: publishes s_row[buf]
                for (uint32_t off = 0; off < span; off += kPiece)
                    bulk_load(dst + off, row - ri.mis + off, min(kPiece, span - off), landed(buf, 0));
                mbar_arrive_expect_tx(landed(buf, 1), 0);
            } else {
                mbar_arrive_expect_tx(landed(buf, 0), head_bytes);   // release: publishes s_row[buf]
                for (uint32_t off = 0; off < head_bytes; off += kPiece)
                    bulk_load(dst + off, row + off, min(kPiece, head_bytes - off), landed(buf, 0));
                mbar_arrive_expect_tx(landed(buf, 1), da.row_bytes - head_bytes);
                for (uint32_t off = head_bytes; off < da.row_bytes; off += kPiece)
                    bulk_load(dst + off, row + off, min(kPiece, da.row_bytes - off), landed(buf, 1));
            }
            if (rows_mine > 0) {
                const long long target = ((i + 1) * pads_early) / rows_mine;
                while (pads_done < target) { zero_fill_next(); ++pads_done; }
            }
        }
        while (pads_done < pads_mine) { zero_fill_next(); ++pads_done; }
        // the last two rows
        for (long long j = i >= 2 ? i - 2 : 0; j < i && !aborted; ++j) drain(j);
        bulk_wait_all();
        return;
    }

    // ---------------------------------------------------------------- consumers
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const int cnt0 = (uint32_t)tid < nvec ? (int)((nvec - tid + kCons - 1) / kCons) : 0;   // this thread's vectors
    const int head_cnt0 = min(cnt0, (int)(head_vecs / kCons) + ((uint32_t)tid < head_vecs % kCons ? 1 : 0));
    // the block's slice of the value loss, while its first row is still on the way (thread 0 keeps the sums)
    double sum_pg = 0.0, sum_vf = 0.0;
    if (p.fused) sum_vf = consumer_sum_double<NW>(value_loss_slice(p, N, tid, kCons), s_dbl, warp, lane);

    long long i = 0;
    for (long long k = blockIdx.x; k < N; k += G, ++i) {
        const int buf = (int)(i & 1), par = buf;
        const uint32_t use = (uint32_t)(i >> 1) & 1u;
        mbar_wait(landed(buf, 0), use, p.status, aborted, p.wait_limit_ns);
        RowInfo ri = s_row[buf];
        if (aborted) { ri.y = 0; ri.bad_id = 1; ri.flat = 0; }      // stale row info: touch nothing
        // where the row sits in the buffer: eoff entries of vector 0 precede it (kAny), vectors [0, row_vecs)
        const uint32_t eoff = kAny ? (ri.mis >> 1) : 0u;
        int cnt = cnt0, head_cnt = head_cnt0;
        int jfirst = -1, jlast = -1;                               // this thread's vectors with entries outside the row
        if (kAny) {
            const uint32_t row_vecs = (ri.mis + da.row_bytes + 15u) >> 4;
            cnt = (uint32_t)tid < row_vecs ? (int)((row_vecs - tid + kCons - 1) / kCons) : 0;
            head_cnt = cnt;
            if (eoff != 0 && tid == 0) jfirst = 0;
            if (((eoff + (uint32_t)p.V) & 7u) != 0 && ((row_vecs - 1) % kCons) == (uint32_t)tid) jlast = (int)((row_vecs - 1) / kCons);
        }
        const uint32_t yvec = (eoff + (uint32_t)ri.y) >> 3;
        const int yj = (int)((eoff + (uint32_t)ri.y) & 7u);
        const bool owner = (yvec % kCons) == (uint32_t)tid;
        const int jy = owner ? (int)(yvec / kCons) : -1;            // which of this thread's vectors holds the label
        // one vector of this thread, with whatever is special about it
        // (kAny) the first and last vector of the row, foreign entries turned into -inf; any other vector unchanged
        auto in_row = [&](const uint4& q, int j) {
            if (kAny && j == jfirst) return mask_vec_outside<kF16>(q, (int)eoff, 8);
            if (kAny && j == jlast) return mask_vec_outside<kF16>(q, 0, (int)((eoff + (uint32_t)p.V) & 7u));
            return q;
        };
        auto add_special = [&](Acc& acc, const uint4& q, int j, float& zy_out) {
            if (j == jy) zy_out = acc_add_vec_label<kF16>(acc, in_row(q, j), yj);
            else acc_add_vec<kF16>(acc, in_row(q, j));
        };
        const uint4* src = (const uint4*)(smem + (size_t)buf * da.row_stride) + tid;

        // ---- pass 1: partition sum
        // Every thread sums against the same reference exponent, taken from one vector of the row that all
        // threads can see, so that the partial sums of the block add up without rescaling.  Blocks of 4 vectors
        // are summed without range handling and their sums checked afterwards, once per row: a thread that met
        // an entry 2^64 above the reference (or found no usable reference) redoes its share of the row with
        // the careful routines under a reference of its own, and the block then merges by the general rule.
        const float Mref = max8_scaled<kF16>(((const uint4*)(smem + (size_t)buf * da.row_stride))[(kAny && eoff != 0) ? 1 : 0]);
        Acc a = acc_empty();
        float zy = 0.f;
        bool redo = !(Mref > kFloorM);
        a.M = Mref;
        auto sum_range = [&](int j0, int j1) {
            int j = j0;
            for (; j + 4 <= j1; j += 4) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) q[u] = src[(size_t)(j + u) * kCons];
                if (kAny && ((unsigned)(jfirst - j) < 4u || (unsigned)(jlast - j) < 4u)) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) q[u] = in_row(q[u], j + u);
                }
                if ((unsigned)(jy - j) < 4u) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (j + u == jy) zy = acc_add_vec_label<kF16>(a, q[u], yj);
                        else acc_add_vec<kF16>(a, q[u]);
                    }
                } else {
                    const float vs = exp_sum_vecs<4, kF16>(q, -a.M);
                    a.s += vs;
                    redo |= !(vs <= 1.8446744e19f);
                }
            }
            for (; j < j1; ++j) add_special(a, src[(size_t)j * kCons], j, zy);
        };
        sum_range(0, head_cnt);
        mbar_wait(landed(buf, 1), use, p.status, aborted, p.wait_limit_ns);
        sum_range(head_cnt, cnt);
        if (redo) {
            a = acc_empty();
            zy = 0.f;
            for (int j = 0; j < cnt; ++j) add_special(a, src[(size_t)j * kCons], j, zy);
        }
        const bool diverged = cnt > 0 && a.M != Mref;               // (a careful routine may also have raised the reference)

        if (owner) s_lab[par] = LabelInfo{zy, a.ey, a.M, 0.f};
        float ws = cnt > 0 ? a.s : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
        if (lane == 0) s_sum[par][warp] = ws;
        Acc tot;
        if (!consumer_barrier_or<NW>(diverged)) {
            // common case: one reference for the whole block; every thread adds the warp sums in the same fixed tree
            tot.M = Mref;
            tot.s = sum_warp_sums<NW>(s_sum[par]);
            tot.ey = s_lab[par].ey;
        } else {
            Acc mine = a;
            if (cnt == 0) mine = acc_empty();
            tot = dbuf_reduce<NW>(mine, s_part[par], &s_lab[par], warp, lane);
        }
        const RowResult r = row_finish_fast(tot, s_lab[par].zy);

        float loss = 0.f, g = 0.f;
        if (!ri.bad_id) ppo_token<true>(r.lp, ri.lp_old, ri.adv, p.clip_eps, scale_over_N, loss, g);
        if (tid == 0 && !aborted) {
            if (p.fused) sum_pg += (double)loss; else p.row_loss[ri.flat] = loss;
            if (p.out_lp_new) p.out_lp_new[ri.flat] = ri.bad_id ? 0.f : r.lp;
        }

        // ---- pass 2: the gradient overwrites the logits in the buffer
        uint4* dst = (uint4*)(smem + (size_t)buf * da.row_stride) + tid;
        if (g == 0.f) {
            for (int j = 0; j < cnt; ++j) dst[(size_t)j * kCons] = make_uint4(0, 0, 0, 0);
        } else {
            const float c2 = lg2(fabsf(g)) - r.lse2;
            const uint32_t sign2 = g > 0.f ? 0x80008000u : 0u;
            const float dy = g * r.one_m_py;
            int j = 0;
            for (; j + 4 <= cnt; j += 4) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) q[u] = src[(size_t)(j + u) * kCons];
                uint4 o[4];
                grad_vecs<4, kF16>(q, o, c2, sign2);
                if ((unsigned)(jy - j) < 4u) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (j + u == jy) patch_label<kF16>(o[u], yj, dy);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) dst[(size_t)(j + u) * kCons] = o[u];
            }
            for (; j < cnt; ++j) {
                uint4 o = grad_vec<kF16>(src[(size_t)j * kCons], c2, sign2);
                if (j == jy) patch_label<kF16>(o, yj, dy);
                dst[(size_t)j * kCons] = o;
            }
        }
        fence_async_smem();                                         // this thread's writes, before the bulk store reads them
        __syncwarp();
        if (lane == 0) mbar_arrive(computed(buf));
    }
    if (p.fused && tid == 0) publish_block_losses(p, N, sum_pg, sum_vf);
}

}  // namespace rlhf
