// Loss forward/backward for rows of which two fit in shared memory (16 KB <= row <= ~111 KB,
// i.e. vocabularies from 8K to 56K entries in bf16) -- the OPT- and Llama-2-shaped cases.
//
// One persistent block per SM: NW consumer warps work on one row at a time, a producer thread keeps
// the other row buffer filling.  While row i is reduced (pass 1) and turned into dlogits (pass 2)
// out of buffer i&1, the bulk copies of row i+1 into the other buffer are already in flight, having
// been issued when that buffer was released a whole row-time earlier; so, except for the very
// first row of a block, consumers never wait for HBM, and DRAM sees each row read once and written
// once.  Synchronisation is per row, not per chunk: two "landed" mbarriers per buffer (a 4-vector
// head part so that the first row can start early, and the rest) and one "released" mbarrier.
// Inside a row every thread runs straight-line blocks of 4 vectors (32 logits) with no per-vector
// branch: range checks are per block, and only the block that holds the generated token takes the
// careful path.
#pragma once
#include "kernels_ring.cuh"

namespace rlhf {

struct DbufArgs {
    RowArgs row;
    unsigned row_bytes;     // 2*V, multiple of 16
    unsigned row_stride;    // row_bytes rounded up to 128: distance between the two buffers
};

inline size_t dbuf_smem_bytes(unsigned row_bytes)
{
    const size_t stride = ((size_t)row_bytes + 127) & ~(size_t)127;
    return 2 * stride + kZeroBytes + 64;       // + 6 mbarriers
}

template <int NW>
__global__ void __launch_bounds__(NW * 32 + 32, 1) loss_dbuf_kernel(DbufArgs da)
{
    constexpr int kCons = NW * 32;
    constexpr int kThreads = kCons + 32;
    constexpr uint32_t kPiece = 16384;           // size of one bulk copy
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ float2 s_part[2][32];
    __shared__ LabelInfo s_lab[2];

    const RowArgs& p = da.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t buf_addr = smem_u32(smem);
    unsigned char* zero_buf = smem + 2 * (size_t)da.row_stride;
    const uint32_t bar_addr = smem_u32(zero_buf + kZeroBytes);
    // barriers: landed[buf][part] at bar_addr + 8*(2*buf+part), released[buf] at bar_addr + 32 + 8*buf
    auto landed = [&](int buf, int part) { return bar_addr + 8u * (2 * buf + part); };
    auto released = [&](int buf) { return bar_addr + 32u + 8u * buf; };

    const uint32_t nvec = da.row_bytes / 16u;
    // head part: the first 4 vectors of every thread, if the row has at least twice that
    const uint32_t head_vecs = nvec >= 8u * kCons ? 4u * kCons : nvec;
    const uint32_t head_bytes = head_vecs * 16u;

    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const long long G = gridDim.x;

    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(bar_addr + 8u * i, 1);
        mbar_init(released(0), NW);
        mbar_init(released(1), NW);
        fence_mbar_init();
    }
    for (int i = tid; i < kZeroBytes / 16; i += kThreads) ((uint4*)zero_buf)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    __syncthreads();

    bool aborted = false;

    if (warp == NW) {
        // ------------------------------------------------------------ producer
        if (lane != 0) return;
        const long long n_pad = (long long)p.B * p.T - N;
        const long long rows_mine = N > blockIdx.x ? (N - blockIdx.x + G - 1) / G : 0;
        const long long pads_mine = n_pad > blockIdx.x ? (n_pad - blockIdx.x + G - 1) / G : 0;
        Cursor cur{0, 0}, pcur{0, 0};
        long long pads_done = 0;
        auto zero_fill_next = [&]() {
            int b, t;
            if (!cursor_seek_padded(pcur, blockIdx.x + pads_done * G, p.lengths, p.B, p.T, b, t)) return;
            unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t);
            for (uint32_t off = 0; off < da.row_bytes; off += kZeroBytes)
                bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kZeroBytes, da.row_bytes - off));
            bulk_commit();
        };
        long long i = 0;
        for (long long k = blockIdx.x; k < N && !aborted; k += G, ++i) {
            int b, t;
            if (!cursor_seek_valid(cur, k, p.lengths, p.B, p.T, b, t)) break;
            const unsigned char* row = (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t);
            const int buf = (int)(i & 1);
            const uint32_t use = (uint32_t)(i >> 1) & 1u;            // parity of this use of the buffer
            mbar_wait(released(buf), use ^ 1u, p.status, aborted);
            if (aborted) break;
            const uint32_t dst = buf_addr + (uint32_t)buf * da.row_stride;
            mbar_arrive_expect_tx(landed(buf, 0), head_bytes);
            for (uint32_t off = 0; off < head_bytes; off += kPiece)
                bulk_load(dst + off, row + off, min(kPiece, head_bytes - off), landed(buf, 0));
            mbar_arrive_expect_tx(landed(buf, 1), da.row_bytes - head_bytes);
            for (uint32_t off = head_bytes; off < da.row_bytes; off += kPiece)
                bulk_load(dst + off, row + off, min(kPiece, da.row_bytes - off), landed(buf, 1));
            if (rows_mine > 0) {
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
    const int cnt = (uint32_t)tid < nvec ? (int)((nvec - tid + kCons - 1) / kCons) : 0;   // this thread's vectors
    const int head_cnt = min(cnt, (int)(head_vecs / kCons) + ((uint32_t)tid < head_vecs % kCons ? 1 : 0));

    Cursor cur{0, 0};
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

    long long i = 0;
    for (long long k = blockIdx.x; k < N; k += G, ++i) {
        const int b = nb, t = nt;
        long long y = ny;
        const float lp_old = n_lp_old, adv = n_adv;
        const long long flat = (long long)b * p.T + t;
        const bool bad_id = (y < 0 || y >= p.V);
        if (bad_id) { y = 0; if (tid == 0) atomicOr(p.status, kErrIdRange); }
        const uint32_t yvec = (uint32_t)(y >> 3);
        const int yj = (int)(y & 7);
        const bool owner = (yvec % kCons) == (uint32_t)tid;
        const int jy = owner ? (int)(yvec / kCons) : -1;            // which of this thread's vectors holds the label

        const int buf = (int)(i & 1), par = buf;
        const uint32_t use = (uint32_t)(i >> 1) & 1u;
        const uint4* src = (const uint4*)(smem + (size_t)buf * da.row_stride) + tid;

        // ---- pass 1: partition sum
        Acc a = acc_empty();
        float zy = 0.f;
        auto sum_range = [&](int j0, int j1) {
            int j = j0;
            for (; j + 4 <= j1; j += 4) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) q[u] = src[(size_t)(j + u) * kCons];
                if (jy >= j && jy < j + 4) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (j + u == jy) zy = acc_add_vec_label(a, q[u], yj);
                        else acc_add_vec(a, q[u]);
                    }
                } else {
                    const float vs = exp_sum_vecs<4>(q, -a.M);
                    if (vs <= 1.8446744e19f) {
                        a.s += vs;
                    } else {
#pragma unroll
                        for (int u = 0; u < 4; ++u) acc_add_vec(a, q[u]);
                    }
                }
            }
            for (; j < j1; ++j) {
                const uint4 q = src[(size_t)j * kCons];
                if (j == jy) zy = acc_add_vec_label(a, q, yj);
                else acc_add_vec(a, q);
            }
        };
        mbar_wait(landed(buf, 0), use, p.status, aborted);
        if (cnt > 0 && jy != 0) a.M = max8_scaled(src[0]);          // this thread's reference exponent for the row
        sum_range(0, head_cnt);
        mbar_wait(landed(buf, 1), use, p.status, aborted);
        sum_range(head_cnt, cnt);

        if (owner) s_lab[par] = LabelInfo{zy, a.ey, a.M, 0.f};
        const Acc tot = consumer_reduce<NW>(a, s_part[par], &s_lab[par], warp, lane);
        const RowResult r = row_finish(tot, s_lab[par].zy);

        fetch_row(k + G);                                           // next row's scalars, in flight during pass 2

        float loss = 0.f, g = 0.f;
        if (!bad_id) ppo_token(r.lp, lp_old, adv, p.clip_eps, scale_over_N, loss, g);
        if (tid == 0) {
            p.row_loss[flat] = loss;
            if (p.out_lp_new) p.out_lp_new[flat] = bad_id ? 0.f : r.lp;
        }

        // ---- pass 2: dlogits from the resident row
        unsigned char* dst = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t) +
                             (size_t)tid * 16;
        if (g == 0.f) {
            for (int j = 0; j < cnt; ++j) store_v4(dst + (size_t)j * kCons * 16, make_uint4(0, 0, 0, 0));
        } else {
            const float c2 = log2f(fabsf(g)) - r.lse2;
            const uint32_t sign2 = g > 0.f ? 0x80008000u : 0u;
            const float dy = g * r.one_m_py;
            int j = 0;
            for (; j + 4 <= cnt; j += 4) {
                uint4 q[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) q[u] = src[(size_t)(j + u) * kCons];
                uint4 o[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) o[u] = grad_vec(q[u], c2, sign2);
                if (jy >= j && jy < j + 4) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (j + u == jy) patch_label(o[u], yj, dy);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) store_v4(dst + (size_t)(j + u) * kCons * 16, o[u]);
            }
            for (; j < cnt; ++j) {
                uint4 o = grad_vec(src[(size_t)j * kCons], c2, sign2);
                if (j == jy) patch_label(o, yj, dy);
                store_v4(dst + (size_t)j * kCons * 16, o);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(released(buf));
    }
}

}  // namespace rlhf
