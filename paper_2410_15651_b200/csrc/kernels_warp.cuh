// Log-prob kernel for 16-byte aligned rows: one warp per row, no block-level synchronisation.
//
// Every warp streams its own rows through a private two-slot ring in shared memory: lane 0 issues
// the bulk asynchronous copies (4 KB chunks, one mbarrier per slot) and runs two chunks ahead of the
// warp, across row boundaries; all 32 lanes sum the chunk that has landed.  The per-row reduction is
// a handful of shuffles inside the warp, so no warp ever waits for another one: while one warp
// finishes a row the others keep the special-function unit and the memory pipe busy.  With 24 warps
// per SM about 190 KB of loads are in flight per SM, and short batches (fewer rows than warps)
// still spread evenly: every row is in flight at once.
#pragma once
#include "kernels_ring.cuh"

namespace rlhf {

constexpr int kWarpChunk = 4096;                  // bytes per bulk copy
constexpr int kWarpSlots = 2;
constexpr int kWarpChunkVecs = kWarpChunk / 16;   // 256 vectors: 8 per lane

// 32-bit walk over the valid tokens (B*T is at most 2^30): b and the number of valid tokens before b.
struct Cursor32 {
    int b;
    int acc;
};
__device__ __forceinline__ bool cursor32_seek(Cursor32& c, int k, const int* __restrict__ lengths, int B, int T,
                                              int& b, int& t)
{
    while (c.b < B) {
        const int len = clamp_len(__ldg(lengths + c.b), T);
        if (k < c.acc + len) { b = c.b; t = k - c.acc; return true; }
        c.acc += len;
        ++c.b;
    }
    return false;
}

struct WarpArgs {
    RowArgs row;            // logits / out_lp: the (first) tensor
    unsigned row_bytes;     // 2*V, multiple of 16
    // kDual: a second logits tensor (the reference model's) read with the same ids in the same launch
    const uint16_t* logits2;
    long long stride2_b, stride2_t;
    float* out_lp2;
    // kEnt: entropy of the softmax of every valid row of the (first) tensor, 0 at padded positions
    float* out_entropy;
};

// ---- sums that also carry what the entropy needs.  Beside (M, s, ey) of Acc a thread keeps
//      ez = sum over the entries that are not the generated token of e * xr,   xr = max(x - M, -150),  e = 2^xr
// (the clamp turns a deleted entry's -inf into a finite factor of a term that is 0 anyway).  Raising the reference
// by d scales s and ey by 2^-d and turns ez into 2^-d * (ez - d * s).
constexpr float kEntClamp = -150.f;

__device__ __forceinline__ void acc_rebase_ent(Acc& a, float& ez, float newM)
{
    const float d = newM - a.M;
    const float sc = ex2(-d);
    ez = sc * (ez - d * a.s);
    a.s *= sc;
    a.ey *= sc;
    a.M = newM;
}

__device__ __forceinline__ void acc_add_ent(Acc& a, float& ez, float z, bool is_label)
{
    const float x = z * kLog2e;
    if (x - a.M > kRebase) acc_rebase_ent(a, ez, x);
    const float xr = fmaxf(x - a.M, kEntClamp);
    const float e = ex2(xr);
    if (is_label) a.ey = e;
    else { a.s += e; ez = fmaf(e, xr, ez); }
}

// Entries [jlo, jhi) of a vector, entry jlabel (if in range) being the generated token; returns its logit (else 0).
template <bool kF16>
__device__ __forceinline__ float acc_add_vec_ent(Acc& a, float& ez, const uint4& q, int jlo, int jhi, int jlabel)
{
    float z[8];
    unpack8<kF16>(q, z);
    float zy = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i >= jlo && i < jhi) {
            acc_add_ent(a, ez, z[i], i == jlabel);
            if (i == jlabel) zy = z[i];
        }
    }
    return zy;
}

// U whole vectors without the generated token against one reference: sum of e and sum of e * xr.
template <int U, bool kF16>
__device__ __forceinline__ float2 exp_sum_vecs_ent(const uint4 (&q)[U], float negM)
{
    float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    float2 accz[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float2 x = __ffma2_rn(El<kF16>::unpack2(w[k]), splat2(kLog2e), splat2(negM));
            x.x = fmaxf(x.x, kEntClamp);
            x.y = fmaxf(x.y, kEntClamp);
            const float2 e = make_float2(ex2(x.x), ex2(x.y));
            acc[k & 1] = __fadd2_rn(acc[k & 1], e);
            accz[k & 1] = __ffma2_rn(e, x, accz[k & 1]);
        }
    }
    return make_float2((acc[0].x + acc[0].y) + (acc[1].x + acc[1].y), (accz[0].x + accz[0].y) + (accz[1].x + accz[1].y));
}

inline size_t warp_kernel_smem_bytes(int warps_per_block)
{
    return (size_t)warps_per_block * (kWarpSlots * kWarpChunk + kWarpSlots * 8);
}

// kAny: rows may start at any even byte address and have any length (V not a multiple of 8): every row
// is then loaded as the 16-byte aligned span that contains it, and the entries of the first and last
// vector that lie outside the row are skipped.  (The span stays inside the 16-byte blocks that hold the
// row's first and last element.)
// kF16: the logits are IEEE binary16 instead of bf16.  kEnt: also write the entropy of every valid row.
template <int WPB, bool kDual, bool kAny, bool kF16 = false, bool kEnt = false>
__global__ void __launch_bounds__(WPB * 32, 1) logprob_warp_kernel(WarpArgs wa)
{
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];

    const RowArgs& p = wa.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* ring = smem + (size_t)warp * (kWarpSlots * kWarpChunk);
    const uint32_t ring_addr = smem_u32(ring);
    const uint32_t bar_addr = smem_u32(smem + (size_t)WPB * (kWarpSlots * kWarpChunk)) + (uint32_t)warp * (kWarpSlots * 8);

    if (lane == 0) {
        for (int s = 0; s < kWarpSlots; ++s) mbar_init(bar_addr + 8u * s, 1);
        fence_mbar_init();
    }
    pdl_wait_prior_grid();                       // nothing above touches global memory
    pdl_release_next_grid();
    const int N1 = (int)block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    __syncthreads();

    // log-prob 0 at padded tokens
    {
        const long long total = (long long)p.B * p.T;
        for (long long i = (long long)blockIdx.x * blockDim.x + tid; i < total; i += (long long)gridDim.x * blockDim.x) {
            int b = (int)(i / p.T), t = (int)(i % p.T);
            if (t >= clamp_len(__ldg(p.lengths + b), p.T)) {
                p.out_lp[i] = 0.f;
                if (kDual) wa.out_lp2[i] = 0.f;
                if (kEnt) wa.out_entropy[i] = 0.f;
            }
        }
    }

    // rows are dealt to blocks first, then to warps: consecutive rows go to different SMs, and a batch
    // with fewer rows than warps still loads every SM equally
    const int N = kDual ? 2 * N1 : N1;                              // rows: tensor 1, then tensor 2
    const int gw = warp * (int)gridDim.x + (int)blockIdx.x;       // this warp's first row
    const int GW = (int)gridDim.x * WPB;
    const uint32_t nvec = wa.row_bytes / 16u;
    const int nchunks = (int)((wa.row_bytes + kWarpChunk - 1) / kWarpChunk);
    const int full_chunks = (int)(wa.row_bytes / kWarpChunk);

    // ---- issue side (lane 0 only uses it): next chunk to request
    Cursor32 icur{0, 0};
    int ik = gw;          // row of the next chunk to request
    int ic = 0;                 // its chunk index
    int islot = 0;
    const unsigned char* irow = nullptr;
    uint32_t ispan = wa.row_bytes;    // bytes to load for the row being requested
    int inchunks = nchunks;
    bool iwrapped = false;
    auto issue_seek = [&]() {
        int b, t;
        const bool second = kDual && ik >= N1;
        if (second && !iwrapped) { icur = Cursor32{0, 0}; iwrapped = true; }
        if (ik < N && cursor32_seek(icur, second ? ik - N1 : ik, p.lengths, p.B, p.T, b, t))
            irow = second ? (const unsigned char*)(wa.logits2 + (long long)b * wa.stride2_b + (long long)t * wa.stride2_t)
                          : (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t);
        else
            ik = N;
        if (kAny && ik < N) {
            const uint32_t mis = (uint32_t)((uintptr_t)irow & 15u);
            irow -= mis;
            ispan = (mis + wa.row_bytes + 15u) & ~15u;
            inchunks = (int)((ispan + kWarpChunk - 1) / kWarpChunk);
        }
    };
    auto issue_next = [&]() {
        if (ik >= N) return;
        const uint32_t off = (uint32_t)ic * kWarpChunk;
        const uint32_t bytes = min((uint32_t)kWarpChunk, ispan - off);
        mbar_arrive_expect_tx(bar_addr + 8u * islot, bytes);
        bulk_load(ring_addr + (uint32_t)islot * kWarpChunk, irow + off, bytes, bar_addr + 8u * islot);
        islot = islot + 1 == kWarpSlots ? 0 : islot + 1;
        if (++ic == inchunks) { ic = 0; ik += GW; issue_seek(); }
    };
    if (lane == 0) {
        issue_seek();
        for (int s = 0; s < kWarpSlots; ++s) issue_next();
    }

    // ---- consume side
    Cursor32 cur{0, 0};
    bool aborted = false;
    int slot = 0;
    uint32_t phases = 0;        // bit s: parity to wait for on slot s
    int nb = 0, nt = 0;
    long long ny = 0;
    bool wrapped = false;
    auto fetch_row = [&](int k) {
        const bool second = kDual && k >= N1;
        if (second && !wrapped) { cur = Cursor32{0, 0}; wrapped = true; }
        if (k < N && cursor32_seek(cur, second ? k - N1 : k, p.lengths, p.B, p.T, nb, nt))
            ny = __ldg(p.ids + (long long)nb * p.ids_stride_b + nt);
    };
    fetch_row(gw);

    for (int k = gw; k < N; k += GW) {
        const int flat = nb * p.T + nt;
        long long y = ny;
        const bool bad_id = (y < 0 || y >= p.V);
        if (bad_id) { y = 0; if (lane == 0) atomicOr(p.status, kErrIdRange); }
        // where the row sits in the loaded span: eoff entries of the first vector precede it
        uint32_t eoff = 0, row_vecs = nvec;
        int row_chunks = nchunks, plain_end = full_chunks;         // chunks [plain_begin, plain_end) hold only whole vectors of the row
        if (kAny) {
            const bool second = kDual && k >= N1;
            const uint16_t* rp = second ? wa.logits2 + (long long)nb * wa.stride2_b + (long long)nt * wa.stride2_t
                                        : p.logits + (long long)nb * p.stride_b + (long long)nt * p.stride_t;
            const uint32_t mis = (uint32_t)((uintptr_t)rp & 15u);
            eoff = mis >> 1;
            const uint32_t span = (mis + wa.row_bytes + 15u) & ~15u;
            row_vecs = span / 16u;
            row_chunks = (int)((span + kWarpChunk - 1) / kWarpChunk);
            plain_end = (int)(((eoff + (uint32_t)p.V) >> 3) / kWarpChunkVecs);
        }
        const int plain_begin = (kAny && eoff != 0) ? 1 : 0;
        const uint32_t yvec = (uint32_t)((eoff + (uint32_t)y) >> 3);
        const int yj = (int)((eoff + (uint32_t)y) & 7);
        const int ychunk = (int)(yvec / kWarpChunkVecs);
        fetch_row(k + GW);                                          // next row's token id, in flight during this row

        Acc a = acc_empty();
        float zy = 0.f;
        float ez = 0.f;                                             // kEnt only
        for (int c = 0; c < row_chunks; ++c) {
            mbar_wait(bar_addr + 8u * slot, (phases >> slot) & 1u, p.status, aborted, p.wait_limit_ns);
            phases ^= 1u << slot;
            const uint4* src = (const uint4*)(ring + (size_t)slot * kWarpChunk) + lane;
            if (c >= plain_begin && c < plain_end && c != ychunk) {
                if (c == 0) {                                       // this lane's reference exponent for the row
                    const float m0 = max8_scaled<kF16>(src[0]);
                    if (kEnt) { if (m0 > kFloorM) a.M = m0; } else a.M = m0;
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint4 q[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) q[u] = src[(4 * h + u) * 32];
                    if (kEnt) {
                        const float2 vs = exp_sum_vecs_ent<4, kF16>(q, -a.M);
                        if (vs.x <= 1.8446744e19f && a.M > kFloorM) {
                            a.s += vs.x;
                            ez += vs.y;
                        } else {
#pragma unroll
                            for (int u = 0; u < 4; ++u) acc_add_vec_ent<kF16>(a, ez, q[u], 0, 8, -1);
                        }
                    } else {
                        const float vs = exp_sum_vecs<4, kF16>(q, -a.M);
                        if (vs <= 1.8446744e19f) {
                            a.s += vs;
                        } else {
#pragma unroll
                            for (int u = 0; u < 4; ++u) acc_add_vec<kF16>(a, q[u]);
                        }
                    }
                }
            } else {
                const uint32_t v0 = (uint32_t)c * kWarpChunkVecs + lane;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const uint32_t v = v0 + u * 32;
                    if (v < row_vecs) {
                        const uint4 q = src[u * 32];
                        const int e0 = (int)(v * 8u) - (int)eoff;      // row index of the vector's first entry
                        if (kEnt) {
                            zy += acc_add_vec_ent<kF16>(a, ez, q, max(0, -e0), min(8, p.V - e0), v == yvec ? yj : -1);
                        } else if (kAny && (e0 < 0 || e0 + 8 > p.V))
                            zy += acc_add_vec_range<kF16>(a, q, max(0, -e0), min(8, p.V - e0), v == yvec ? yj : -1);
                        else if (v == yvec) zy = acc_add_vec_label<kF16>(a, q, yj);
                        else acc_add_vec<kF16>(a, q);
                    }
                }
            }
            __syncwarp();                                           // every lane is done with the slot
            if (lane == 0) issue_next();
            slot = slot + 1 == kWarpSlots ? 0 : slot + 1;
        }

        // warp-wide total: common reference, one rescale, sums by shuffle; the label's owner lane broadcasts its term
        float M = a.M;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        const float sc = ex2(a.M - M);
        float s = a.s * sc;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const int owner = (int)(yvec & 31u);
        const float ey = __shfl_sync(0xffffffffu, a.ey * sc, owner);
        zy = __shfl_sync(0xffffffffu, zy, owner);
        float ezw = 0.f;
        if (kEnt) {
            // every lane's ez against the common reference (see acc_rebase_ent), then the warp's sum
            ezw = sc * (ez - (M - a.M) * a.s);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ezw += __shfl_xor_sync(0xffffffffu, ezw, o);
        }
        if (lane == 0 && !aborted) {
            const RowResult r = row_finish(Acc{M, s, ey}, zy);
            float* out = (kDual && k >= N1) ? wa.out_lp2 : p.out_lp;
            out[flat] = bad_id ? 0.f : r.lp;
            if (kEnt && !(kDual && k >= N1)) {
                // H = ln2 * (log2 S - (sum_v e_v (x_v - M)) / S),  S = s + ey; the generated token's term joins the sum here
                const float S = s + ey;
                const float xyr = fmaxf(fmaf(zy, kLog2e, -M), kEntClamp);
                wa.out_entropy[flat] = kLn2 * (log2f(S) - (ezw + ey * xyr) / S);
            }
        }
    }
}

}  // namespace rlhf
