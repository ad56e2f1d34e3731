// Fast row kernels for 16-byte aligned rows (sm_100a).
//
// Each persistent block owns a ring of shared-memory slots.  One elected producer thread streams
// the block's rows into the ring with bulk asynchronous copies (cp.async.bulk, completion counted
// on an mbarrier per slot); 8 consumer warps reduce the slots as they land.  HBM latency is
// covered by the bytes the ring keeps in flight, not by registers or occupancy.
//
//   log-prob kernel   every slot is released as soon as it has been summed (streaming).
//   loss kernel       if a whole row fits in the ring ("resident"), the row is summed as it lands,
//                     kept, and then turned into dlogits straight from shared memory, so that DRAM
//                     sees one read and one write per row; slots are released chunk by chunk in
//                     the second pass and refilled with the next row at once.  Rows larger than
//                     the ring are streamed twice (the second read is served by L2).
//                     Padded rows are zero-filled by bulk stores from a zeroed shared buffer,
//                     issued by the producer thread between its loads.
//
// Work assignment is static: block i takes valid rows i, i+G, i+2G, ... (and padded rows likewise),
// so results never depend on timing.  Every wait on an mbarrier is bounded; if one runs out the
// thread flags RLHF_ERR_TIMEOUT, stops waiting and lets the block drain.
#pragma once
#include "common.cuh"
#include "kernels_generic.cuh"

namespace rlhf {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kRingThreads = kConsumerThreads + 32;
constexpr int kZeroBytes = 4096;                       // zeroed buffer that feeds the bulk zero-fill
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

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
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, unsigned* status)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > kWaitLimitNs) {
            atomicOr(status, kErrTimeout);
            return false;
        }
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, unsigned* status, bool& aborted)
{
    if (aborted) return;
    if (mbar_try_wait(bar, parity)) return;
    if (!mbar_wait_slow(bar, parity, status)) aborted = true;
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
__device__ __forceinline__ void consumer_barrier()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ void store_v4(void* p, const uint4& q)
{
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(q.x), "r"(q.y), "r"(q.z), "r"(q.w)
                 : "memory");
}

// ---------------------------------------------------------------- 8 logits at a time
__device__ __forceinline__ void unpack8(const uint4& q, float (&z)[8])
{
    z[0] = bf16_lo(q.x); z[1] = bf16_hi(q.x);
    z[2] = bf16_lo(q.y); z[3] = bf16_hi(q.y);
    z[4] = bf16_lo(q.z); z[5] = bf16_hi(q.z);
    z[6] = bf16_lo(q.w); z[7] = bf16_hi(q.w);
}

// Adds 8 entries none of which is the generated token.  The exponentials are formed against the
// thread's current reference first; only if their sum is out of range (first vector of a thread, or
// a logit more than 64 binades above the reference) is the reference raised and the vector redone.
__device__ __forceinline__ void acc_add_vec(Acc& a, const uint4& q)
{
    float z[8], e[8];
    unpack8(q, z);
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
__device__ __forceinline__ float acc_add_vec_label(Acc& a, const uint4& q, int j)
{
    float z[8];
    unpack8(q, z);
    float zy = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        acc_add(a, z[i], i == j);
        if (i == j) zy = z[i];
    }
    return zy;
}

// dlogits for 8 entries: sign * 2^(x + c2), packed to bf16.
__device__ __forceinline__ uint4 grad_vec(const uint4& q, float c2, uint32_t sign2)
{
    float z[8], d[8];
    unpack8(q, z);
#pragma unroll
    for (int i = 0; i < 8; ++i) d[i] = ex2(fmaf(z[i], kLog2e, c2));
    uint4 o;
    o.x = pack_bf16x2(d[0], d[1]) ^ sign2;
    o.y = pack_bf16x2(d[2], d[3]) ^ sign2;
    o.z = pack_bf16x2(d[4], d[5]) ^ sign2;
    o.w = pack_bf16x2(d[6], d[7]) ^ sign2;
    return o;
}

__device__ __forceinline__ void patch_label(uint4& o, int j, float value)
{
    const uint32_t h = pack_bf16x2(value, 0.f) & 0xffffu;
    uint32_t* w = j < 2 ? &o.x : (j < 4 ? &o.y : (j < 6 ? &o.z : &o.w));
    *w = (j & 1) ? ((*w & 0x0000ffffu) | (h << 16)) : ((*w & 0xffff0000u) | h);
}

// ---------------------------------------------------------------- the kernel
// Dynamic shared memory: [n_slots * chunk][full barriers n_slots * 8][empty barriers n_slots * 8][zero buffer].
template <bool kLoss, int U>
__global__ void __launch_bounds__(kRingThreads) row_ring_kernel(RingArgs ra)
{
    constexpr uint32_t kChunk = (uint32_t)kConsumerThreads * 16u * U;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ long long s_cnt[33];
    __shared__ Acc s_part[2][kConsumerWarps];
    __shared__ float s_zy[2];

    const RowArgs& p = ra.row;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = ra.n_slots, chunks = ra.chunks_per_row;
    const uint32_t slots_addr = smem_u32(smem);
    const uint32_t full_addr = slots_addr + (uint32_t)S * kChunk;
    const uint32_t empty_addr = full_addr + (uint32_t)S * 8u;
    unsigned char* zero_buf = smem + (size_t)S * kChunk + (size_t)S * 16;

    const long long N = block_count_valid(p.lengths, p.B, p.T, s_cnt, blockIdx.x == 0 ? p.status : nullptr);
    const long long G = gridDim.x;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_addr + 8u * s, 1);
            mbar_init(empty_addr + 8u * s, kConsumerWarps);
        }
        fence_mbar_init();
    }
    if (kLoss) {
        for (int i = tid; i < kZeroBytes / 16; i += kRingThreads) ((uint4*)zero_buf)[i] = make_uint4(0, 0, 0, 0);
        fence_async_smem();
    }
    __syncthreads();

    bool aborted = false;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane != 0) return;
        const long long n_pad = (long long)p.B * p.T - N;
        const long long rows_mine = N > blockIdx.x ? (N - blockIdx.x + G - 1) / G : 0;
        const long long pads_mine = (kLoss && n_pad > blockIdx.x) ? (n_pad - blockIdx.x + G - 1) / G : 0;
        Cursor cur{0, 0}, pcur{0, 0};
        long long pads_done = 0;
        auto zero_fill_next = [&]() {
            int b, t;
            if (!cursor_seek_padded(pcur, blockIdx.x + pads_done * G, p.lengths, p.B, p.T, b, t)) return;
            unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t);
            for (uint32_t off = 0; off < ra.row_bytes; off += kZeroBytes)
                bulk_store(drow + off, smem_u32(zero_buf), min((uint32_t)kZeroBytes, ra.row_bytes - off));
            bulk_commit();
        };
        int slot = 0;
        uint32_t phase = 0;
        const int loads_per_row = (kLoss && !ra.resident) ? 2 * chunks : chunks;
        long long i = 0;
        for (long long k = blockIdx.x; k < N && !aborted; k += G, ++i) {
            int b, t;
            if (!cursor_seek_valid(cur, k, p.lengths, p.B, p.T, b, t)) break;
            const unsigned char* row = (const unsigned char*)(p.logits + (long long)b * p.stride_b + (long long)t * p.stride_t);
            for (int j = 0; j < loads_per_row; ++j) {
                const int c = j >= chunks ? j - chunks : j;
                mbar_wait(empty_addr + 8u * slot, phase ^ 1u, p.status, aborted);
                if (aborted) break;
                const uint32_t off = (uint32_t)c * kChunk;
                const uint32_t bytes = min(kChunk, ra.row_bytes - off);
                mbar_arrive_expect_tx(full_addr + 8u * slot, bytes);
                bulk_load(slots_addr + (uint32_t)slot * kChunk, row + off, bytes, full_addr + 8u * slot);
                if (++slot == S) { slot = 0; phase ^= 1u; }
            }
            if (kLoss) {
                const long long target = ((i + 1) * pads_mine) / rows_mine;
                while (pads_done < target) { zero_fill_next(); ++pads_done; }
            }
        }
        if (kLoss) {
            while (pads_done < pads_mine) { zero_fill_next(); ++pads_done; }
            bulk_wait_all();
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    if (!kLoss) {
        // log-prob 0 at padded tokens
        const long long total = (long long)p.B * p.T;
        for (long long i = (long long)blockIdx.x * kConsumerThreads + tid; i < total; i += G * kConsumerThreads) {
            int b = (int)(i / p.T), t = (int)(i % p.T);
            if (t >= clamp_len(__ldg(p.lengths + b), p.T)) p.out_lp[i] = 0.f;
        }
    }
    const float scale_over_N = N > 0 ? p.grad_scale / (float)N : 0.f;
    const uint32_t nvec = ra.row_bytes / 16u;

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
            if (kLoss) {
                const long long f = (long long)nb * p.T + nt;
                n_lp_old = __ldg(p.lp_old + f);
                n_adv = __ldg(p.adv + f);
            }
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

        const int slot0 = slot;
        const uint32_t phase0 = phase;

        // ---- pass 1: partition sum
        Acc a = acc_empty();
        for (int c = 0; c < chunks; ++c) {
            mbar_wait(full_addr + 8u * slot, phase, p.status, aborted);
            const uint4* src = (const uint4*)(smem + (size_t)slot * kChunk);
            const uint32_t v0 = (uint32_t)c * (kConsumerThreads * U) + tid;
            uint4 q[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (v0 + u * kConsumerThreads < nvec) q[u] = src[u * kConsumerThreads + tid];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = v0 + u * kConsumerThreads;
                if (v < nvec) {
                    if (v == yvec) s_zy[par] = acc_add_vec_label(a, q[u], yj);
                    else acc_add_vec(a, q[u]);
                }
            }
            if (!(kLoss && ra.resident)) {
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_addr + 8u * slot);
            }
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
        a = acc_warp_reduce(a);
        if (lane == 0) s_part[par][warp] = a;
        consumer_barrier();
        Acc tot = s_part[par][0];
#pragma unroll
        for (int w = 1; w < kConsumerWarps; ++w) tot = acc_merge(tot, s_part[par][w]);
        const RowResult r = row_finish(tot, s_zy[par]);

        // scalars of the next row, in flight while this row is finished
        fetch_row(k + G);

        if (!kLoss) {
            if (tid == 0) p.out_lp[flat] = bad_id ? 0.f : r.lp;
            continue;
        }

        float loss = 0.f, g = 0.f;
        if (!bad_id) ppo_token(r.lp, lp_old, adv, p.clip_eps, scale_over_N, loss, g);
        if (tid == 0) {
            p.row_loss[flat] = loss;
            if (p.out_lp_new) p.out_lp_new[flat] = bad_id ? 0.f : r.lp;
        }

        // ---- pass 2: dlogits
        if (ra.resident) { slot = slot0; phase = phase0; }
        unsigned char* drow = (unsigned char*)(p.dlogits + (long long)b * p.dl_stride_b + (long long)t * p.dl_stride_t);
        const float c2 = log2f(fabsf(g)) - r.lse2;
        const uint32_t sign2 = g > 0.f ? 0x80008000u : 0u;
        const float dy = g * r.one_m_py;
        for (int c = 0; c < chunks; ++c) {
            if (!ra.resident) mbar_wait(full_addr + 8u * slot, phase, p.status, aborted);
            const uint4* src = (const uint4*)(smem + (size_t)slot * kChunk);
            const uint32_t v0 = (uint32_t)c * (kConsumerThreads * U) + tid;
            if (g == 0.f) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t v = v0 + u * kConsumerThreads;
                    if (v < nvec) store_v4(drow + (size_t)v * 16, make_uint4(0, 0, 0, 0));
                }
            } else {
                uint4 q[U];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (v0 + u * kConsumerThreads < nvec) q[u] = src[u * kConsumerThreads + tid];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t v = v0 + u * kConsumerThreads;
                    if (v < nvec) {
                        uint4 o = grad_vec(q[u], c2, sign2);
                        if (v == yvec) patch_label(o, yj, dy);
                        store_v4(drow + (size_t)v * 16, o);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_addr + 8u * slot);
            if (++slot == S) { slot = 0; phase ^= 1u; }
        }
    }
}

// ---------------------------------------------------------------- host-side plan
struct RingPlan {
    int U = 0;                 // 16-byte vectors per consumer thread per chunk (1 or 2); 0 = not applicable
    int n_slots = 0;
    int chunks_per_row = 0;
    int resident = 0;
    int blocks_per_sm = 0;
    size_t smem_bytes = 0;
};

inline size_t ring_smem_bytes(int U, int n_slots, bool loss)
{
    return (size_t)n_slots * (kConsumerThreads * 16 * U) + (size_t)n_slots * 16 + (loss ? kZeroBytes : 0);
}

// Chooses chunk size, ring depth and blocks per SM for rows of `row_bytes`.
// sm_smem: shared memory per SM; block_smem_max: opt-in maximum per block.  The system reserves
// 1 KB per resident block.
inline RingPlan plan_ring(unsigned row_bytes, bool loss, int sm_smem, int block_smem_max)
{
    constexpr size_t kStatic = 1024;                   // static shared memory of the kernel, rounded up
    constexpr size_t kReserved = 1024;
    constexpr int kMaxBlocksByThreads = 2048 / kRingThreads;      // 7
    RingPlan best;
    if (loss) {
        // resident if a whole row fits: as many blocks per SM as can hold a row each; among chunk
        // sizes that reach that count take the largest; the ring then grows into what is left.
        // 8 KB chunks unless the row is short or 4 KB chunks let one more block fit per SM
        const int order[2] = {row_bytes >= 16384 ? 2 : 1, row_bytes >= 16384 ? 1 : 2};
        for (int U : order) {
            const size_t chunk = (size_t)kConsumerThreads * 16 * U;
            const int chunks = (int)((row_bytes + chunk - 1) / chunk);
            const size_t need = ring_smem_bytes(U, chunks, true) + kStatic;
            if (need > (size_t)block_smem_max) continue;
            int k = (int)std::min<size_t>(kMaxBlocksByThreads, (size_t)sm_smem / (need + kReserved));
            if (k < 1) continue;
            if (k <= best.blocks_per_sm) continue;
            const size_t per_block = std::min<size_t>((size_t)sm_smem / k - kReserved, (size_t)block_smem_max) - kStatic;
            int S = chunks;
            while (ring_smem_bytes(U, S + 1, true) <= per_block) ++S;
            best = RingPlan{U, S, chunks, 1, k, ring_smem_bytes(U, S, true)};
        }
        if (best.U) return best;
    }
    // streaming: 4 blocks per SM with about 48 KB in flight each
    const int U = row_bytes > 4096 ? 2 : 1;
    const size_t chunk = (size_t)kConsumerThreads * 16 * U;
    const int chunks = (int)((row_bytes + chunk - 1) / chunk);
    const int S = (int)((48 * 1024) / chunk);
    return RingPlan{U, S, chunks, 0, 4, ring_smem_bytes(U, S, loss)};
}

}  // namespace rlhf
