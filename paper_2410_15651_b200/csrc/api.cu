// C ABI of the token-level PPO library: argument checks and kernel launches.
// Declarations and the meaning of every argument are in include/rlhf_ppo.h.
#include "../../include/rlhf_ppo.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "kernels_generic.cuh"
#include "kernels_ring.cuh"
#include "kernels_creg.cuh"
#include "kernels_cring.cuh"
#include "kernels_warp.cuh"
#include "kernels_small.cuh"

namespace {

using namespace rlhf;

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* what)
{
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", what, cudaGetErrorString(e));
    return RLHF_ERR_CUDA;
}

#define RLHF_CUDA(call)                                   \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

// Workspace layout (bytes): [0,4) status flags, [4,8) reduction ticket, [8,16) mean and 1/std of the
// advantage whitening, [16,20) row counter of the loss kernel that deals its rows dynamically, [256, kRowLossOffset) block
// partial sums of the two losses (2 doubles per block of the kernel that reduces them),
// [kRowLossOffset, +4*B*T) per-token policy loss terms (kernels without the fused finalisation).
constexpr size_t kPartialsOffset = 256;
constexpr size_t kRowLossOffset = 24576;
constexpr int kMaxFusedBlocks = (int)((kRowLossOffset - kPartialsOffset) / 16);   // block partials that fit the header

constexpr long long kMaxTokens = 1ll << 29;

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_shape(int B, int T, int V)
{
    if (B <= 0 || T <= 0 || V <= 0) return RLHF_ERR_SHAPE;
    // the log-prob kernel walks up to 2*B*T rows (two tensors in one launch) plus one grid stride with 32-bit
    // indices, so B*T stays at or below 2^29
    if ((long long)B * (long long)T > kMaxTokens) return RLHF_ERR_SHAPE;
    return RLHF_OK;
}

// Bytes of the workspace that rlhf_ppo_loss_fwd_bwd touches: header + per-token policy loss terms.
size_t loss_workspace_bytes(int B, int T) { return kRowLossOffset + 4 * (size_t)B * (size_t)T; }

int check_workspace(const void* ws, size_t bytes, size_t need)
{
    if (!ws) return RLHF_ERR_NULL;
    if (!aligned(ws, 256)) return RLHF_ERR_ALIGN;
    if (bytes < need) return RLHF_ERR_WORKSPACE;
    return RLHF_OK;
}

struct DeviceInfo {
    int sm_count = 0;
    int max_smem_optin = 0;     // per block
    int smem_per_sm = 0;
};

// Queried per call: the library keeps no state, and the two attributes are cheap to read.
int device_info(DeviceInfo& d)
{
    int dev = 0;
    RLHF_CUDA(cudaGetDevice(&dev));
    RLHF_CUDA(cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev));
    RLHF_CUDA(cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    RLHF_CUDA(cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev));
    return RLHF_OK;
}

// Rows can take the 16-byte path if every row starts on a 16-byte boundary and is a whole number
// of 16-byte vectors long.
bool rows_16B(const void* base, long long stride_b, long long stride_t, int V)
{
    return aligned(base, 16) && (stride_b % 8) == 0 && (stride_t % 8) == 0 && (V % 8) == 0;
}

// Launches `kernel` with programmatic stream serialisation allowed (see pdl_wait_prior_grid): the launch
// itself and the kernel's set-up overlap the tail of the kernel before it in the stream.
// `cluster` > 1 launches the grid as thread-block clusters of that many blocks.
void fill_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute (&attr)[2], int grid, int block, size_t smem,
                        int cluster, cudaStream_t s)
{
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cluster > 1) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
}

template <typename... Params, typename... Args>
cudaError_t launch_kernel_cluster(void (*kernel)(Params...), int grid, int block, size_t smem, int cluster,
                                  cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    fill_launch_config(cfg, attr, grid, block, smem, cluster, s);
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <typename... Params, typename... Args>
cudaError_t launch_kernel(void (*kernel)(Params...), int grid, int block, size_t smem, cudaStream_t s, Args&&... args)
{
    return launch_kernel_cluster(kernel, grid, block, smem, 1, s, static_cast<Args&&>(args)...);
}

template <int NW, int U>
int launch_ring_as(const RingArgs& ra, const RingPlan& pl, int grid, cudaStream_t s)
{
    RLHF_CUDA(cudaFuncSetAttribute(row_ring_kernel<NW, U>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)pl.smem_bytes));
    RLHF_CUDA(launch_kernel(row_ring_kernel<NW, U>, grid, NW * 32 + 32, pl.smem_bytes, s, ra));
    return RLHF_OK;
}

constexpr int kLogprobWarps = 24;

template <bool kDual, bool kAny, bool kF16, bool kEnt>
int launch_warp_logprob_as(const WarpArgs& wa_in, const DeviceInfo& dev, cudaStream_t s)
{
    WarpArgs wa = wa_in;
    wa.row_bytes = 2u * (unsigned)wa.row.V;
    const size_t smem = warp_kernel_smem_bytes(kLogprobWarps);
    const long long rows = (long long)wa.row.B * wa.row.T;
    const int grid = (int)std::min<long long>(rows, dev.sm_count);
    RLHF_CUDA(cudaFuncSetAttribute(logprob_warp_kernel<kLogprobWarps, kDual, kAny, kF16, kEnt>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    RLHF_CUDA(launch_kernel(logprob_warp_kernel<kLogprobWarps, kDual, kAny, kF16, kEnt>, grid, kLogprobWarps * 32, smem, s, wa));
    return RLHF_OK;
}

// f16: the logits are IEEE binary16; the entropy variant is taken when wa.out_entropy is set.
template <bool kDual, bool kAny>
int launch_warp_logprob(const WarpArgs& wa, bool f16, const DeviceInfo& dev, cudaStream_t s)
{
    const bool ent = wa.out_entropy != nullptr;
    if (f16) return ent ? launch_warp_logprob_as<kDual, kAny, true, true>(wa, dev, s)
                        : launch_warp_logprob_as<kDual, kAny, true, false>(wa, dev, s);
    return ent ? launch_warp_logprob_as<kDual, kAny, false, true>(wa, dev, s)
               : launch_warp_logprob_as<kDual, kAny, false, false>(wa, dev, s);
}

// Loss kernel that keeps a row's exponentials on chip (kernels_creg.cuh): in registers if a consumer thread has at
// most kRegVecsOnly vectors of a row, else in registers for its first kRegVecsTmem vectors and in tensor memory for
// up to kTmemVecs more.  A block holds two buffers of its share of
// a row; rows that do not fit twice are shared by a cluster of up to 4 blocks.
#ifndef RLHF_CREG_WARPS
#define RLHF_CREG_WARPS 16
#endif
constexpr int kCregWarps = RLHF_CREG_WARPS;

struct CregPlan {
    int cluster = 0;            // blocks per cluster, 1..4; 0 = the kernel does not apply
    unsigned slice_vecs = 0;
    unsigned tmem_cols = 0;
    int n_buf = 0;              // slice buffers per block
    size_t smem_bytes = 0;
};

CregPlan plan_creg(unsigned row_bytes, const DeviceInfo& dev)
{
    CregPlan pl;
    if (row_bytes < 16384 || row_bytes % 16 != 0) return pl;
    const unsigned row_vecs = row_bytes / 16;
    const unsigned cap = (unsigned)kCregWarps * 32 * (kRegVecsTmem + kTmemVecs);
    for (int c = 1; c <= 4; ++c) {
        const unsigned sv = (row_vecs + c - 1) / c;
        if (sv > cap) continue;
        int nb = kCregMaxBufs;
        while (nb >= 2 && creg_smem_bytes(sv, kCregWarps, nb) + 2048 > (size_t)dev.max_smem_optin) --nb;
        if (nb < 2) continue;
        pl.cluster = c;
        pl.slice_vecs = sv;
        pl.tmem_cols = creg_tmem_cols(sv, kCregWarps);
        pl.n_buf = nb;
        pl.smem_bytes = creg_smem_bytes(sv, kCregWarps, nb);
        return pl;
    }
    return pl;
}

// Clusters of the kernel that the device holds at once (one block per SM); looked up once per device and
// cluster size.  It only sizes the persistent grid: a larger grid would still be correct.
template <int NW, int C, bool kTmem, bool kF16, bool kAny>
int creg_resident_clusters(const CregPlan& pl, const DeviceInfo& dev, int& out)
{
    if (C == 1) { out = dev.sm_count; return RLHF_OK; }
    static std::mutex mu;
    static int cached[64] = {};
    int d = 0;
    RLHF_CUDA(cudaGetDevice(&d));
    std::lock_guard<std::mutex> lock(mu);
    if (d < 0 || d >= 64 || cached[d] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute attr[2];
        fill_launch_config(cfg, attr, dev.sm_count / C * C, NW * 32 + 32, pl.smem_bytes, C, nullptr);
        RLHF_CUDA(cudaOccupancyMaxActiveClusters(&n, loss_creg_kernel<NW, C, kTmem, kF16, kAny>, &cfg));
        if (n < 1) n = 1;
        if (d < 0 || d >= 64) { out = n; return RLHF_OK; }
        cached[d] = n;
    }
    out = cached[d];
    return RLHF_OK;
}

template <int NW, int C, bool kTmem, bool kF16, bool kAny = false>
int launch_creg(const RowArgs& a, const CregPlan& pl, const DeviceInfo& dev, cudaStream_t s)
{
    CregArgs ca{};
    ca.row = a;
    ca.row_bytes = 2u * (unsigned)a.V;
    ca.slice_vecs = pl.slice_vecs;
    ca.buf_stride = (unsigned)creg_buf_stride(pl.slice_vecs, NW);
    ca.tmem_cols = pl.tmem_cols;
    ca.n_buf = pl.n_buf;
    ca.row_counter = (unsigned*)((char*)a.status + 16);
    RLHF_CUDA(cudaFuncSetAttribute(loss_creg_kernel<NW, C, kTmem, kF16, kAny>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)pl.smem_bytes));
    int clusters = 0;
    if (int e = creg_resident_clusters<NW, C, kTmem, kF16, kAny>(pl, dev, clusters)) return e;
    const long long rows = (long long)a.B * a.T;
    const int grid = (int)std::min<long long>(rows, clusters) * C;
    RLHF_CUDA(launch_kernel_cluster(loss_creg_kernel<NW, C, kTmem, kF16, kAny>, grid, NW * 32 + 32, pl.smem_bytes, C, s, ca));
    return RLHF_OK;
}

template <int NW, bool kTmem, bool kF16>
int launch_creg_cluster(const RowArgs& a, const CregPlan& pl, const DeviceInfo& dev, cudaStream_t s)
{
    switch (pl.cluster) {
        case 1: return launch_creg<NW, 1, kTmem, kF16>(a, pl, dev, s);
        case 2: return launch_creg<NW, 2, kTmem, kF16>(a, pl, dev, s);
        case 3: return launch_creg<NW, 3, kTmem, kF16>(a, pl, dev, s);
        default: return launch_creg<NW, 4, kTmem, kF16>(a, pl, dev, s);
    }
}

// The chunk-ring variant of the on-chip-exponentials kernel: a slice may be as long as registers and tensor memory hold
// exponentials for (8 chunks of 16 KB), so some rows need fewer blocks per cluster than with whole-slice buffers.
struct CringPlan {
    int cluster = 0;
    unsigned slice_vecs = 0, tmem_cols = 0;
    int n_slots = 0, chunks = 0;
    size_t smem_bytes = 0;
};

CringPlan plan_cring(unsigned row_bytes, const DeviceInfo& dev)
{
    CringPlan pl;
    if (row_bytes % 16 != 0) return pl;
    const unsigned row_vecs = row_bytes / 16;
    const size_t chunk = cring_chunk_bytes(kCregWarps);
    int R = kCringMaxSlots;
    while (R > 0 && cring_smem_bytes(kCregWarps, R) + 3072 > (size_t)dev.max_smem_optin) --R;
    for (int c = 1; c <= 4; ++c) {
        const unsigned sv = (row_vecs + c - 1) / c;
        const int C = (int)(((size_t)sv * 16 + chunk - 1) / chunk);
        // a slice's chunks stay in the ring from pass 1 to pass 2, and the kernel is fast only while at least five
        // more slots prefetch the next slice
        if (C < 3 || C > R - 5 || kCringU * C - kRegVecsTmem > kTmemVecs) continue;
        if ((size_t)row_vecs <= (size_t)(c - 1) * sv) continue;        // every block of the cluster has a share
        unsigned cols = 32;
        while (cols < (unsigned)(kCringU * C - kRegVecsTmem) * 8u * ((kCregWarps + 3) / 4)) cols *= 2;
        pl.cluster = c;
        pl.slice_vecs = sv;
        pl.tmem_cols = cols;
        pl.n_slots = R;
        pl.chunks = C;
        pl.smem_bytes = cring_smem_bytes(kCregWarps, R);
        return pl;
    }
    return pl;
}

template <int C, bool kF16>
int launch_cring(const RowArgs& a, const CringPlan& pl, const DeviceInfo& dev, cudaStream_t s)
{
    constexpr int NW = kCregWarps;
    CringArgs ca{};
    ca.row = a;
    ca.row_bytes = 2u * (unsigned)a.V;
    ca.slice_vecs = pl.slice_vecs;
    ca.tmem_cols = pl.tmem_cols;
    ca.n_slots = pl.n_slots;
    ca.chunks = pl.chunks;
    ca.row_counter = (unsigned*)((char*)a.status + 16);
    RLHF_CUDA(cudaFuncSetAttribute(loss_cring_kernel<NW, C, kF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)pl.smem_bytes));
    // clusters that the device holds at once (one block per SM); looked up once per device
    static std::mutex mu;
    static int cached[64] = {};
    int d = 0, clusters = 0;
    RLHF_CUDA(cudaGetDevice(&d));
    if (C == 1) {
        clusters = dev.sm_count;
    } else {
        std::lock_guard<std::mutex> lock(mu);
        if (d < 0 || d >= 64 || cached[d] == 0) {
            int n = 0;
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[2];
            fill_launch_config(cfg, attr, dev.sm_count / C * C, NW * 32 + 32, pl.smem_bytes, C, nullptr);
            RLHF_CUDA(cudaOccupancyMaxActiveClusters(&n, loss_cring_kernel<NW, C, kF16>, &cfg));
            if (n < 1) n = 1;
            if (d >= 0 && d < 64) cached[d] = n;
            clusters = n;
        } else {
            clusters = cached[d];
        }
    }
    const long long rows = (long long)a.B * a.T;
    const int grid = (int)std::min<long long>(rows, clusters) * C;
    RLHF_CUDA(launch_kernel_cluster(loss_cring_kernel<NW, C, kF16>, grid, NW * 32 + 32, pl.smem_bytes, C, s, ca));
    return RLHF_OK;
}

template <bool kF16>
int launch_cring_cluster(const RowArgs& a, const CringPlan& pl, const DeviceInfo& dev, cudaStream_t s)
{
    switch (pl.cluster) {
        case 1: return launch_cring<1, kF16>(a, pl, dev, s);
        case 2: return launch_cring<2, kF16>(a, pl, dev, s);
        case 3: return launch_cring<3, kF16>(a, pl, dev, s);
        default: return launch_cring<4, kF16>(a, pl, dev, s);
    }
}

// The loss row kernel for 16-byte aligned rows: exponentials kept on chip where the row (or its share in a
// cluster) fits, else the chunk ring.
// Rows off 16-byte boundaries: the kernel loads the aligned span around a row, at most 14 bytes before it and 14 after;
// only single blocks take such rows.
CregPlan plan_creg_any(int V, const DeviceInfo& dev)
{
    const unsigned span = (14u + 2u * (unsigned)V + 15u) & ~15u;
    CregPlan pl = plan_creg(span, dev);
    if (pl.cluster != 1) pl.cluster = 0;
    return pl;
}

template <bool kF16>
int launch_creg_any(const RowArgs& a, const CregPlan& pl, const DeviceInfo& dev, cudaStream_t s)
{
    return pl.tmem_cols != 0 ? launch_creg<kCregWarps, 1, true, kF16, true>(a, pl, dev, s)
                             : launch_creg<kCregWarps, 1, false, kF16, true>(a, pl, dev, s);
}

// Which of the two takes a row length that both can take.  Measured on V = 57344 ... 256000 (T = 512, 4 GB of logits):
// the chunk ring wins where it needs fewer blocks per row and at most two (rows of 105-128 KB in one block: 1.02 of the
// copy rate against 0.86-0.93 in a cluster of two; rows of 210-256 KB in two blocks on all SMs: 0.98 against 0.88-0.92 in
// three); in clusters of three and four it does not (0.85 against 0.89 at 320 KB), and whole-slice buffers are at their
// best with slices of 85-105 KB (0.97-1.0).  Rows beyond the largest cluster of whole-slice buffers (426-512 KB) go to
// the chunk ring in a cluster of four (0.86 against 0.65 for streaming the row twice).
inline bool use_cring(const CregPlan& cp, const CringPlan& rp)
{
    if (rp.cluster == 0) return false;
    if (cp.cluster == 0) return true;
    return rp.cluster < cp.cluster && rp.cluster <= 2;
}

// The fast loss kernels for 16-byte aligned rows of this length (binary16 rows: the on-chip-exponentials kernel
// only; the chunk ring is a bf16 kernel).
bool fast_loss_rows_apply(int V, bool f16, const DeviceInfo& dev)
{
    return !f16 || plan_cring(2u * (unsigned)V, dev).cluster > 0 || plan_creg(2u * (unsigned)V, dev).cluster > 0;
}

int launch_loss_rows(const RowArgs& a, bool f16, const DeviceInfo& dev, cudaStream_t s)
{
    const unsigned row_bytes = 2u * (unsigned)a.V;
    const CregPlan cp = plan_creg(row_bytes, dev);
    const CringPlan rp = plan_cring(row_bytes, dev);
    if (use_cring(cp, rp)) return f16 ? launch_cring_cluster<true>(a, rp, dev, s) : launch_cring_cluster<false>(a, rp, dev, s);
    if (cp.cluster > 0) {
        if (f16)
            return cp.tmem_cols != 0 ? launch_creg_cluster<kCregWarps, true, true>(a, cp, dev, s)
                                     : launch_creg_cluster<kCregWarps, false, true>(a, cp, dev, s);
        return cp.tmem_cols != 0 ? launch_creg_cluster<kCregWarps, true, false>(a, cp, dev, s)
                                 : launch_creg_cluster<kCregWarps, false, false>(a, cp, dev, s);
    }
    const RingPlan pl = plan_ring(row_bytes, dev.smem_per_sm, dev.max_smem_optin);
    RingArgs ra{};
    ra.row = a;
    ra.n_slots = pl.n_slots;
    ra.chunks_per_row = pl.chunks_per_row;
    ra.resident = pl.resident;
    ra.row_bytes = row_bytes;
    const long long rows = (long long)a.B * a.T;
    const int grid = (int)std::min<long long>(rows, (long long)dev.sm_count * pl.blocks_per_sm);
    if (pl.NW == 16) return launch_ring_as<16, 4>(ra, pl, grid, s);
    if (pl.U == 1) return launch_ring_as<8, 1>(ra, pl, grid, s);
    return launch_ring_as<8, 2>(ra, pl, grid, s);
}

// The row kernels run with the largest shared-memory carve-out.  A kernel that prefers another
// split makes the SMs switch configuration before and after it, which costs microseconds per
// launch; so the small kernels between them ask for the same carve-out.
template <typename K>
int keep_max_carveout(K kernel)
{
    RLHF_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    return RLHF_OK;
}

// Host-side checks of the loss call's arguments, the workspace apart (shared by the two loss entry points).
int check_loss_args(const void* logits, long long stride_b, long long stride_t, const long long* ids,
                    long long ids_stride_b, const int* lengths, const float* lp_old, const float* adv,
                    const float* values_new, const float* values_old, const float* returns, int B, int T, int V,
                    float clip_eps, float value_clip, float grad_scale, const float* out_loss_pg,
                    const float* out_loss_vf, const void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                    const float* out_dvalues, const float* out_lp_new)
{
    if (!logits || !ids || !lengths || !lp_old || !adv || !values_new || !values_old || !returns ||
        !out_loss_pg || !out_loss_vf || !out_dlogits || !out_dvalues)
        return RLHF_ERR_NULL;
    if (int e = check_shape(B, T, V)) return e;
    if (stride_b < 0 || stride_t < 0 || ids_stride_b < 0 || dl_stride_b < 0 || dl_stride_t < 0)
        return RLHF_ERR_STRIDE;
    if (T > 1 && (stride_t < V || dl_stride_t < V)) return RLHF_ERR_STRIDE;
    if (B > 1 && dl_stride_b < (long long)(T - 1) * dl_stride_t + V) return RLHF_ERR_STRIDE;
    if (out_dlogits == logits && (dl_stride_b != stride_b || dl_stride_t != stride_t)) return RLHF_ERR_STRIDE;
    if (!(clip_eps > 0.f && clip_eps < 1.f) || !std::isfinite(value_clip) || value_clip < 0.f ||
        !std::isfinite(grad_scale))
        return RLHF_ERR_SCALAR;
    if (!aligned(logits, 2) || !aligned(out_dlogits, 2) || !aligned(ids, 8) || !aligned(lengths, 4) ||
        !aligned(lp_old, 4) || !aligned(adv, 4) || !aligned(values_new, 4) || !aligned(values_old, 4) ||
        !aligned(returns, 4) || !aligned(out_loss_pg, 4) || !aligned(out_loss_vf, 4) ||
        !aligned(out_dvalues, 4) || (out_lp_new && !aligned(out_lp_new, 4)))
        return RLHF_ERR_ALIGN;
    return RLHF_OK;
}

int launch_check(const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, what);
    return RLHF_OK;
}

}  // namespace

extern "C" {

const char* rlhf_status_string(int status)
{
    switch (status) {
        case RLHF_OK: return "RLHF_OK";
        case RLHF_ERR_NULL: return "RLHF_ERR_NULL";
        case RLHF_ERR_SHAPE: return "RLHF_ERR_SHAPE";
        case RLHF_ERR_ALIGN: return "RLHF_ERR_ALIGN";
        case RLHF_ERR_STRIDE: return "RLHF_ERR_STRIDE";
        case RLHF_ERR_WORKSPACE: return "RLHF_ERR_WORKSPACE";
        case RLHF_ERR_SCALAR: return "RLHF_ERR_SCALAR";
        case RLHF_ERR_CUDA: return "RLHF_ERR_CUDA";
        case RLHF_ERR_TOO_LARGE: return "RLHF_ERR_TOO_LARGE";
        default: break;
    }
    if (status > 0 && (status & ~(RLHF_ERR_ID_RANGE | RLHF_ERR_LENGTH_RANGE | RLHF_ERR_TIMEOUT)) == 0) {
        static const char* const names[8] = {
            "RLHF_OK",
            "RLHF_ERR_ID_RANGE",
            "RLHF_ERR_LENGTH_RANGE",
            "RLHF_ERR_ID_RANGE|RLHF_ERR_LENGTH_RANGE",
            "RLHF_ERR_TIMEOUT",
            "RLHF_ERR_ID_RANGE|RLHF_ERR_TIMEOUT",
            "RLHF_ERR_LENGTH_RANGE|RLHF_ERR_TIMEOUT",
            "RLHF_ERR_ID_RANGE|RLHF_ERR_LENGTH_RANGE|RLHF_ERR_TIMEOUT",
        };
        return names[(status >> 4) & 7];
    }
    return "RLHF_ERR_UNKNOWN";
}

const char* rlhf_last_cuda_error(void) { return g_cuda_error; }

int rlhf_pad_share(long long n_valid, long long n_padded, int n_blocks, int block, long long* start, long long* count)
{
    if (!start || !count) return RLHF_ERR_NULL;
    if (n_blocks <= 0 || block < 0 || block >= n_blocks || n_valid < 0 || n_padded < 0) return RLHF_ERR_SHAPE;
    const PadShare s = pad_share(n_valid, n_padded, n_blocks, block);
    *start = s.start;
    *count = s.count;
    return RLHF_OK;
}

size_t rlhf_workspace_bytes(int B, int T)
{
    if (B <= 0 || T <= 0) return 0;
    size_t n = loss_workspace_bytes(B, T);
    return (n + 255) & ~(size_t)255;
}

int rlhf_workspace_init(void* workspace, size_t workspace_bytes, void* stream)
{
    if (!workspace) return RLHF_ERR_NULL;
    if (!aligned(workspace, 256)) return RLHF_ERR_ALIGN;
    if (workspace_bytes < kRowLossOffset) return RLHF_ERR_WORKSPACE;
    RLHF_CUDA(cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream));
    return RLHF_OK;
}

int rlhf_poll_status(void* workspace, void* stream)
{
    if (!workspace) return RLHF_ERR_NULL;
    unsigned flags = 0;
    cudaStream_t s = (cudaStream_t)stream;
    RLHF_CUDA(cudaMemcpyAsync(&flags, workspace, sizeof flags, cudaMemcpyDeviceToHost, s));
    RLHF_CUDA(cudaStreamSynchronize(s));
    if (flags != 0) {
        RLHF_CUDA(cudaMemsetAsync(workspace, 0, sizeof flags, s));
        RLHF_CUDA(cudaStreamSynchronize(s));
    }
    return (int)flags;
}

int rlhf_selftest_bounded_wait(void* workspace, size_t workspace_bytes, unsigned long long limit_ns, void* stream)
{
    if (int e = check_workspace(workspace, workspace_bytes, kRowLossOffset)) return e;
    if (limit_ns == 0 || limit_ns > kWaitLimitNs) return RLHF_ERR_SCALAR;
    RLHF_CUDA(launch_kernel(bounded_wait_selftest_kernel, 1, 32, 0, (cudaStream_t)stream, (unsigned*)workspace, limit_ns));
    return launch_check("bounded_wait_selftest_kernel");
}

int rlhf_gather_logprobs_ex(const void* logits, int logits_dtype, long long stride_b, long long stride_t,
                            const long long* ids, long long ids_stride_b, const int* lengths,
                            int B, int T, int V, float* out_logprobs, float* out_entropy,
                            void* workspace, size_t workspace_bytes, void* stream)
{
    if (!logits || !ids || !lengths || !out_logprobs) return RLHF_ERR_NULL;
    if (logits_dtype != RLHF_BF16 && logits_dtype != RLHF_F16) return RLHF_ERR_SCALAR;
    if (int e = check_shape(B, T, V)) return e;
    if (stride_b < 0 || stride_t < 0 || ids_stride_b < 0) return RLHF_ERR_STRIDE;
    if (T > 1 && stride_t < V) return RLHF_ERR_STRIDE;
    if (!aligned(logits, 2) || !aligned(ids, 8) || !aligned(lengths, 4) || !aligned(out_logprobs, 4) ||
        (out_entropy && !aligned(out_entropy, 4)))
        return RLHF_ERR_ALIGN;
    if (out_entropy && out_entropy == out_logprobs) return RLHF_ERR_STRIDE;
    if (int e = check_workspace(workspace, workspace_bytes, rlhf_workspace_bytes(B, T))) return e;
    DeviceInfo dev;
    if (int e = device_info(dev)) return e;

    RowArgs a{};
    a.logits = (const uint16_t*)logits;
    a.stride_b = stride_b;
    a.stride_t = stride_t;
    a.ids = ids;
    a.ids_stride_b = ids_stride_b;
    a.lengths = lengths;
    a.B = B; a.T = T; a.V = V;
    a.status = (unsigned*)workspace;
    a.wait_limit_ns = kWaitLimitNs;
    a.out_lp = out_logprobs;

    WarpArgs wa{};
    wa.row = a;
    wa.out_entropy = out_entropy;
    const bool f16 = logits_dtype == RLHF_F16;
    if (rows_16B(logits, stride_b, stride_t, V)) {
        if (int e = launch_warp_logprob<false, false>(wa, f16, dev, (cudaStream_t)stream)) return e;
    } else {
        // rows that start or end off a 16-byte boundary (odd V, odd strides): same kernel, aligned spans
        if (int e = launch_warp_logprob<false, true>(wa, f16, dev, (cudaStream_t)stream)) return e;
    }
    return launch_check("logprob_warp_kernel");
}

int rlhf_gather_logprobs(const void* logits, long long stride_b, long long stride_t,
                         const long long* ids, long long ids_stride_b, const int* lengths,
                         int B, int T, int V, float* out_logprobs,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    return rlhf_gather_logprobs_ex(logits, RLHF_BF16, stride_b, stride_t, ids, ids_stride_b, lengths, B, T, V,
                                   out_logprobs, nullptr, workspace, workspace_bytes, stream);
}

int rlhf_kl_reward(const float* lp_old, const float* lp_ref, const float* score, const int* lengths,
                   int B, int T, float beta_kl, float reward_clip, float* out_rewards, void* stream)
{
    if (!lp_old || !lp_ref || !score || !lengths || !out_rewards) return RLHF_ERR_NULL;
    if (int e = check_shape(B, T, 1)) return e;
    if (!std::isfinite(beta_kl) || beta_kl < 0.f || !std::isfinite(reward_clip) || reward_clip < 0.f)
        return RLHF_ERR_SCALAR;
    if (!aligned(lp_old, 4) || !aligned(lp_ref, 4) || !aligned(score, 4) || !aligned(lengths, 4) ||
        !aligned(out_rewards, 4))
        return RLHF_ERR_ALIGN;
    long long total = (long long)B * T;
    int grid = (int)std::min<long long>((total + 255) / 256, 1184);
    if (int e = keep_max_carveout(kl_reward_kernel)) return e;
    RLHF_CUDA(launch_kernel(kl_reward_kernel, grid, 256, 0, (cudaStream_t)stream, lp_old, lp_ref, score, lengths, B, T,
                            beta_kl, reward_clip, out_rewards));
    return launch_check("kl_reward_kernel");
}

int rlhf_gae(const float* rewards, const float* values_old, const int* lengths, int B, int T,
             float gamma, float lambda, float* out_adv, float* out_returns, void* stream)
{
    if (!rewards || !values_old || !lengths || !out_adv || !out_returns) return RLHF_ERR_NULL;
    if (int e = check_shape(B, T, 1)) return e;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return RLHF_ERR_SCALAR;
    if (!aligned(rewards, 4) || !aligned(values_old, 4) || !aligned(lengths, 4) || !aligned(out_adv, 4) ||
        !aligned(out_returns, 4))
        return RLHF_ERR_ALIGN;
    if (out_adv == rewards || out_adv == values_old || out_returns == rewards ||
        out_returns == values_old || out_adv == out_returns)
        return RLHF_ERR_STRIDE;
    int grid = (B + kGaeWarpsPerBlock - 1) / kGaeWarpsPerBlock;
    if (int e = keep_max_carveout(gae_kernel)) return e;
    RLHF_CUDA(launch_kernel(gae_kernel, grid, kGaeWarpsPerBlock * 32, 0, (cudaStream_t)stream, rewards, values_old,
                            lengths, B, T, gamma, lambda, out_adv, out_returns));
    return launch_check("gae_kernel");
}

int rlhf_whiten_advantages(const float* adv, const int* lengths, int B, int T, float eps, float* out_adv,
                           void* workspace, size_t workspace_bytes, void* stream)
{
    if (!adv || !lengths || !out_adv) return RLHF_ERR_NULL;
    if (int e = check_shape(B, T, 1)) return e;
    if (!std::isfinite(eps) || eps < 0.f) return RLHF_ERR_SCALAR;
    if (!aligned(adv, 4) || !aligned(lengths, 4) || !aligned(out_adv, 4)) return RLHF_ERR_ALIGN;
    if (int e = check_workspace(workspace, workspace_bytes, rlhf_workspace_bytes(B, T))) return e;
    char* ws = (char*)workspace;
    WhitenArgs w{};
    w.adv = adv;
    w.lengths = lengths;
    w.B = B; w.T = T;
    w.eps = eps;
    w.out = out_adv;
    w.ticket = (unsigned*)(ws + 4);
    w.partials = (double*)(ws + kPartialsOffset);
    w.mean_rstd = (float*)(ws + 8);
    const long long total = (long long)B * T;
    const int grid = (int)std::min<long long>((total + 4095) / 4096, kWhitenMaxBlocks);
    cudaStream_t s = (cudaStream_t)stream;
    if (int e = keep_max_carveout(whiten_stats_kernel)) return e;
    RLHF_CUDA(launch_kernel(whiten_stats_kernel, grid, kWhitenThreads, 0, s, w));
    if (int e = launch_check("whiten_stats_kernel")) return e;
    if (int e = keep_max_carveout(whiten_apply_kernel)) return e;
    const int agrid = (int)std::min<long long>((total + 255) / 256, 1184);
    RLHF_CUDA(launch_kernel(whiten_apply_kernel, agrid, 256, 0, s, w));
    return launch_check("whiten_apply_kernel");
}

int rlhf_ppo_stats(const float* lp_new, const float* lp_old, const float* adv, const int* lengths, int B, int T,
                   float clip_eps, float* out_stats, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!lp_new || !lp_old || !adv || !lengths || !out_stats) return RLHF_ERR_NULL;
    if (int e = check_shape(B, T, 1)) return e;
    if (!(clip_eps > 0.f && clip_eps < 1.f)) return RLHF_ERR_SCALAR;
    if (!aligned(lp_new, 4) || !aligned(lp_old, 4) || !aligned(adv, 4) || !aligned(lengths, 4) || !aligned(out_stats, 4))
        return RLHF_ERR_ALIGN;
    if (int e = check_workspace(workspace, workspace_bytes, rlhf_workspace_bytes(B, T))) return e;
    char* ws = (char*)workspace;
    StatsArgs a{};
    a.lp_new = lp_new;
    a.lp_old = lp_old;
    a.adv = adv;
    a.lengths = lengths;
    a.B = B; a.T = T;
    a.clip_eps = clip_eps;
    a.out = out_stats;
    a.ticket = (unsigned*)(ws + 4);
    a.partials = (double*)(ws + kPartialsOffset);
    const long long total = (long long)B * T;
    const int grid = (int)std::min<long long>((total + 4095) / 4096, kWhitenMaxBlocks);
    if (int e = keep_max_carveout(ppo_stats_kernel)) return e;
    RLHF_CUDA(launch_kernel(ppo_stats_kernel, grid, kWhitenThreads, 0, (cudaStream_t)stream, a));
    return launch_check("ppo_stats_kernel");
}

int rlhf_experience_ex(const void* actor_logits, long long actor_stride_b, long long actor_stride_t,
                       const void* ref_logits, long long ref_stride_b, long long ref_stride_t, int logits_dtype,
                       const long long* ids, long long ids_stride_b, const int* lengths,
                       const float* score, const float* values_old, const float* lp_old,
                       int B, int T, int V, float beta_kl, float reward_clip, float gamma, float lambda,
                       float* out_lp_actor, float* out_lp_ref, float* out_rewards, float* out_adv,
                       float* out_returns, float* out_entropy, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!actor_logits || !ref_logits || !ids || !lengths || !score || !values_old || !out_lp_actor ||
        !out_lp_ref || !out_rewards || !out_adv || !out_returns)
        return RLHF_ERR_NULL;
    if (logits_dtype != RLHF_BF16 && logits_dtype != RLHF_F16) return RLHF_ERR_SCALAR;
    if (int e = check_shape(B, T, V)) return e;
    if (actor_stride_b < 0 || actor_stride_t < 0 || ref_stride_b < 0 || ref_stride_t < 0 || ids_stride_b < 0)
        return RLHF_ERR_STRIDE;
    if (T > 1 && (actor_stride_t < V || ref_stride_t < V)) return RLHF_ERR_STRIDE;
    if (!std::isfinite(beta_kl) || beta_kl < 0.f || !std::isfinite(reward_clip) || reward_clip < 0.f ||
        !(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f))
        return RLHF_ERR_SCALAR;
    if (!aligned(actor_logits, 2) || !aligned(ref_logits, 2) || !aligned(ids, 8) || !aligned(lengths, 4) ||
        !aligned(score, 4) || !aligned(values_old, 4) || (lp_old && !aligned(lp_old, 4)) ||
        !aligned(out_lp_actor, 4) || !aligned(out_lp_ref, 4) || !aligned(out_rewards, 4) ||
        !aligned(out_adv, 4) || !aligned(out_returns, 4) || (out_entropy && !aligned(out_entropy, 4)))
        return RLHF_ERR_ALIGN;
    {
        const float* outs[6] = {out_lp_actor, out_lp_ref, out_rewards, out_adv, out_returns, out_entropy};
        for (int i = 0; i < 6; ++i) {
            if (!outs[i]) continue;
            if (outs[i] == values_old || outs[i] == lp_old) return RLHF_ERR_STRIDE;
            for (int j = i + 1; j < 6; ++j)
                if (outs[i] == outs[j]) return RLHF_ERR_STRIDE;
        }
    }
    if (int e = check_workspace(workspace, workspace_bytes, rlhf_workspace_bytes(B, T))) return e;

    const bool all_16B = rows_16B(actor_logits, actor_stride_b, actor_stride_t, V) &&
                         rows_16B(ref_logits, ref_stride_b, ref_stride_t, V);
    DeviceInfo dev;
    if (int e = device_info(dev)) return e;
    WarpArgs wa{};
    wa.row.logits = (const uint16_t*)actor_logits;
    wa.row.stride_b = actor_stride_b;
    wa.row.stride_t = actor_stride_t;
    wa.row.ids = ids;
    wa.row.ids_stride_b = ids_stride_b;
    wa.row.lengths = lengths;
    wa.row.B = B; wa.row.T = T; wa.row.V = V;
    wa.row.status = (unsigned*)workspace;
    wa.row.wait_limit_ns = kWaitLimitNs;
    wa.row.out_lp = out_lp_actor;
    wa.logits2 = (const uint16_t*)ref_logits;
    wa.stride2_b = ref_stride_b;
    wa.stride2_t = ref_stride_t;
    wa.out_lp2 = out_lp_ref;
    wa.out_entropy = out_entropy;
    const bool f16 = logits_dtype == RLHF_F16;
    cudaStream_t s = (cudaStream_t)stream;
    if (all_16B) {
        if (int e = launch_warp_logprob<true, false>(wa, f16, dev, s)) return e;
    } else {
        if (int e = launch_warp_logprob<true, true>(wa, f16, dev, s)) return e;
    }
    if (int e = launch_check("logprob_warp_kernel<dual>")) return e;
    if (int e = keep_max_carveout(reward_gae_kernel)) return e;
    const int grid = (B + kGaeWarpsPerBlock - 1) / kGaeWarpsPerBlock;
    RLHF_CUDA(launch_kernel(reward_gae_kernel, grid, kGaeWarpsPerBlock * 32, 0, s, lp_old ? lp_old : out_lp_actor,
                            out_lp_ref, score, values_old, lengths, B, T, beta_kl, reward_clip, gamma, lambda,
                            out_rewards, out_adv, out_returns));
    return launch_check("reward_gae_kernel");
}

int rlhf_experience(const void* actor_logits, long long actor_stride_b, long long actor_stride_t,
                    const void* ref_logits, long long ref_stride_b, long long ref_stride_t,
                    const long long* ids, long long ids_stride_b, const int* lengths,
                    const float* score, const float* values_old, const float* lp_old,
                    int B, int T, int V, float beta_kl, float reward_clip, float gamma, float lambda,
                    float* out_lp_actor, float* out_lp_ref, float* out_rewards, float* out_adv,
                    float* out_returns, void* workspace, size_t workspace_bytes, void* stream)
{
    return rlhf_experience_ex(actor_logits, actor_stride_b, actor_stride_t, ref_logits, ref_stride_b, ref_stride_t,
                              RLHF_BF16, ids, ids_stride_b, lengths, score, values_old, lp_old, B, T, V, beta_kl,
                              reward_clip, gamma, lambda, out_lp_actor, out_lp_ref, out_rewards, out_adv, out_returns,
                              nullptr, workspace, workspace_bytes, stream);
}

int rlhf_ppo_loss_fwd_bwd_ex(const void* logits, int logits_dtype, long long stride_b, long long stride_t,
                             const long long* ids, long long ids_stride_b, const int* lengths,
                             const float* lp_old, const float* adv, const float* values_new,
                             const float* values_old, const float* returns,
                             int B, int T, int V, float clip_eps, float value_clip, float grad_scale,
                             float* out_loss_pg, float* out_loss_vf,
                             void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                             float* out_dvalues, float* out_lp_new,
                             void* workspace, size_t workspace_bytes, void* stream)
{
    if (logits_dtype != RLHF_BF16 && logits_dtype != RLHF_F16) return RLHF_ERR_SCALAR;
    const bool f16 = logits_dtype == RLHF_F16;
    if (int e = check_loss_args(logits, stride_b, stride_t, ids, ids_stride_b, lengths, lp_old, adv, values_new,
                                values_old, returns, B, T, V, clip_eps, value_clip, grad_scale, out_loss_pg,
                                out_loss_vf, out_dlogits, dl_stride_b, dl_stride_t, out_dvalues, out_lp_new))
        return e;
    if (int e = check_workspace(workspace, workspace_bytes, loss_workspace_bytes(B, T))) return e;
    DeviceInfo dev;
    if (int e = device_info(dev)) return e;

    char* ws = (char*)workspace;
    RowArgs a{};
    a.logits = (const uint16_t*)logits;
    a.stride_b = stride_b;
    a.stride_t = stride_t;
    a.ids = ids;
    a.ids_stride_b = ids_stride_b;
    a.lengths = lengths;
    a.B = B; a.T = T; a.V = V;
    a.status = (unsigned*)ws;
    a.wait_limit_ns = kWaitLimitNs;
    a.lp_old = lp_old;
    a.adv = adv;
    a.clip_eps = clip_eps;
    a.grad_scale = grad_scale;
    a.dlogits = (uint16_t*)out_dlogits;
    a.dl_stride_b = dl_stride_b;
    a.dl_stride_t = dl_stride_t;
    a.row_loss = (float*)(ws + kRowLossOffset);
    a.out_lp_new = out_lp_new;

    cudaStream_t s = (cudaStream_t)stream;
    long long rows = (long long)B * T;
    const bool all_16B = rows_16B(logits, stride_b, stride_t, V) && rows_16B(out_dlogits, dl_stride_b, dl_stride_t, V);
    // rows off 16-byte boundaries can still take the fast kernel if every dlogits row is as far off a boundary as
    // its logits row (in place, or a second tensor of the same layout)
    const bool same_offsets = ((reinterpret_cast<uintptr_t>(out_dlogits) - reinterpret_cast<uintptr_t>(logits)) % 16) == 0 &&
                              ((dl_stride_b - stride_b) % 8) == 0 && ((dl_stride_t - stride_t) % 8) == 0;
    const CregPlan any_plan = plan_creg_any(V, dev);
    const bool ragged_fast = !all_16B && same_offsets && any_plan.cluster == 1;
    if (((all_16B && fast_loss_rows_apply(V, f16, dev)) || ragged_fast) && dev.sm_count * 7 <= kMaxFusedBlocks) {
        // fast path: the row kernel also does the finalisation (value loss, dvalues, loss reduction)
        a.fused = 1;
        a.values_new = values_new;
        a.values_old = values_old;
        a.returns = returns;
        a.value_clip = value_clip;
        a.out_dvalues = out_dvalues;
        a.out_loss_pg = out_loss_pg;
        a.out_loss_vf = out_loss_vf;
        a.ticket = (unsigned*)(ws + 4);
        a.partials = (double*)(ws + kPartialsOffset);
        if (ragged_fast) {
            if (int e = f16 ? launch_creg_any<true>(a, any_plan, dev, s) : launch_creg_any<false>(a, any_plan, dev, s)) return e;
        } else {
            if (int e = launch_loss_rows(a, f16, dev, s)) return e;
        }
        return launch_check("loss row kernel");
    } else {
        int grid = (int)std::min<long long>(rows, (long long)dev.sm_count * 8);
        if (f16) RLHF_CUDA(launch_kernel(row_generic_kernel<true, true>, grid, kGenericThreads, 0, s, a));
        else RLHF_CUDA(launch_kernel(row_generic_kernel<true, false>, grid, kGenericThreads, 0, s, a));
        if (int e = launch_check("row_generic_kernel<loss>")) return e;
    }

    FinalArgs f{};
    f.lengths = lengths;
    f.B = B; f.T = T;
    f.values_new = values_new;
    f.values_old = values_old;
    f.returns = returns;
    f.row_loss = a.row_loss;
    f.value_clip = value_clip;
    f.grad_scale = grad_scale;
    f.out_dvalues = out_dvalues;
    f.out_lp_new = out_lp_new;
    f.out_loss_pg = out_loss_pg;
    f.out_loss_vf = out_loss_vf;
    f.status = (unsigned*)ws;
    f.ticket = (unsigned*)(ws + 4);
    f.partials = (double*)(ws + kPartialsOffset);
    int fgrid = (int)std::min<long long>((rows + 1023) / 1024, kFinalMaxBlocks);
    if (int e = keep_max_carveout(ppo_finalize_kernel)) return e;
    RLHF_CUDA(launch_kernel(ppo_finalize_kernel, fgrid, kFinalThreads, 0, s, f));
    return launch_check("ppo_finalize_kernel");
}

int rlhf_ppo_loss_fwd_bwd(const void* logits, long long stride_b, long long stride_t,
                          const long long* ids, long long ids_stride_b, const int* lengths,
                          const float* lp_old, const float* adv, const float* values_new,
                          const float* values_old, const float* returns,
                          int B, int T, int V, float clip_eps, float value_clip, float grad_scale,
                          float* out_loss_pg, float* out_loss_vf,
                          void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                          float* out_dvalues, float* out_lp_new,
                          void* workspace, size_t workspace_bytes, void* stream)
{
    return rlhf_ppo_loss_fwd_bwd_ex(logits, RLHF_BF16, stride_b, stride_t, ids, ids_stride_b, lengths, lp_old, adv,
                                    values_new, values_old, returns, B, T, V, clip_eps, value_clip, grad_scale,
                                    out_loss_pg, out_loss_vf, out_dlogits, dl_stride_b, dl_stride_t, out_dvalues,
                                    out_lp_new, workspace, workspace_bytes, stream);
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Entry point for callers that cannot allocate: scratch lives in a fixed device array of this image.
constexpr size_t kNoallocScratchBytes = 24576 + 4 * (size_t)RLHF_NOALLOC_MAX_TOKENS;

// In host code this name is only a handle for the symbol, not a device address; the address is
// obtained per device with cudaGetSymbolAddress below and that pointer is what the kernels get.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocScratchBytes];

namespace {

static_assert(kNoallocScratchBytes == kRowLossOffset + 4 * (size_t)RLHF_NOALLOC_MAX_TOKENS,
              "scratch array must hold the workspace of RLHF_NOALLOC_MAX_TOKENS tokens");
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device, looked up on first use per device.
int noalloc_scratch(void** out)
{
    int dev = 0;
    RLHF_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return cuda_fail(cudaErrorInvalidDevice, "device ordinal above 63");
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        RLHF_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        if (!ptr) return cuda_fail(cudaErrorInvalidSymbol, "cudaGetSymbolAddress returned a null address");
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return RLHF_OK;
}

}  // namespace

extern "C" int rlhf_ppo_loss_fwd_bwd_noalloc(const void* logits, long long stride_b, long long stride_t,
                                             const long long* ids, long long ids_stride_b, const int* lengths,
                                             const float* lp_old, const float* adv, const float* values_new,
                                             const float* values_old, const float* returns,
                                             int B, int T, int V, float clip_eps, float value_clip,
                                             float grad_scale, float* out_loss_pg, float* out_loss_vf,
                                             void* out_dlogits, long long dl_stride_b, long long dl_stride_t,
                                             float* out_dvalues, float* out_lp_new,
                                             unsigned int* out_device_status, void* stream)
{
    if (B <= 0 || T <= 0) return RLHF_ERR_SHAPE;
    if ((long long)B * (long long)T > (long long)RLHF_NOALLOC_MAX_TOKENS) return RLHF_ERR_TOO_LARGE;
    if (out_device_status && !aligned(out_device_status, 4)) return RLHF_ERR_ALIGN;
    // every host-side check first: a refused call must not have queued anything on the stream
    if (int e = check_loss_args(logits, stride_b, stride_t, ids, ids_stride_b, lengths, lp_old, adv, values_new,
                                values_old, returns, B, T, V, clip_eps, value_clip, grad_scale, out_loss_pg,
                                out_loss_vf, out_dlogits, dl_stride_b, dl_stride_t, out_dvalues, out_lp_new))
        return e;
    void* scratch = nullptr;
    if (int e = noalloc_scratch(&scratch)) return e;
    cudaStream_t s = (cudaStream_t)stream;
    // the status word, the reduction ticket and the row counter must start at zero; the rest is written before it is read
    RLHF_CUDA(cudaMemsetAsync(scratch, 0, 32, s));
    int e = rlhf_ppo_loss_fwd_bwd(logits, stride_b, stride_t, ids, ids_stride_b, lengths, lp_old, adv,
                                  values_new, values_old, returns, B, T, V, clip_eps, value_clip, grad_scale,
                                  out_loss_pg, out_loss_vf, out_dlogits, dl_stride_b, dl_stride_t,
                                  out_dvalues, out_lp_new, scratch, kNoallocScratchBytes, stream);
    if (e != RLHF_OK) return e;
    if (out_device_status)
        RLHF_CUDA(cudaMemcpyAsync(out_device_status, scratch, 4, cudaMemcpyDeviceToDevice, s));
    return RLHF_OK;
}
