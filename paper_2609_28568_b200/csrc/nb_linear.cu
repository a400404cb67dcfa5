// Host side of the nb_linear C ABI: argument checks, TMA descriptors, kernel selection, launches.
// Declarations and argument documentation live in include/nb_linear.h.
#include "nb_linear.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_map>

#include "elementwise.cuh"
#include "gemm_sm100.cuh"
#include "layer_bwd_sm100.cuh"
#include "lora_udb_sm100.cuh"

namespace {

using namespace nb;

constexpr int kMaxDevices = 64;
constexpr unsigned long long kDefaultTimeoutNs = 2000000000ull;  // 2 s per wait

std::atomic<long long> g_launches{0};
const bool g_use_pdl = [] {
    const char *e = getenv("NB_PDL");  // debugging aid: NB_PDL=0 turns dependent launch off
    return !(e && e[0] == '0');
}();
thread_local std::string g_err;
thread_local cudaStream_t g_stream = nullptr;

int fail(int code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

#define NB_CUDA(call)                                                                        \
    do {                                                                                     \
        cudaError_t e_ = (call);                                                             \
        if (e_ != cudaSuccess)                                                               \
            return fail(NB_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));        \
    } while (0)

// ----------------------------------------------------------------------------- per-device state
struct TmapKey {
    const void *ptr;
    uint64_t rows, cols, ld;
    uint32_t box_cols, box_rows, dtype;
    bool operator==(const TmapKey &o) const
    {
        return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_cols == o.box_cols &&
               box_rows == o.box_rows && dtype == o.dtype;
    }
};
struct TmapKeyHash {
    size_t operator()(const TmapKey &k) const
    {
        uint64_t h = reinterpret_cast<uint64_t>(k.ptr) * 0x9E3779B97F4A7C15ull;
        h ^= (k.rows + 0x7F4A7C15ull) * 0xBF58476D1CE4E5B9ull;
        h ^= (k.cols + 0x165667B1ull) * 0x94D049BB133111EBull;
        h ^= (k.ld + 0x2545F491ull) * 0xD6E8FEB86659FD93ull;
        h ^= (static_cast<uint64_t>(k.box_cols) << 40) ^ (static_cast<uint64_t>(k.box_rows) << 20) ^
             k.dtype;
        return static_cast<size_t>(h ^ (h >> 29));
    }
};

struct DeviceState {
    bool init = false;
    int num_sms = 0;
    int *status = nullptr;   // 16 ints on the device
    void *workspace = nullptr;
    size_t workspace_bytes = 0;
    std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> tmaps;
};

std::mutex g_mu;
DeviceState g_dev[kMaxDevices];

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int get_state(DeviceState **out)
{
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(NB_ERR_UNSUPPORTED, "device index %d", dev);
    DeviceState &s = g_dev[dev];
    if (!s.init) {
        cudaDeviceProp prop;
        NB_CUDA(cudaGetDeviceProperties(&prop, dev));
        if (prop.major != 10)
            return fail(NB_ERR_UNSUPPORTED,
                        "device %d is sm_%d%d; this library only runs on sm_100 (B200)", dev,
                        prop.major, prop.minor);
        s.num_sms = prop.multiProcessorCount;
        NB_CUDA(cudaMalloc(reinterpret_cast<void **>(&s.status), 64));
        NB_CUDA(cudaMemset(s.status, 0, 64));
        if (!g_encode) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            NB_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
            if (qres != cudaDriverEntryPointSuccess || !fn)
                return fail(NB_ERR_CUDA, "cuTensorMapEncodeTiled is not available in this driver");
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        s.init = true;
    }
    *out = &s;
    return NB_OK;
}

// Row-major [rows, cols] tensor, tiles of box_rows x box_cols with the 128-byte swizzle.
// dtype: 0 bf16, 1 fp32. The innermost box extent is always 128 bytes (64 bf16 / 32 fp32).
// ld: elements from one row to the next (0: dense, = cols); a column slice of a wider tensor is a
// view with ld > cols, and what lies beyond its cols reads as zero and is never written.
int get_tmap(DeviceState &s, CUtensorMap *out, const void *ptr, uint64_t rows, uint64_t cols,
             uint32_t dtype, uint32_t box_rows, uint64_t ld = 0)
{
    const uint32_t esz = dtype == 0 ? 2u : 4u;
    const uint32_t box_cols = 128u / esz;
    if (ld == 0) ld = cols;
    if (ld < cols || (ld * esz) % 16 != 0)
        return fail(NB_ERR_UNSUPPORTED, "row stride of %llu elements is not a multiple of 16 bytes",
                    static_cast<unsigned long long>(ld));
    TmapKey key{ptr, rows, cols, ld, box_cols, box_rows, dtype};
    auto it = s.tmaps.find(key);
    if (it != s.tmaps.end()) {
        *out = it->second;
        return NB_OK;
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * esz};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    // The encoder does not write every byte of the opaque descriptor: start from zeros, otherwise
    // stack garbage ends up in fields the TMA unit reads.
    alignas(64) CUtensorMap m;
    memset(&m, 0, sizeof(m));
    CUresult r = g_encode(&m, dtype == 0 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                          2, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(NB_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) for [%llu, %llu] at %p",
                    static_cast<int>(r), static_cast<unsigned long long>(rows),
                    static_cast<unsigned long long>(cols), ptr);
    if (s.tmaps.size() > 8192) s.tmaps.clear();
    s.tmaps.emplace(key, m);
    *out = m;
    return NB_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_dims(int64_t BT, int64_t C, int64_t OC)
{
    if (BT < 0 || C <= 0 || OC <= 0) return fail(NB_ERR_INVALID_ARG, "negative or zero dimension");
    if (BT >= (1ll << 31) || C >= (1ll << 31) || OC >= (1ll << 31) || BT * OC >= (1ll << 40) ||
        BT * C >= (1ll << 40))
        return fail(NB_ERR_UNSUPPORTED, "dimension too large");
    if (C % 8 != 0 || OC % 8 != 0)
        return fail(NB_ERR_UNSUPPORTED, "C (%lld) and OC (%lld) must be multiples of 8",
                    static_cast<long long>(C), static_cast<long long>(OC));
    return NB_OK;
}

// Programmatic dependent launch is used unless it is switched off, or the stream is being captured
// and this launch has more than one dependency (see launch_gemm).
bool dependent_launch_allowed(cudaStream_t stream)
{
    if (!g_use_pdl) return false;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    const cudaGraphNode_t *deps = nullptr;
    size_t ndeps = 0;
    if (cudaStreamGetCaptureInfo(stream, &cs, nullptr, nullptr, &deps, &ndeps) != cudaSuccess) {
        (void)cudaGetLastError();
        cs = cudaStreamCaptureStatusNone;
    }
    return !(cs == cudaStreamCaptureStatusActive && ndeps != 1);
}

// ----------------------------------------------------------------------------- GEMM launch
struct GemmArgs {
    const void *A;  uint64_t a_rows, a_cols;   // global tensor of the A operand (bf16)
    const void *B;  uint64_t b_rows, b_cols;   // global tensor of the B operand (bf16)
    void *D;        uint64_t d_rows, d_cols;  uint32_t d_dtype;
    const void *E;  uint64_t e_rows, e_cols;   // second bf16 tensor (pre-activation / aux) or null
    int M, N, K;
    const void *bias;
    int swiglu_h;
    int reduce;
    int splits;
    float *dbias;  // wgrad: bias gradient fused into the pass over dz, or null
    // adapter term D += A2 . B2^T over k2 columns (k2 <= 64), read after the main k range
    const void *A2; uint64_t a2_rows, a2_cols;
    const void *B2; uint64_t b2_rows, b2_cols;
    int k2;
    float alpha;   // D = alpha * acc (+ bias); 0 is read as 1
    uint64_t a_ld, b_ld, d_ld, a2_ld;  // row strides in elements of A, B, D, A2 when they are column slices (0: dense)
    float2 *stats; // forward with softmax statistics: [M, stats_ld]
    int stats_ld;
    int v_real;
    int debug_stop_kb;                  // nb_debug_gemm_timeout only: see GemmParams; 0 = unset (-1 is passed on)
    unsigned long long debug_timeout_ns;  //   and its shortened wait limit
};

template <class Cfg>
int launch_gemm(DeviceState &s, const GemmArgs &a, cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    static int max_clusters[kMaxDevices] = {};
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (!attr_set[dev]) {
        NB_CUDA(cudaFuncSetAttribute(gemm_kernel<Cfg>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(Cfg::SMEM_BYTES)));
        max_clusters[dev] = s.num_sms / Cfg::CG;
        if (Cfg::CG == 2) {  // how many CTA pairs can be resident at once
            cudaLaunchConfig_t qc = {};
            qc.gridDim = dim3(static_cast<unsigned>(s.num_sms));
            qc.blockDim = dim3(Cfg::THREADS);
            qc.dynamicSmemBytes = Cfg::SMEM_BYTES;
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 2;
            qa[0].val.clusterDim.y = 1;
            qa[0].val.clusterDim.z = 1;
            qc.attrs = qa;
            qc.numAttrs = 1;
            int n = 0;
            NB_CUDA(cudaOccupancyMaxActiveClusters(&n, gemm_kernel<Cfg>, &qc));
            if (n < 1) return fail(NB_ERR_CUDA, "no CTA pair of this kernel fits on the device");
            if (n < max_clusters[dev]) max_clusters[dev] = n;
        }
        attr_set[dev] = true;
    }
    CUtensorMap tA, tB, tD, tE;
    int rc;
    // operands are fetched as 64 x 64 boxes; results (and the aux tile) move as 128-row chunks
    if ((rc = get_tmap(s, &tA, a.A, a.a_rows, a.a_cols, 0, 64, a.a_ld)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tB, a.B, a.b_rows, a.b_cols, 0, 64, a.b_ld)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tD, a.D, a.d_rows, a.d_cols, a.d_dtype, Cfg::OUT_BOX_ROWS, a.d_ld)) != NB_OK) return rc;
    if (a.E) {
        if ((rc = get_tmap(s, &tE, a.E, a.e_rows, a.e_cols, 0, Cfg::OUT_BOX_ROWS)) != NB_OK) return rc;
    } else {
        tE = tD;
    }
    CUtensorMap tA2 = tA, tB2 = tB;
    if (a.A2 && a.B2 && a.k2 > 0) {
        if ((rc = get_tmap(s, &tA2, a.A2, a.a2_rows, a.a2_cols, 0, 64, a.a2_ld)) != NB_OK) return rc;
        if ((rc = get_tmap(s, &tB2, a.B2, a.b2_rows, a.b2_cols, 0, 64)) != NB_OK) return rc;
    }
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.M = a.M;
    p.N = a.N;
    p.K = a.K;
    p.tiles_m = (a.M + Cfg::TILE_M - 1) / Cfg::TILE_M;
    const int n_span = (Cfg::EPI == kEpiSwiglu) ? a.swiglu_h : a.N;
    const int n_tile = (Cfg::EPI == kEpiSwiglu) ? 128 : Cfg::BLOCK_N;
    p.tiles_n = (n_span + n_tile - 1) / n_tile;
    p.kblocks = (a.K + kBlockK - 1) / kBlockK;
    int splits = a.splits < 1 ? 1 : a.splits;
    if (splits > p.kblocks) splits = p.kblocks;
    p.kblocks_per_split = (p.kblocks + splits - 1) / splits;
    p.splits = (p.kblocks + p.kblocks_per_split - 1) / p.kblocks_per_split;
    // rasterisation: units walk `group_m` row tiles for each column tile before moving to the next
    // column tile. Many column tiles (the head): a tall group keeps the weight tiles' reuse in L2;
    // few column tiles: a short group keeps the row tiles' (measured on B200, 1-2 % either way)
    p.kblocks_ext = (a.A2 && a.B2 && a.k2 > 0 && p.splits == 1) ? (a.k2 + kBlockK - 1) / kBlockK : 0;
    p.alpha = a.alpha == 0.0f ? 1.0f : a.alpha;
    p.group_m = (p.tiles_n >= 64 ? 64 : p.tiles_n <= 4 ? 4 : 16) / Cfg::CG;
    p.swiglu_h = a.swiglu_h;
    p.reduce = a.reduce;
    p.bias = static_cast<const __nv_bfloat16 *>(a.bias);
    p.dbias = a.dbias;
    p.stats = a.stats;
    p.stats_ld = a.stats_ld;
    p.v_real = a.v_real;
    p.status = s.status;
    p.timeout_ns = a.debug_timeout_ns ? a.debug_timeout_ns : kDefaultTimeoutNs;
    p.debug_stop_kb = a.debug_stop_kb > 0 ? a.debug_stop_kb : -1;
    const long long units = 1ll * p.tiles_m * p.tiles_n * p.splits;
    if (units <= 0 || units >= (1ll << 31)) return fail(NB_ERR_UNSUPPORTED, "tile count out of range");
    const int clusters = static_cast<int>(units < max_clusters[dev] ? units : max_clusters[dev]);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(clusters * Cfg::CG));
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = Cfg::CG;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    // programmatic dependent launch: the kernel's set-up overlaps the previous kernel's tail; the
    // kernel itself waits for that kernel before it touches global memory
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    // While a stream is being captured into a graph, a launch that follows a wait on another
    // stream has more than one dependency; with the programmatic attribute all of them became
    // programmatic edges and the kernel then waited for only one (observed: a consumer started
    // before its cross-stream producer had finished). Such a launch keeps full dependencies.
    cfg.numAttrs = dependent_launch_allowed(stream) ? 2 : 1;
    NB_CUDA(cudaLaunchKernelEx(&cfg, gemm_kernel<Cfg>, tA, tB, tD, tE, tA2, tB2, p));
    ++g_launches;
    return NB_OK;
}

// Kernel configurations: <CTAs per tile, BLOCK_N, stages, staging buffers, A MN-major, B MN-major,
// epilogue>. The pair forms (256-row tiles) are used whenever there is more than one 128-row block;
// the single-CTA forms serve small row counts.
using FwdStore1 = GemmCfg<1, 256, 4, 2, false, false, kEpiStore>;
using FwdGelu1 = GemmCfg<1, 256, 3, 4, false, false, kEpiGelu>;
using FwdSwiglu1 = GemmCfg<1, 256, 3, 3, false, false, kEpiSwiglu>;
using DgradStore1 = GemmCfg<1, 256, 4, 2, false, true, kEpiStore>;
using DgradMulGelu1 = GemmCfg<1, 256, 2, 2, false, true, kEpiMulGeluGrad>;
using WgradF32_1 = GemmCfg<1, 256, 3, 4, true, true, kEpiF32>;
using WgradBf16_1 = GemmCfg<1, 256, 4, 2, true, true, kEpiStore>;
using FwdStore2 = GemmCfg<2, 256, 6, 2, false, false, kEpiStore>;
using FwdStoreStats1 = GemmCfg<1, 256, 4, 2, false, false, kEpiStoreStats>;
using FwdStoreStats2 = GemmCfg<2, 256, 6, 2, false, false, kEpiStoreStats>;
using FwdGelu2 = GemmCfg<2, 256, 5, 4, false, false, kEpiGelu>;
using FwdSwiglu2 = GemmCfg<2, 256, 5, 3, false, false, kEpiSwiglu>;
using DgradStore2 = GemmCfg<2, 256, 6, 2, false, true, kEpiStore>;
using DgradMulGelu2 = GemmCfg<2, 256, 4, 2, false, true, kEpiMulGeluGrad>;
using WgradF32_2 = GemmCfg<2, 256, 5, 4, true, true, kEpiF32>;
using WgradF32Bias1 = GemmCfg<1, 256, 3, 4, true, true, kEpiF32, true>;
using WgradF32Bias2 = GemmCfg<2, 256, 5, 4, true, true, kEpiF32, true>;
using WgradBf16_2 = GemmCfg<2, 256, 6, 2, true, true, kEpiStore>;
// Narrow results (N <= 64: the rank-r products of the adapter layer). A 256-wide tile would spend
// 4-16x the tensor-core time on padding; a 64-wide one leaves these products bound by the read of
// their tall operand, so they run one CTA per tile with a deep ring.
using FwdStoreNarrow = GemmCfg<1, 64, 7, 2, false, false, kEpiStore>;
using DgradStoreNarrow = GemmCfg<1, 64, 7, 2, false, true, kEpiStore>;
using WgradF32Narrow = GemmCfg<1, 64, 7, 2, true, true, kEpiF32>;
constexpr int kNarrowN = 64;

bool use_pairs(int M)
{
    static const int force = [] {
        const char *e = getenv("NB_CTA_GROUP");  // debugging aid: 1 or 2 forces one form
        return e ? atoi(e) : 0;
    }();
    if (force == 1) return false;
    if (force == 2) return true;
    return M > kBlockM;
}

template <class C1, class C2>
int launch_gemm_auto(DeviceState &s, const GemmArgs &a, cudaStream_t stream)
{
    return use_pairs(a.M) ? launch_gemm<C2>(s, a, stream) : launch_gemm<C1>(s, a, stream);
}

// Split-K factor for wgrad: the one whose waves of (tiles x splits) units over `slots` resident
// tiles take the least time, counting a fixed cost per unit (epilogue and pipeline ramp, about six
// k-blocks' worth). Every (m, n, k-range) is covered exactly once whatever the choice.
int choose_splits(int tiles, int kblocks, int slots)
{
    const int kUnitOverhead = 6;
    int best = 1;
    long long best_cost = -1;
    const int max_splits = kblocks / 4 > 1 ? kblocks / 4 : 1;
    for (int sp = 1; sp <= max_splits && sp <= 128; ++sp) {
        const int kps = (kblocks + sp - 1) / sp;
        const int eff = (kblocks + kps - 1) / kps;  // splits that are not empty
        const long long units = 1ll * tiles * eff;
        const long long waves = (units + slots - 1) / slots;
        const long long cost = waves * (kps + kUnitOverhead);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = eff;
        }
    }
    return best;
}

int ensure_workspace(DeviceState &s, size_t bytes, cudaStream_t stream = nullptr)
{
    if (s.workspace_bytes >= bytes) return NB_OK;
    // growing synchronises the device and frees memory that kernels of a graph under
    // construction may refer to: refuse instead of failing inside the runtime
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (stream != nullptr && cudaStreamIsCapturing(stream, &cs) != cudaSuccess) (void)cudaGetLastError();
    if (cs != cudaStreamCaptureStatusNone)
        return fail(NB_ERR_UNSUPPORTED,
                    "the workspace would have to grow to %zu bytes during stream capture; call "
                    "nb_workspace_reserve before capturing", bytes);
    if (s.workspace) {
        NB_CUDA(cudaDeviceSynchronize());
        NB_CUDA(cudaFree(s.workspace));
        s.workspace = nullptr;
        s.workspace_bytes = 0;
    }
    const size_t want = (bytes + (1u << 20) - 1) & ~static_cast<size_t>((1u << 20) - 1);
    NB_CUDA(cudaMalloc(&s.workspace, want));
    s.workspace_bytes = want;
    return NB_OK;
}

int launch_dbias(DeviceState &s, float *dbias, const void *dz, int64_t BT, int64_t OC, int accumulate,
                 cudaStream_t stream)
{
    if (!accumulate) NB_CUDA(cudaMemsetAsync(dbias, 0, static_cast<size_t>(OC) * 4, stream));
    if (BT == 0) return NB_OK;
    const int col_blocks = static_cast<int>((OC + kDbiasCols - 1) / kDbiasCols);
    // about three blocks per SM: with six (or one) the same kernel was 15-25 % slower on the stack's
    // shapes (measured: 16.6 us against 19.2 us for 16384 x 2304)
    long long want_row_blocks = (3ll * s.num_sms + col_blocks - 1) / col_blocks;
    long long rows_per_block = (BT + want_row_blocks - 1) / want_row_blocks;
    rows_per_block = ((rows_per_block + 127) / 128) * 128;  // a block sweeps 128 rows per iteration
    if (rows_per_block < 128) rows_per_block = 128;
    const long long row_blocks = (BT + rows_per_block - 1) / rows_per_block;
    if (row_blocks > 65535) return fail(NB_ERR_UNSUPPORTED, "BT too large for the dbias grid");
    dim3 grid(col_blocks, static_cast<unsigned>(row_blocks));
    dbias_kernel<<<grid, kDbiasThreads, 0, stream>>>(dbias, static_cast<const __nv_bfloat16 *>(dz), BT,
                                                     static_cast<int>(OC),
                                                     static_cast<int>(rows_per_block));
    NB_CUDA(cudaGetLastError());
    ++g_launches;
    return NB_OK;
}

int elementwise_grid(const DeviceState &s, long long nvec)
{
    long long blocks = (nvec + 255) / 256;
    const long long cap = 16ll * s.num_sms;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return static_cast<int>(blocks);
}

// dweight[M_, N_] (+)= dz^T . inp over BT rows, fp32, with the split-K factor chosen per shape;
// dz [BT, M_], inp [BT, N_]. dbias (or null) is summed inside the same kernel.
int run_wgrad_f32(DeviceState &s, const void *dz, const void *inp, void *dweight, float *dbias,
                  int64_t BT, int64_t M_, int64_t N_, int accumulate, cudaStream_t stream,
                  uint64_t inp_ld = 0)
{
    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = dz; a.a_rows = BT; a.a_cols = M_;
    a.B = inp; a.b_rows = BT; a.b_cols = N_; a.b_ld = inp_ld;
    a.D = dweight; a.d_rows = M_; a.d_cols = N_; a.d_dtype = 1;
    a.M = static_cast<int>(M_); a.N = static_cast<int>(N_); a.K = static_cast<int>(BT);
    const bool narrow = dbias == nullptr && a.N <= kNarrowN;
    const bool pairs = !narrow && use_pairs(a.M);
    const int tile_m = pairs ? 2 * kBlockM : kBlockM;
    const int tile_n = narrow ? kNarrowN : 256;
    const int tiles = ((a.M + tile_m - 1) / tile_m) * ((a.N + tile_n - 1) / tile_n);
    const int kblocks = (a.K + kBlockK - 1) / kBlockK;
    const int slots = s.num_sms / (pairs ? 2 : 1);  // tiles resident at once
    const int splits = choose_splits(tiles, kblocks, slots);
    a.splits = splits;
    a.reduce = (accumulate || splits > 1) ? 1 : 0;
    if (!accumulate && splits > 1)
        NB_CUDA(cudaMemsetAsync(dweight, 0, static_cast<size_t>(M_ * N_) * 4, stream));
    if (dbias) {  // the bias gradient rides along: reducer warps sum dz while it is in shared memory
        if (!accumulate) NB_CUDA(cudaMemsetAsync(dbias, 0, static_cast<size_t>(M_) * 4, stream));
        a.dbias = dbias;
        return launch_gemm_auto<WgradF32Bias1, WgradF32Bias2>(s, a, stream);
    }
    if (narrow) return launch_gemm<WgradF32Narrow>(s, a, stream);
    return launch_gemm_auto<WgradF32_1, WgradF32_2>(s, a, stream);
}

// u = bf16(scale * dy . B) and dB (+)= dy^T . t of one adapted projection from one pass over dy
// (lora_udb_sm100.cuh). u and t may be column slices of wider tensors (row strides u_ld, t_ld).
// x and dlora_a both non-NULL: the A gradient dlora_a [r, C] (+)= u^T . x rides on the same launch
// (only with the whole of u in one call: u_ld == r).
int launch_lora_udb(DeviceState &s, const void *dy, const void *lora_b, const void *t, uint64_t t_ld, void *dlora_b,
                    void *u, uint64_t u_ld, float scale, int64_t BT, int64_t OC, int64_t r, int accumulate,
                    cudaStream_t stream, const void *x = nullptr, void *dlora_a = nullptr, int64_t C = 0)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (!attr_set[dev]) {
        NB_CUDA(cudaFuncSetAttribute(lora_udb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(kUdbSmemBytes)));
        attr_set[dev] = true;
    }
    const bool want_da = x != nullptr && dlora_a != nullptr;
    CUtensorMap tDy, tB, tT, tDb, tX, tDa;
    int rc;
    if ((rc = get_tmap(s, &tDy, dy, BT, OC, 0, 64)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tB, lora_b, OC, r, 0, 64)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tT, t, BT, r, 0, 64, t_ld)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tDb, dlora_b, OC, r, 1, 32)) != NB_OK) return rc;
    if (want_da) {
        if ((rc = get_tmap(s, &tX, x, BT, C, 0, 64)) != NB_OK) return rc;
        if ((rc = get_tmap(s, &tDa, dlora_a, r, C, 1, 32)) != NB_OK) return rc;
    } else {
        tX = tDy;   // never dereferenced
        tDa = tDb;
    }
    // every panel reduce-adds its share, so a fresh gradient starts from zero
    if (!accumulate) {
        NB_CUDA(cudaMemsetAsync(dlora_b, 0, static_cast<size_t>(OC * r) * 4, stream));
        if (want_da) NB_CUDA(cudaMemsetAsync(dlora_a, 0, static_cast<size_t>(r * C) * 4, stream));
    }
    UdbParams p;
    memset(&p, 0, sizeof(p));
    p.BT = static_cast<int>(BT);
    p.OC = static_cast<int>(OC);
    p.r = static_cast<int>(r);
    p.panels = static_cast<int>((BT + 127) / 128);
    p.tiles = static_cast<int>((OC + 127) / 128);
    p.want_db = 1;
    p.want_da = want_da ? 1 : 0;
    p.C = static_cast<int>(C);
    p.xtiles = want_da ? static_cast<int>((C + 127) / 128) : 0;
    p.alpha = scale;
    p.u = static_cast<__nv_bfloat16 *>(u);
    p.u_ld = static_cast<int>(u_ld);
    p.status = s.status;
    p.timeout_ns = kDefaultTimeoutNs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.panels < s.num_sms ? p.panels : s.num_sms));
    cfg.blockDim = dim3(kUdbThreads);
    cfg.dynamicSmemBytes = kUdbSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = dependent_launch_allowed(stream) ? 1 : 0;
    NB_CUDA(cudaLaunchKernelEx(&cfg, lora_udb_kernel, tDy, tB, tT, tDb, tX, tDa, p));
    ++g_launches;
    return NB_OK;
}

// ----------------------------------------------------------------------------- one launch per layer backward
int env_int(const char *name, int dflt)
{
    const char *e = getenv(name);
    return (e && *e) ? atoi(e) : dflt;
}

// The schedule of layer_bwd_kernel for P CTA pairs (layer_bwd_sm100.cuh describes the unit list).
// Costs are counted in k-blocks of tensor-core time: a D unit costs its k-blocks plus eD (the part
// of its epilogue the next main loop does not hide: larger with gelu'), a W unit its k-blocks plus
// eW. Every pair should end up with the same cost.
//  1. K = BT of the weight gradient is cut into chunks so that there are about two W units per
//     pair, none shorter than 32 k-blocks (every unit reduce-adds a whole fp32 tile: fewer, longer
//     units mean less traffic; in-step timings did not tell 16 to 128 k-blocks apart).
//  2. Whole rounds (one unit per pair) are dealt first; W rounds are spread evenly among D rounds.
//  3. The last D round is partial: pairs [0, d_tail) take one more tile. The W units left over are
//     laid out as one line of k-blocks and cut into P ranges, shorter by one D unit's cost for the
//     pairs that took a tail tile. If the line is too short for that, one W round is taken back.
// Returns NB_ERR_UNSUPPORTED when the shape needs more rounds than the order mask holds.
int plan_layer_bwd(LayerBwdParams &p, int64_t BT, int64_t C, int64_t OC, int P, bool gelu_grad)
{
    memset(&p, 0, sizeof(p));
    if (P < 1 || P > kMaxPairs) return fail(NB_ERR_UNSUPPORTED, "CTA pair count %d out of range", P);
    static const int eD_plain = env_int("NB_LB_ED", 3);
    static const int eD_gelu = env_int("NB_LB_ED_GELU", 8);
    static const int eW = env_int("NB_LB_EW", 3);
    static const int kbc_forced = env_int("NB_LB_KBC", 0);
    const int eD = gelu_grad ? eD_gelu : eD_plain;
    p.BT = static_cast<int>(BT);
    p.C = static_cast<int>(C);
    p.OC = static_cast<int>(OC);
    p.num_pairs = P;
    p.d_tiles_m = static_cast<int>((BT + 255) / 256);
    p.d_tiles_n = static_cast<int>((C + 255) / 256);
    p.d_tiles = p.d_tiles_m * p.d_tiles_n;
    p.d_kblocks = static_cast<int>((OC + kBlockK - 1) / kBlockK);
    p.d_group_m = (p.d_tiles_n >= 64 ? 64 : p.d_tiles_n <= 4 ? 4 : 16) / 2;
    p.w_tiles_m = static_cast<int>((OC + 255) / 256);
    p.w_tiles_n = p.d_tiles_n;
    p.w_tiles = p.w_tiles_m * p.w_tiles_n;
    p.w_kblocks = static_cast<int>((BT + kBlockK - 1) / kBlockK);
    int chunks = (2 * P + p.w_tiles - 1) / p.w_tiles;
    const int max_chunks = p.w_kblocks / 32 > 1 ? p.w_kblocks / 32 : 1;
    if (chunks > max_chunks) chunks = max_chunks;
    if (chunks < 1) chunks = 1;
    p.w_kbc = (p.w_kblocks + chunks - 1) / chunks;
    if (kbc_forced > 0) p.w_kbc = kbc_forced < p.w_kblocks ? kbc_forced : p.w_kblocks;
    chunks = (p.w_kblocks + p.w_kbc - 1) / p.w_kbc;
    const long long w_units = 1ll * chunks * p.w_tiles;
    if (w_units >= (1ll << 24) || p.d_tiles >= (1 << 24)) return fail(NB_ERR_UNSUPPORTED, "too many work units");
    p.w_units = static_cast<int>(w_units);
    p.d_rounds = p.d_tiles / P;
    p.d_tail = p.d_tiles % P;
    const double cD = p.d_kblocks + eD;
    // the units of the last chunk may be shorter than the others: they all stay in the tail, where
    // lengths are counted exactly
    p.w_last_len = p.w_kblocks - (chunks - 1) * p.w_kbc;
    const int even_units = p.w_last_len == p.w_kbc ? p.w_units : p.w_units - p.w_tiles;
    int aW = even_units / P;
    double b_hi = 0.0, b_lo = 0.0;  // tail k-blocks of a pair without / with a tail D tile
    long long Rk = 0;
    for (;; --aW) {
        const long long tail_full = 1ll * (even_units - aW * P) * p.w_kbc;
        Rk = tail_full + 1ll * (p.w_units - even_units) * p.w_last_len;
        p.w_tail_full = static_cast<int>(tail_full < (1ll << 30) ? tail_full : (1ll << 30));
        b_hi = static_cast<double>(Rk) / P + cD * p.d_tail / P;
        b_lo = b_hi - cD;
        const bool fits = p.d_tail == 0 ? (Rk == 0 || Rk >= 8ll * P) : b_lo >= 8.0;
        if (fits || aW == 0) break;
    }
    if (Rk >= (1ll << 30)) return fail(NB_ERR_UNSUPPORTED, "weight-gradient tail too long");
    p.w_rounds = aW;
    const int rounds = p.d_rounds + p.w_rounds;
    if (rounds > kLbMaxRounds) return fail(NB_ERR_UNSUPPORTED, "more than %d rounds", kLbMaxRounds);
    p.round_is_w = 0;
    for (int r = 0; r < rounds; ++r)
        if (1ll * (r + 1) * aW / rounds > 1ll * r * aW / rounds) p.round_is_w |= 1ull << r;
    // Tail ranges. Pair q's share is what levels the cost of the pairs still to be served: the
    // k-blocks and per-piece allowances left on the line plus their fixed costs (tail D tile),
    // divided among them, minus its own fixed cost. A range ends on a multiple of four k-blocks of
    // its unit or at the unit's end.
    (void)b_hi;
    (void)b_lo;
    const int tail_units = p.w_units - aW * P;
    const long long full_units = p.w_tail_full / p.w_kbc;
    auto unit_at = [&](long long x, long long &u_idx, long long &u_left) {
        if (x < p.w_tail_full) {
            u_idx = x / p.w_kbc;
            u_left = p.w_kbc - x % p.w_kbc;
        } else {
            const long long xr = x - p.w_tail_full;
            u_idx = full_units + xr / p.w_last_len;
            u_left = p.w_last_len - xr % p.w_last_len;
        }
    };
    long long x = 0;
    p.w_tail_begin[0] = 0;
    for (int q = 0; q < P; ++q) {
        if (q == P - 1) {
            x = Rk;
        } else if (x < Rk) {
            long long u_idx, u_left;
            unit_at(x, u_idx, u_left);
            const int pairs_left = P - q;
            const int tail_d_left = p.d_tail > q ? p.d_tail - q : 0;
            const double line_cost = static_cast<double>(Rk - x) + 1.0 * eW * (tail_units - u_idx) +
                                     1.0 * eW * (pairs_left - 1);
            double rem = (line_cost + cD * tail_d_left) / pairs_left - (q < p.d_tail ? cD : 0.0);
            while (x < Rk && rem >= eW + 4) {
                unit_at(x, u_idx, u_left);
                long long take = static_cast<long long>(rem - eW);
                if (take >= u_left) {
                    take = u_left;
                } else {
                    take = take / 4 * 4;
                    if (take <= 0) break;
                }
                x += take;
                rem -= eW + take;
                if (take < u_left) break;
            }
        }
        p.w_tail_begin[q + 1] = static_cast<int>(x);
    }
    for (int q = P + 1; q <= kMaxPairs; ++q) p.w_tail_begin[q] = static_cast<int>(Rk);
    return NB_OK;
}

using LayerBwdPlain = LbCfg<false, false>;
using LayerBwdBias = LbCfg<false, true>;
using LayerBwdGelu = LbCfg<true, false>;
using LayerBwdGeluBias = LbCfg<true, true>;

template <class Cfg>
int launch_layer_bwd(DeviceState &s, const void *dz, const void *weight, const void *inp, void *dinp,
                     const void *inp_pre, void *dweight, float *dbias, int64_t BT, int64_t C, int64_t OC,
                     int accumulate, cudaStream_t stream)
{
    static bool attr_set[kMaxDevices] = {};
    static int max_pairs[kMaxDevices] = {};
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (!attr_set[dev]) {
        NB_CUDA(cudaFuncSetAttribute(layer_bwd_kernel<Cfg>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(Cfg::SMEM_BYTES)));
        cudaLaunchConfig_t qc = {};
        qc.gridDim = dim3(static_cast<unsigned>(s.num_sms));
        qc.blockDim = dim3(kLbThreads);
        qc.dynamicSmemBytes = Cfg::SMEM_BYTES;
        cudaLaunchAttribute qa[1];
        qa[0].id = cudaLaunchAttributeClusterDimension;
        qa[0].val.clusterDim.x = 2;
        qa[0].val.clusterDim.y = 1;
        qa[0].val.clusterDim.z = 1;
        qc.attrs = qa;
        qc.numAttrs = 1;
        int n = 0;
        NB_CUDA(cudaOccupancyMaxActiveClusters(&n, layer_bwd_kernel<Cfg>, &qc));
        if (n < 1) return fail(NB_ERR_CUDA, "no CTA pair of the layer-backward kernel fits on the device");
        max_pairs[dev] = n < s.num_sms / 2 ? n : s.num_sms / 2;
        if (max_pairs[dev] > kMaxPairs) max_pairs[dev] = kMaxPairs;
        attr_set[dev] = true;
    }
    LayerBwdParams p;
    int rc = plan_layer_bwd(p, BT, C, OC, max_pairs[dev], Cfg::GELU_GRAD);
    if (rc != NB_OK) return rc;
    p.dbias = Cfg::DBIAS ? dbias : nullptr;
    p.status = s.status;
    p.timeout_ns = kDefaultTimeoutNs;
    CUtensorMap tDz, tW, tInp, tDinp, tPre, tDw;
    if ((rc = get_tmap(s, &tDz, dz, BT, OC, 0, 64)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tW, weight, OC, C, 0, 64)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tInp, inp, BT, C, 0, 64)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tDinp, dinp, BT, C, 0, 32)) != NB_OK) return rc;
    if ((rc = get_tmap(s, &tDw, dweight, OC, C, 1, 32)) != NB_OK) return rc;
    tPre = tDinp;
    if (Cfg::GELU_GRAD && (rc = get_tmap(s, &tPre, inp_pre, BT, C, 0, 32)) != NB_OK) return rc;
    // partial sums of every W unit are reduce-added, so a fresh gradient starts from zero
    if (!accumulate) {
        NB_CUDA(cudaMemsetAsync(dweight, 0, static_cast<size_t>(OC * C) * 4, stream));
        if (Cfg::DBIAS) NB_CUDA(cudaMemsetAsync(dbias, 0, static_cast<size_t>(OC) * 4, stream));
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * p.num_pairs));
    cfg.blockDim = dim3(kLbThreads);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = 2;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = dependent_launch_allowed(stream) ? 2 : 1;
    NB_CUDA(cudaLaunchKernelEx(&cfg, layer_bwd_kernel<Cfg>, tDz, tW, tInp, tDinp, tPre, tDw, p));
    ++g_launches;
    return NB_OK;
}

// dinp, fp32 dweight and (optionally) dbias of one layer from its dz in one launch. Returns
// NB_ERR_UNSUPPORTED (and launches nothing) for shapes the schedule does not cover; the caller
// then issues the products one by one.
int run_layer_bwd(DeviceState &s, const void *dz, const void *weight, const void *inp, void *dinp,
                  const void *inp_pre, void *dweight, float *dbias, int64_t BT, int64_t C, int64_t OC,
                  int accumulate, cudaStream_t stream)
{
    if (inp_pre) {
        if (dbias) return launch_layer_bwd<LayerBwdGeluBias>(s, dz, weight, inp, dinp, inp_pre, dweight, dbias, BT, C, OC, accumulate, stream);
        return launch_layer_bwd<LayerBwdGelu>(s, dz, weight, inp, dinp, inp_pre, dweight, dbias, BT, C, OC, accumulate, stream);
    }
    if (dbias) return launch_layer_bwd<LayerBwdBias>(s, dz, weight, inp, dinp, inp_pre, dweight, dbias, BT, C, OC, accumulate, stream);
    return launch_layer_bwd<LayerBwdPlain>(s, dz, weight, inp, dinp, inp_pre, dweight, dbias, BT, C, OC, accumulate, stream);
}

}  // namespace

// ================================================================================ C ABI
extern "C" {

int nb_version(void) { return 100; }

const char *nb_last_error(void) { return g_err.c_str(); }

int nb_set_stream(void *stream)
{
    g_stream = static_cast<cudaStream_t>(stream);
    return NB_OK;
}
void *nb_get_stream(void) { return g_stream; }

int64_t nb_linear_out_elems(int64_t BT, int64_t OC, int act)
{
    if (BT < 0 || OC < 0) return -1;
    switch (act) {
        case NB_ACT_NONE: return BT * OC;
        case NB_ACT_GELU: return 2 * BT * OC;
        case NB_ACT_SWIGLU: return (OC % 2) ? -1 : BT * (OC / 2) + BT * OC;
        default: return -1;
    }
}

int nb_linear_forward_ex(void *out, void *pre_act, const void *inp, const void *weight,
                         const void *bias, int64_t BT, int64_t C, int64_t OC, int act, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (act != NB_ACT_NONE && act != NB_ACT_GELU && act != NB_ACT_SWIGLU)
        return fail(NB_ERR_INVALID_ARG, "unknown activation %d", act);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if (act == NB_ACT_SWIGLU && OC % 16 != 0)
        return fail(NB_ERR_UNSUPPORTED, "SwiGLU needs OC/2 to be a multiple of 8");
    if (!out || !inp || !weight) return fail(NB_ERR_INVALID_ARG, "out, inp and weight must not be NULL");
    if (!aligned16(out) || !aligned16(inp) || !aligned16(weight) || !aligned16(pre_act) ||
        (bias && (reinterpret_cast<uintptr_t>(bias) & 1u)))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;

    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = weight; a.b_rows = OC; a.b_cols = C;
    a.D = out; a.d_rows = BT; a.d_cols = (act == NB_ACT_SWIGLU) ? OC / 2 : OC; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(OC); a.K = static_cast<int>(C);
    a.bias = bias;
    a.splits = 1;
    if (act == NB_ACT_NONE) return launch_gemm_auto<FwdStore1, FwdStore2>(*s, a, stream);
    if (!pre_act) {
        // the activated result without its pre-activation: only NONE can skip the second plane
        return fail(NB_ERR_INVALID_ARG, "pre_act must be given when act != NONE");
    }
    a.E = pre_act; a.e_rows = BT; a.e_cols = OC;
    if (act == NB_ACT_GELU) return launch_gemm_auto<FwdGelu1, FwdGelu2>(*s, a, stream);
    a.swiglu_h = static_cast<int>(OC / 2);
    return launch_gemm_auto<FwdSwiglu1, FwdSwiglu2>(*s, a, stream);
}

int nb_linear_forward(void *out, const void *inp, const void *weight, const void *bias, int64_t BT,
                      int64_t C, int64_t OC, int act)
{
    void *pre = nullptr;
    if (out && BT >= 0 && OC >= 0) {
        if (act == NB_ACT_GELU) pre = static_cast<uint16_t *>(out) + BT * OC;
        if (act == NB_ACT_SWIGLU) pre = static_cast<uint16_t *>(out) + BT * (OC / 2);
    }
    return nb_linear_forward_ex(out, pre, inp, weight, bias, BT, C, OC, act, g_stream);
}

int nb_linear_backward_ex(void *dinp, void *dweight, void *dbias, const void *dout, const void *inp,
                          const void *weight, const void *pre_act, const void *inp_pre_act,
                          int64_t BT, int64_t C, int64_t OC, int act, int accumulate,
                          int dweight_dtype, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (act != NB_ACT_NONE && act != NB_ACT_GELU && act != NB_ACT_SWIGLU)
        return fail(NB_ERR_INVALID_ARG, "unknown activation %d", act);
    if (dweight_dtype != NB_DTYPE_F32 && dweight_dtype != NB_DTYPE_BF16)
        return fail(NB_ERR_INVALID_ARG, "unknown dweight dtype %d", dweight_dtype);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if (act == NB_ACT_SWIGLU && OC % 16 != 0)
        return fail(NB_ERR_UNSUPPORTED, "SwiGLU needs OC/2 to be a multiple of 8");
    if (!dout) return fail(NB_ERR_INVALID_ARG, "dout must not be NULL");
    if (act != NB_ACT_NONE && !pre_act)
        return fail(NB_ERR_INVALID_ARG, "pre_act is required when act != NONE");
    if (dinp && !weight) return fail(NB_ERR_INVALID_ARG, "weight is required to compute dinp");
    if (dweight && !inp) return fail(NB_ERR_INVALID_ARG, "inp is required to compute dweight");
    if (inp_pre_act && !dinp) return fail(NB_ERR_INVALID_ARG, "inp_pre_act given without dinp");
    if (dweight_dtype == NB_DTYPE_BF16 && accumulate && dweight)
        return fail(NB_ERR_UNSUPPORTED, "bf16 dweight cannot be accumulated across micro-steps");
    if (!aligned16(dinp) || !aligned16(dweight) || !aligned16(dbias) || !aligned16(dout) ||
        !aligned16(inp) || !aligned16(weight) || !aligned16(pre_act) || !aligned16(inp_pre_act))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");

    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;

    if (BT == 0) {
        if (!accumulate) {
            const size_t wsz = dweight_dtype == NB_DTYPE_F32 ? 4 : 2;
            if (dweight) NB_CUDA(cudaMemsetAsync(dweight, 0, static_cast<size_t>(OC * C) * wsz, stream));
            if (dbias) NB_CUDA(cudaMemsetAsync(dbias, 0, static_cast<size_t>(OC) * 4, stream));
        }
        return NB_OK;
    }

    // dz: either dout itself, or dout times this layer's activation derivative (workspace)
    const void *dz = dout;
    if (act != NB_ACT_NONE) {
        if ((rc = ensure_workspace(*s, static_cast<size_t>(BT * OC) * 2, stream)) != NB_OK) return rc;
        if (act == NB_ACT_GELU) {
            const long long nvec = BT * OC / 8;
            gelu_backward_kernel<<<elementwise_grid(*s, nvec), 256, 0, stream>>>(
                static_cast<uint4 *>(s->workspace), static_cast<const uint4 *>(dout),
                static_cast<const uint4 *>(pre_act), nvec);
        } else {
            const int hvec = static_cast<int>(OC / 16);
            swiglu_backward_kernel<<<elementwise_grid(*s, BT * hvec), 256, 0, stream>>>(
                static_cast<uint4 *>(s->workspace), static_cast<const uint4 *>(dout),
                static_cast<const uint4 *>(pre_act), BT, hvec);
        }
        NB_CUDA(cudaGetLastError());
        ++g_launches;
        dz = s->workspace;
    }

    // Both products of the layer in one launch (the usual case of a training step): the weight
    // gradient's k-blocks fill the waves the input gradient's tiles leave partly empty.
    static const bool merged = env_int("NB_MERGED_BWD", 1) != 0;
    if (merged && dinp && dweight && dweight_dtype == NB_DTYPE_F32 && use_pairs(static_cast<int>(BT))) {
        rc = run_layer_bwd(*s, dz, weight, inp, dinp, inp_pre_act, dweight, static_cast<float *>(dbias), BT, C,
                           OC, accumulate, stream);
        if (rc != NB_ERR_UNSUPPORTED) return rc;
    }

    if (dinp) {  // dinp[BT, C] = dz[BT, OC] . W[OC, C]
        GemmArgs a;
        memset(&a, 0, sizeof(a));
        a.A = dz; a.a_rows = BT; a.a_cols = OC;
        a.B = weight; a.b_rows = OC; a.b_cols = C;
        a.D = dinp; a.d_rows = BT; a.d_cols = C; a.d_dtype = 0;
        a.M = static_cast<int>(BT); a.N = static_cast<int>(C); a.K = static_cast<int>(OC);
        a.splits = 1;
        if (inp_pre_act) {
            a.E = inp_pre_act; a.e_rows = BT; a.e_cols = C;
            rc = launch_gemm_auto<DgradMulGelu1, DgradMulGelu2>(*s, a, stream);
        } else {
            rc = launch_gemm_auto<DgradStore1, DgradStore2>(*s, a, stream);
        }
        if (rc != NB_OK) return rc;
    }

    if (dweight) {  // dweight[OC, C] (+)= dz^T[OC, BT] . inp[BT, C]
        GemmArgs a;
        memset(&a, 0, sizeof(a));
        a.A = dz; a.a_rows = BT; a.a_cols = OC;
        a.B = inp; a.b_rows = BT; a.b_cols = C;
        a.D = dweight; a.d_rows = OC; a.d_cols = C;
        a.M = static_cast<int>(OC); a.N = static_cast<int>(C); a.K = static_cast<int>(BT);
        if (dweight_dtype == NB_DTYPE_F32) {
            rc = run_wgrad_f32(*s, dz, inp, dweight, static_cast<float *>(dbias), BT, OC, C, accumulate,
                               stream);
            dbias = nullptr;  // done inside the wgrad kernel
        } else {
            a.d_dtype = 0;
            a.splits = 1;
            rc = launch_gemm_auto<WgradBf16_1, WgradBf16_2>(*s, a, stream);
        }
        if (rc != NB_OK) return rc;
    }

    if (dbias) {
        if ((rc = launch_dbias(*s, static_cast<float *>(dbias), dz, BT, OC, accumulate, stream)) != NB_OK)
            return rc;
    }
    return NB_OK;
}

int nb_linear_backward(void *dinp, void *dweight, void *dbias, const void *dout, const void *inp,
                       const void *weight, const void *pre_act, int64_t BT, int64_t C, int64_t OC,
                       int accumulate)
{
    return nb_linear_backward_ex(dinp, dweight, dbias, dout, inp, weight, pre_act, nullptr, BT, C, OC,
                                 pre_act ? NB_ACT_GELU : NB_ACT_NONE, accumulate, NB_DTYPE_F32,
                                 g_stream);
}

int nb_reduce_dbias(void *dbias, const void *dout, int64_t BT, int64_t OC, int accumulate)
{
    if (!dbias || !dout) return fail(NB_ERR_INVALID_ARG, "dbias and dout must not be NULL");
    if (BT < 0 || OC <= 0) return fail(NB_ERR_INVALID_ARG, "negative or zero dimension");
    if (OC % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "OC must be a multiple of 8");
    if (!aligned16(dbias) || !aligned16(dout))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    return launch_dbias(*s, static_cast<float *>(dbias), dout, BT, OC, accumulate, g_stream);
}

int nb_lm_head_ce_forward(void *logits, void *loss, void *lse, const void *inp, const void *weight,
                          const void *targets, int64_t BT, int64_t C, int64_t Vp, int64_t V,
                          void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, Vp);
    if (rc != NB_OK) return rc;
    if (V <= 0 || V > Vp) return fail(NB_ERR_INVALID_ARG, "V must be within (0, Vp]");
    if (!logits || !loss || !lse || !inp || !weight || !targets)
        return fail(NB_ERR_INVALID_ARG, "all pointers must be given");
    if (!aligned16(logits) || !aligned16(inp) || !aligned16(weight) ||
        (reinterpret_cast<uintptr_t>(loss) & 3u) || (reinterpret_cast<uintptr_t>(lse) & 3u) ||
        (reinterpret_cast<uintptr_t>(targets) & 3u))
        return fail(NB_ERR_INVALID_ARG, "misaligned pointer");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    const int stats_ld = 2 * static_cast<int>((Vp + 255) / 256);
    if ((rc = ensure_workspace(*s, static_cast<size_t>(BT) * stats_ld * sizeof(float2), stream)) != NB_OK) return rc;
    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = weight; a.b_rows = Vp; a.b_cols = C;
    a.D = logits; a.d_rows = BT; a.d_cols = Vp; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(Vp); a.K = static_cast<int>(C);
    a.splits = 1;
    a.stats = static_cast<float2 *>(s->workspace);
    a.stats_ld = stats_ld;
    a.v_real = static_cast<int>(V);
    if ((rc = launch_gemm_auto<FwdStoreStats1, FwdStoreStats2>(*s, a, stream)) != NB_OK) return rc;
    const unsigned blocks = static_cast<unsigned>((BT + 7) / 8);
    ce_reduce_kernel<<<blocks, 256, 0, stream>>>(static_cast<float *>(loss), static_cast<float *>(lse),
                                                 static_cast<const float2 *>(s->workspace), stats_ld,
                                                 static_cast<const __nv_bfloat16 *>(logits), Vp,
                                                 static_cast<const int *>(targets), BT, static_cast<int>(V));
    NB_CUDA(cudaGetLastError());
    ++g_launches;
    return NB_OK;
}

int nb_ce_backward(void *dlogits, const void *logits, const void *lse, const void *targets, float gscale,
                   int64_t BT, int64_t Vp, int64_t V, void *stream_)
{
    if (BT < 0 || Vp <= 0 || V <= 0 || V > Vp) return fail(NB_ERR_INVALID_ARG, "bad dimension");
    if (Vp % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "Vp must be a multiple of 8");
    if (BT >= (1ll << 31) || Vp >= (1ll << 31)) return fail(NB_ERR_UNSUPPORTED, "dimension too large");
    if (!dlogits || !logits || !lse || !targets) return fail(NB_ERR_INVALID_ARG, "all pointers must be given");
    if (!aligned16(dlogits) || !aligned16(logits)) return fail(NB_ERR_INVALID_ARG, "misaligned pointer");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    const int vec_per_row = static_cast<int>(Vp / 8);
    ce_backward_kernel<<<elementwise_grid(*s, BT * vec_per_row), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
        static_cast<uint4 *>(dlogits), static_cast<const uint4 *>(logits), static_cast<const float *>(lse),
        static_cast<const int *>(targets), gscale, BT, vec_per_row, static_cast<int>(V));
    NB_CUDA(cudaGetLastError());
    ++g_launches;
    return NB_OK;
}

int nb_lora_linear_forward(void *out, void *t, const void *inp, const void *weight, const void *bias,
                           const void *lora_a, const void *lora_b, float scale, int64_t BT, int64_t C,
                           int64_t OC, int64_t r, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if (r < 8 || r > 64 || r % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "rank must be 8..64, a multiple of 8");
    if (!out || !t || !inp || !weight || !lora_a || !lora_b)
        return fail(NB_ERR_INVALID_ARG, "out, t, inp, weight, lora_a and lora_b must not be NULL");
    if (!aligned16(out) || !aligned16(t) || !aligned16(inp) || !aligned16(weight) || !aligned16(lora_a) ||
        !aligned16(lora_b))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    GemmArgs a;
    memset(&a, 0, sizeof(a));  // t = scale * inp . A^T
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = lora_a; a.b_rows = r; a.b_cols = C;
    a.D = t; a.d_rows = BT; a.d_cols = r; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(r); a.K = static_cast<int>(C);
    a.splits = 1;
    a.alpha = scale;
    if ((rc = launch_gemm<FwdStoreNarrow>(*s, a, stream)) != NB_OK) return rc;
    memset(&a, 0, sizeof(a));  // out = inp . W^T (+ bias) + t . B^T: r extra columns of K
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = weight; a.b_rows = OC; a.b_cols = C;
    a.D = out; a.d_rows = BT; a.d_cols = OC; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(OC); a.K = static_cast<int>(C);
    a.bias = bias;
    a.splits = 1;
    a.A2 = t; a.a2_rows = BT; a.a2_cols = r;
    a.B2 = lora_b; a.b2_rows = OC; a.b2_cols = r;
    a.k2 = static_cast<int>(r);
    return launch_gemm_auto<FwdStore1, FwdStore2>(*s, a, stream);
}

int nb_lora_linear_backward(void *dinp, void *dlora_a, void *dlora_b, void *u, const void *dout,
                            const void *inp, const void *weight, const void *lora_a, const void *lora_b,
                            const void *t, float scale, int64_t BT, int64_t C, int64_t OC, int64_t r,
                            int accumulate, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if (r < 8 || r > 64 || r % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "rank must be 8..64, a multiple of 8");
    if (!u || !dout || !inp || !lora_a || !lora_b)
        return fail(NB_ERR_INVALID_ARG, "u, dout, inp, lora_a and lora_b must not be NULL");
    if (dinp && !weight) return fail(NB_ERR_INVALID_ARG, "weight is required to compute dinp");
    if (dlora_b && !t) return fail(NB_ERR_INVALID_ARG, "t (from the forward call) is required for dlora_b");
    if (!aligned16(dinp) || !aligned16(dlora_a) || !aligned16(dlora_b) || !aligned16(u) || !aligned16(dout) ||
        !aligned16(inp) || !aligned16(weight) || !aligned16(lora_a) || !aligned16(lora_b) || !aligned16(t))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    if (BT == 0) {
        if (!accumulate) {
            if (dlora_a) NB_CUDA(cudaMemsetAsync(dlora_a, 0, static_cast<size_t>(r * C) * 4, stream));
            if (dlora_b) NB_CUDA(cudaMemsetAsync(dlora_b, 0, static_cast<size_t>(OC * r) * 4, stream));
        }
        return NB_OK;
    }
    GemmArgs a;
    static const bool fused_udb = env_int("NB_LORA_FUSED", 1) != 0;
    static const bool fused_da = env_int("NB_LORA_FUSED_DA", 1) != 0;
    if (fused_udb && dlora_b) {  // u and dB from one pass over dout; dA from one pass over inp in the same launch
        const bool with_da = fused_da && dlora_a != nullptr;
        if ((rc = launch_lora_udb(*s, dout, lora_b, t, 0, dlora_b, u, static_cast<uint64_t>(r), scale, BT, OC, r,
                                  accumulate, stream, with_da ? inp : nullptr, with_da ? dlora_a : nullptr, C)) != NB_OK)
            return rc;
        dlora_b = nullptr;
        if (with_da) dlora_a = nullptr;
    } else {
        memset(&a, 0, sizeof(a));  // u = scale * dout . B   (B [OC, r] read as an MN-major operand)
        a.A = dout; a.a_rows = BT; a.a_cols = OC;
        a.B = lora_b; a.b_rows = OC; a.b_cols = r;
        a.D = u; a.d_rows = BT; a.d_cols = r; a.d_dtype = 0;
        a.M = static_cast<int>(BT); a.N = static_cast<int>(r); a.K = static_cast<int>(OC);
        a.splits = 1;
        a.alpha = scale;
        if ((rc = launch_gemm<DgradStoreNarrow>(*s, a, stream)) != NB_OK) return rc;
    }
    // dB right after u: both stream dout, and what the first pass brought into L2 serves the second
    if (dlora_b)  // dB [OC, r] (+)= dout^T . t      (t already carries the scale)
        if ((rc = run_wgrad_f32(*s, dout, t, dlora_b, nullptr, BT, OC, r, accumulate, stream)) != NB_OK)
            return rc;
    if (dinp) {  // dinp = dout . W + u . A: r extra rows of K
        memset(&a, 0, sizeof(a));
        a.A = dout; a.a_rows = BT; a.a_cols = OC;
        a.B = weight; a.b_rows = OC; a.b_cols = C;
        a.D = dinp; a.d_rows = BT; a.d_cols = C; a.d_dtype = 0;
        a.M = static_cast<int>(BT); a.N = static_cast<int>(C); a.K = static_cast<int>(OC);
        a.splits = 1;
        a.A2 = u; a.a2_rows = BT; a.a2_cols = r;
        a.B2 = lora_a; a.b2_rows = r; a.b2_cols = C;
        a.k2 = static_cast<int>(r);
        if ((rc = launch_gemm_auto<DgradStore1, DgradStore2>(*s, a, stream)) != NB_OK) return rc;
    }
    if (dlora_a)  // dA [r, C] (+)= u^T . inp        (u already carries the scale)
        if ((rc = run_wgrad_f32(*s, u, inp, dlora_a, nullptr, BT, r, C, accumulate, stream)) != NB_OK)
            return rc;
    return NB_OK;
}

// --- adapters that share an input, stacked (q, k, v; gate, up): one rank-R product for all of them
namespace {
int check_stack(int64_t r, int64_t R, int64_t off)
{
    if (r < 8 || r > 64 || r % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "rank must be 8..64, a multiple of 8");
    if (R < r || R > 64 || R % 8 != 0)
        return fail(NB_ERR_UNSUPPORTED, "stacked rank must be a multiple of 8, at least r and at most 64");
    if (off < 0 || off % 8 != 0 || off + r > R)
        return fail(NB_ERR_INVALID_ARG, "slice [%lld, %lld) does not lie in the %lld stacked columns",
                    static_cast<long long>(off), static_cast<long long>(off + r), static_cast<long long>(R));
    return NB_OK;
}
}  // namespace

int nb_lora_down_stacked(void *t_stack, const void *inp, const void *a_stack, float scale, int64_t BT,
                         int64_t C, int64_t R, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, R);
    if (rc != NB_OK) return rc;
    if (R > 64) return fail(NB_ERR_UNSUPPORTED, "stacked rank must be at most 64");
    if (!t_stack || !inp || !a_stack) return fail(NB_ERR_INVALID_ARG, "t_stack, inp and a_stack must not be NULL");
    if (!aligned16(t_stack) || !aligned16(inp) || !aligned16(a_stack))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    GemmArgs a;
    memset(&a, 0, sizeof(a));  // t_stack = scale * inp . a_stack^T
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = a_stack; a.b_rows = R; a.b_cols = C;
    a.D = t_stack; a.d_rows = BT; a.d_cols = R; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(R); a.K = static_cast<int>(C);
    a.splits = 1;
    a.alpha = scale;
    return launch_gemm<FwdStoreNarrow>(*s, a, stream);
}

int nb_lora_linear_forward_stacked(void *out, const void *inp, const void *weight, const void *bias,
                                   const void *t_stack, const void *lora_b, int64_t BT, int64_t C,
                                   int64_t OC, int64_t r, int64_t R, int64_t off, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if ((rc = check_stack(r, R, off)) != NB_OK) return rc;
    if (!out || !inp || !weight || !t_stack || !lora_b)
        return fail(NB_ERR_INVALID_ARG, "out, inp, weight, t_stack and lora_b must not be NULL");
    if (!aligned16(out) || !aligned16(inp) || !aligned16(weight) || !aligned16(t_stack) || !aligned16(lora_b))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (BT == 0) return NB_OK;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    GemmArgs a;
    memset(&a, 0, sizeof(a));  // out = inp . W^T (+ bias) + t_slice . B^T: r extra columns of K
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = weight; a.b_rows = OC; a.b_cols = C;
    a.D = out; a.d_rows = BT; a.d_cols = OC; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(OC); a.K = static_cast<int>(C);
    a.bias = bias;
    a.splits = 1;
    a.A2 = static_cast<const uint16_t *>(t_stack) + off; a.a2_rows = BT; a.a2_cols = r; a.a2_ld = R;
    a.B2 = lora_b; a.b2_rows = OC; a.b2_cols = r;
    a.k2 = static_cast<int>(r);
    return launch_gemm_auto<FwdStore1, FwdStore2>(*s, a, stream);
}

int nb_lora_linear_backward_stacked(void *dinp, void *dlora_b, void *u_stack, const void *dout,
                                    const void *weight, const void *lora_a, const void *lora_b,
                                    const void *t_stack, float scale, int64_t BT, int64_t C, int64_t OC,
                                    int64_t r, int64_t R, int64_t off, int accumulate, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, OC);
    if (rc != NB_OK) return rc;
    if ((rc = check_stack(r, R, off)) != NB_OK) return rc;
    if (!u_stack || !dout || !lora_a || !lora_b)
        return fail(NB_ERR_INVALID_ARG, "u_stack, dout, lora_a and lora_b must not be NULL");
    if (dinp && !weight) return fail(NB_ERR_INVALID_ARG, "weight is required to compute dinp");
    if (dlora_b && !t_stack) return fail(NB_ERR_INVALID_ARG, "t_stack (from the forward calls) is required for dlora_b");
    if (!aligned16(dinp) || !aligned16(dlora_b) || !aligned16(u_stack) || !aligned16(dout) || !aligned16(weight) ||
        !aligned16(lora_a) || !aligned16(lora_b) || !aligned16(t_stack))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    if (BT == 0) {
        if (!accumulate && dlora_b) NB_CUDA(cudaMemsetAsync(dlora_b, 0, static_cast<size_t>(OC * r) * 4, stream));
        return NB_OK;
    }
    uint16_t *u_slice = static_cast<uint16_t *>(u_stack) + off;
    GemmArgs a;
    static const bool fused_udb = env_int("NB_LORA_FUSED", 1) != 0;
    if (fused_udb && dlora_b) {  // u_slice and dB from one pass over dout
        if ((rc = launch_lora_udb(*s, dout, lora_b, static_cast<const uint16_t *>(t_stack) + off, static_cast<uint64_t>(R),
                                  dlora_b, u_slice, static_cast<uint64_t>(R), scale, BT, OC, r, accumulate,
                                  stream)) != NB_OK)
            return rc;
        dlora_b = nullptr;
    } else {
        memset(&a, 0, sizeof(a));  // u_slice = scale * dout . B
        a.A = dout; a.a_rows = BT; a.a_cols = OC;
        a.B = lora_b; a.b_rows = OC; a.b_cols = r;
        a.D = u_slice; a.d_rows = BT; a.d_cols = r; a.d_dtype = 0; a.d_ld = R;
        a.M = static_cast<int>(BT); a.N = static_cast<int>(r); a.K = static_cast<int>(OC);
        a.splits = 1;
        a.alpha = scale;
        if ((rc = launch_gemm<DgradStoreNarrow>(*s, a, stream)) != NB_OK) return rc;
    }
    // dB right after u: both stream dout, and what the first pass brought into L2 serves the second
    if (dlora_b)  // dB [OC, r] (+)= dout^T . t_slice
        if ((rc = run_wgrad_f32(*s, dout, static_cast<const uint16_t *>(t_stack) + off, dlora_b, nullptr, BT, OC, r,
                                accumulate, stream, static_cast<uint64_t>(R))) != NB_OK)
            return rc;
    if (dinp) {  // dinp = dout . W + u_slice . A
        memset(&a, 0, sizeof(a));
        a.A = dout; a.a_rows = BT; a.a_cols = OC;
        a.B = weight; a.b_rows = OC; a.b_cols = C;
        a.D = dinp; a.d_rows = BT; a.d_cols = C; a.d_dtype = 0;
        a.M = static_cast<int>(BT); a.N = static_cast<int>(C); a.K = static_cast<int>(OC);
        a.splits = 1;
        a.A2 = u_slice; a.a2_rows = BT; a.a2_cols = r; a.a2_ld = R;
        a.B2 = lora_a; a.b2_rows = r; a.b2_cols = C;
        a.k2 = static_cast<int>(r);
        if ((rc = launch_gemm_auto<DgradStore1, DgradStore2>(*s, a, stream)) != NB_OK) return rc;
    }
    return NB_OK;
}

int nb_lora_da_stacked(void *da_stack, const void *u_stack, const void *inp, int64_t BT, int64_t C, int64_t R,
                       int accumulate, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = check_dims(BT, C, R);
    if (rc != NB_OK) return rc;
    if (R > 64) return fail(NB_ERR_UNSUPPORTED, "stacked rank must be at most 64");
    if (!da_stack || !u_stack || !inp) return fail(NB_ERR_INVALID_ARG, "da_stack, u_stack and inp must not be NULL");
    if (!aligned16(da_stack) || !aligned16(u_stack) || !aligned16(inp))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    if ((rc = get_state(&s)) != NB_OK) return rc;
    if (BT == 0) {
        if (!accumulate) NB_CUDA(cudaMemsetAsync(da_stack, 0, static_cast<size_t>(R * C) * 4, stream));
        return NB_OK;
    }
    return run_wgrad_f32(*s, u_stack, inp, da_stack, nullptr, BT, R, C, accumulate, stream);  // dA (+)= u^T . inp
}

int nb_cast_f32_to_bf16(void *dst, const void *src, int64_t n, void *stream_)
{
    if (n < 0) return fail(NB_ERR_INVALID_ARG, "negative size");
    if (n == 0) return NB_OK;
    if (!dst || !src) return fail(NB_ERR_INVALID_ARG, "dst and src must not be NULL");
    if (!aligned16(dst) || !aligned16(src))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    cast_f32_bf16_kernel<<<elementwise_grid(*s, n / 8 + 1), 256, 0, static_cast<cudaStream_t>(stream_)>>>(
        static_cast<__nv_bfloat16 *>(dst), static_cast<const float *>(src), n);
    NB_CUDA(cudaGetLastError());
    ++g_launches;
    return NB_OK;
}

int nb_workspace_reserve(int64_t bytes)
{
    if (bytes < 0) return fail(NB_ERR_INVALID_ARG, "negative size");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    return ensure_workspace(*s, static_cast<size_t>(bytes));
}

int nb_release(void)
{
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(NB_ERR_UNSUPPORTED, "device index %d", dev);
    DeviceState &s = g_dev[dev];
    if (!s.init) return NB_OK;
    NB_CUDA(cudaDeviceSynchronize());
    if (s.workspace) NB_CUDA(cudaFree(s.workspace));
    if (s.status) NB_CUDA(cudaFree(s.status));
    s = DeviceState();
    return NB_OK;
}

int nb_check_status(void)
{
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    NB_CUDA(cudaDeviceSynchronize());
    int host[4] = {0, 0, 0, 0};
    NB_CUDA(cudaMemcpy(host, s->status, sizeof(host), cudaMemcpyDeviceToHost));
    if (host[0] == 0) return NB_OK;
    NB_CUDA(cudaMemset(s->status, 0, 64));
    if (host[0] == kStatusTimeout)
        return fail(NB_ERR_TIMEOUT, "a bounded device wait expired (wait id %d, block %d)", host[1],
                    host[2]);
    return fail(NB_ERR_CUDA, "kernel reported internal error %d (block %d)", host[0], host[2]);
}

int64_t nb_kernel_launches(void) { return g_launches.load(); }

int nb_debug_split_plan(int64_t M, int64_t N, int64_t K, int slots, int tile_m, int *out)
{
    if (!out || M <= 0 || N <= 0 || K <= 0 || slots <= 0 || (tile_m != 128 && tile_m != 256))
        return fail(NB_ERR_INVALID_ARG, "bad argument");
    const int tiles_m = static_cast<int>((M + tile_m - 1) / tile_m);
    const int tiles_n = static_cast<int>((N + 255) / 256);
    const int kblocks = static_cast<int>((K + kBlockK - 1) / kBlockK);
    int splits = choose_splits(tiles_m * tiles_n, kblocks, slots);
    const int kps = (kblocks + splits - 1) / splits;  // as launch_gemm derives it
    splits = (kblocks + kps - 1) / kps;
    out[0] = tiles_m;
    out[1] = tiles_n;
    out[2] = splits;
    out[3] = kps;
    out[4] = kblocks;
    return NB_OK;
}

int nb_debug_layer_bwd_plan(int64_t BT, int64_t C, int64_t OC, int pairs, int gelu_grad, int *out,
                            int64_t cap)
{
    if (!out || cap < 8 || BT <= 0 || C <= 0 || OC <= 0) return -fail(NB_ERR_INVALID_ARG, "bad argument");
    LayerBwdParams p;
    const int rc = plan_layer_bwd(p, BT, C, OC, pairs, gelu_grad != 0);
    if (rc != NB_OK) return -rc;
    out[0] = p.d_tiles_m; out[1] = p.d_tiles_n; out[2] = p.d_kblocks;
    out[3] = p.w_tiles_m; out[4] = p.w_tiles_n; out[5] = p.w_kblocks;
    out[6] = p.w_kbc; out[7] = p.d_rounds + p.w_rounds;
    int64_t n = 8;
    int records = 0;
    for (int q = 0; q < pairs; ++q) {
        LbIter it(p, q);
        LbUnit u;
        while (it.next(p, u)) {
            if (n + 6 > cap) return -fail(NB_ERR_INVALID_ARG, "output buffer too small");
            out[n++] = q; out[n++] = u.is_w; out[n++] = u.m_blk; out[n++] = u.n_blk;
            out[n++] = u.kb0; out[n++] = u.kb1;
            ++records;
        }
    }
    return records;
}

int nb_debug_gemm_timeout(void *out, const void *inp, const void *weight, int64_t limit_us)
{
    if (!out || !inp || !weight) return fail(NB_ERR_INVALID_ARG, "out, inp and weight must not be NULL");
    if (!aligned16(out) || !aligned16(inp) || !aligned16(weight))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (limit_us < 100 || limit_us > 1000000)
        return fail(NB_ERR_INVALID_ARG, "limit_us must be within [100, 1000000]");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    const int64_t BT = 128, C = 256, OC = 256;  // one tile, one CTA, four k-blocks
    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.A = inp; a.a_rows = BT; a.a_cols = C;
    a.B = weight; a.b_rows = OC; a.b_cols = C;
    a.D = out; a.d_rows = BT; a.d_cols = OC; a.d_dtype = 0;
    a.M = static_cast<int>(BT); a.N = static_cast<int>(OC); a.K = static_cast<int>(C);
    a.splits = 1;
    a.debug_stop_kb = 2;  // the first two k-blocks are loaded, the third never is
    a.debug_timeout_ns = static_cast<unsigned long long>(limit_us) * 1000ull;
    return launch_gemm<FwdStore1>(*s, a, g_stream);
}

int nb_debug_wait_timeout(int64_t limit_us)
{
    if (limit_us < 1 || limit_us > 1000000)
        return fail(NB_ERR_INVALID_ARG, "limit_us must be within [1, 1000000]");
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceState *s;
    int rc = get_state(&s);
    if (rc != NB_OK) return rc;
    wait_timeout_kernel<<<1, 32, 0, g_stream>>>(s->status, static_cast<unsigned long long>(limit_us) * 1000ull);
    NB_CUDA(cudaGetLastError());
    ++g_launches;
    return NB_OK;
}

// ----------------------------------------------------------------------------- no allocation
// Scratch for nb_gelu_dbias_noalloc: part of the library image, so it exists on every device that
// loads the library without anyone allocating it. In host code `nb_noalloc_scratch` is only a
// handle for the runtime, not a device address: the address a kernel can use comes from
// cudaGetSymbolAddress, once per device.
}  // extern "C" (the array and its bookkeeping have internal linkage)

namespace {
static __device__ __align__(256) unsigned char nb_noalloc_scratch[NB_NOALLOC_MAX_ELEMS * 2];
void *g_noalloc_ptr[kMaxDevices] = {};
int g_noalloc_sms[kMaxDevices] = {};
}  // namespace

extern "C" {

int nb_gelu_dbias_noalloc(void *dbias, const void *dout, const void *pre_act, int64_t BT, int64_t OC,
                          int accumulate, void *stream_)
{
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!dbias || !dout || !pre_act)
        return fail(NB_ERR_INVALID_ARG, "dbias, dout and pre_act must not be NULL");
    if (BT < 0 || OC <= 0) return fail(NB_ERR_INVALID_ARG, "negative or zero dimension");
    if (OC % 8 != 0) return fail(NB_ERR_UNSUPPORTED, "OC must be a multiple of 8");
    if (!aligned16(dbias) || !aligned16(dout) || !aligned16(pre_act))
        return fail(NB_ERR_INVALID_ARG, "tensor pointers must be 16-byte aligned");
    if (BT >= (1ll << 31) || OC >= (1ll << 31) || BT * OC > static_cast<int64_t>(NB_NOALLOC_MAX_ELEMS))
        return fail(NB_ERR_UNSUPPORTED,
                    "BT*OC = %lld exceeds the built-in scratch of %d elements (NB_NOALLOC_MAX_ELEMS); "
                    "use nb_linear_backward_ex, which allocates a workspace",
                    static_cast<long long>(BT * OC), NB_NOALLOC_MAX_ELEMS);

    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    NB_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(NB_ERR_UNSUPPORTED, "device index %d", dev);
    if (!g_noalloc_ptr[dev]) {  // set-up, once per device, with that device current
        void *ptr = nullptr;
        NB_CUDA(cudaGetSymbolAddress(&ptr, nb_noalloc_scratch));
        int sms = 0;
        NB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (!ptr || sms <= 0) return fail(NB_ERR_CUDA, "could not resolve the built-in scratch array");
        g_noalloc_sms[dev] = sms;
        g_noalloc_ptr[dev] = ptr;
    }
    DeviceState local;  // only the SM count is read by the launch helpers below
    local.num_sms = g_noalloc_sms[dev];
    void *dz = g_noalloc_ptr[dev];

    if (BT > 0) {
        // dz = dout * gelu'(pre_act) overwrites the first BT*OC elements of the scratch
        const long long nvec = BT * OC / 8;
        gelu_backward_kernel<<<elementwise_grid(local, nvec), 256, 0, stream>>>(
            static_cast<uint4 *>(dz), static_cast<const uint4 *>(dout),
            static_cast<const uint4 *>(pre_act), nvec);
        NB_CUDA(cudaGetLastError());
        ++g_launches;
    }
    return launch_dbias(local, static_cast<float *>(dbias), dz, BT, OC, accumulate, stream);
}

}  // extern "C"
