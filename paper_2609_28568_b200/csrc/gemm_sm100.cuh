// Persistent, warp-specialised bf16 GEMM for sm_100a:  D[M,N] = sum_k A[m,k] * B[n,k]
//
//   warp 0      TMA producer: fills a ring of shared-memory stages (A tile 128x64, B tile Nx64)
//   warp 1      MMA issuer: one thread issues tcgen05.mma (128 x BLOCK_N x 16) into TMEM;
//               two accumulators so the next tile's main loop overlaps this tile's epilogue
//   warps 2..9  epilogue: tcgen05.ld -> fp32 registers -> bias / activation -> swizzled
//               shared staging -> TMA store (or TMA reduce-add for split-K fp32 results);
//               two warps per TMEM lane quarter, each taking half of a step's columns
//
//   warps 10..13 (wgrad with fused bias gradient only) sum the A tiles over k from shared memory
//
// Operand layouts. "K-major" means the reduction index is contiguous in global memory (forward:
// both operands). "MN-major" means the output index is contiguous (dgrad reads the weight as
// B[n=c, k=o] from W[o, c]; wgrad reads dz and inp as A[m=o, k=row], B[n=c, k=row]); those tiles
// are fetched as 64(k) x 64(mn) boxes and described to the tensor core as MN-major, so no
// transpose is ever materialised.
//
// CTA pairs (CG = 2). Two CTAs of a cluster share one 256-row tile: each loads its own 128 rows of
// A and its own half of B's N extent, the leader CTA issues tcgen05.mma.cta_group::2 reading both
// CTAs' shared memory, and each CTA's TMEM receives its 128 rows of the result. Per SM this halves
// the B traffic and the stage size, which buys a deeper ring. Both CTAs' loads are counted on the
// leader's "full" barrier; MMA completion is multicast to both CTAs' "empty" / "tmem_full" barriers;
// both CTAs' epilogues arrive on the leader's "tmem_empty" barrier.
//
// Every wait on an mbarrier is bounded in time; on expiry the kernel records the event in the
// status word, stops issuing work, and all threads leave through the common exit.
#pragma once
#include "ptx.cuh"

namespace nb {

constexpr int kBlockM = 128;
constexpr int kBlockK = 64;   // bf16 elements per stage along K = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kNumThreads = 320;  // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int kEpiThreads = 256;
constexpr int kEpiWarps = 8;
constexpr uint32_t kStgBytes = 16384;  // one staging buffer: 128 rows x 128 bytes
constexpr int kStatusTimeout = 4;      // == NB_ERR_TIMEOUT
constexpr int kStatusBadSmem = 5;

enum EpiMode : int {
    kEpiStore = 0,        // D(bf16) = acc (+ bias)
    kEpiGelu = 1,         // E(bf16) = z = acc + bias ; D(bf16) = gelu(z)
    kEpiSwiglu = 2,       // E = z (gate | up planes) ; D[:, j] = silu(gate_j) * up_j
    kEpiMulGeluGrad = 3,  // D(bf16) = acc * gelu'(E)    (E is read)
    kEpiF32 = 4,          // D(fp32) = acc, stored or reduce-added
    kEpiStoreStats = 5    // kEpiStore, plus per-row (max, sum of exp) of the stored values over the
                          // tile's columns below v_real: the softmax statistics of the head's logits
};

struct GemmParams {
    int M, N, K;
    int tiles_m, tiles_n;
    int splits;             // split-K factor (kEpiF32), else 1
    int kblocks_per_split;  // 64-wide k blocks handled by one unit
    int kblocks;            // ceil(K / 64)
    int kblocks_ext;        // extra k-blocks read through the second pair of tensor maps (A2, B2):
                            // D += A2 . B2^T, the low-rank adapter term; only with splits == 1
    float alpha;            // kEpiStore family: D = alpha * acc + bias
    int group_m;            // rasterisation: m-tiles per group
    int swiglu_h;           // kEpiSwiglu: H (gate rows [0,H), up rows [H,2H) of B)
    int reduce;             // kEpiF32: 1 reduce-add into D, 0 overwrite
    const __nv_bfloat16 *bias;  // [N] or nullptr
    float *dbias;               // wgrad with fused bias gradient: dbias[m] += sum_k A[m,k]
    float2 *stats;              // kEpiStoreStats: [M, stats_ld] partial (max, sum exp) per row
    int stats_ld;               //   two entries per column tile (one per column half of a step)
    int v_real;                 //   columns >= v_real take no part in the statistics
    int *status;
    unsigned long long timeout_ns;
    int debug_stop_kb;  // self-test of the time-out exit: the producer stops before this k-block
                        // (counted over the CTA's whole run); negative in normal use
};

template <int CG_, int BLOCK_N_, int STAGES_, int NSTG_, bool A_MN_, bool B_MN_, int EPI_,
          bool DBIAS_ = false>
struct GemmCfg {
    // DBIAS: four extra warps sum the A tiles (dz^T in wgrad) over k while the tensor core reads
    // them, so the bias gradient needs no pass of its own over dz
    static constexpr bool DBIAS = DBIAS_;
    static constexpr int THREADS = kNumThreads + (DBIAS_ ? 128 : 0);
    static constexpr int CG = CG_;              // CTAs per tile: 1, or 2 (a cta_group::2 pair)
    static constexpr int TILE_M = kBlockM * CG_;
    static constexpr int BLOCK_N = BLOCK_N_;
    static constexpr int STAGES = STAGES_;
    static constexpr int NSTG = NSTG_;
    static constexpr bool A_MN = A_MN_;
    static constexpr bool B_MN = B_MN_;
    static constexpr int EPI = EPI_;
    static constexpr uint32_t A_BYTES = kBlockM * kBlockK * 2;
    static constexpr int B_ROWS = BLOCK_N / CG_;  // rows of B's N extent held by one CTA
    static constexpr uint32_t B_BYTES = B_ROWS * kBlockK * 2;
    static constexpr uint32_t OFF_A = 0;
    static constexpr uint32_t OFF_B = STAGES * A_BYTES;
    static constexpr uint32_t OFF_STG = STAGES * (A_BYTES + B_BYTES);
    // kEpiMulGeluGrad: a ring of NAUX buffers receives the pre-activation tiles, apart from the
    // staging buffers, so the prefetch never waits for a store to drain
    static constexpr int NAUX = (EPI_ == kEpiMulGeluGrad) ? 4 : 0;
    static constexpr uint32_t OFF_AUX = OFF_STG + NSTG * kStgBytes;
    static constexpr uint32_t OFF_BIAS = OFF_AUX + NAUX * kStgBytes;
    // Warp-private epilogue (bf16 results of full-width tiles): every epilogue warp stages and
    // stores its own 32-row boxes, no barrier joins the warps. The bias then lives in two buffers
    // (by tile parity) and each warp has its own pair of pre-activation barriers.
    static constexpr bool WARP_EPI = BLOCK_N_ == 256 &&
                                     (EPI_ == kEpiStore || EPI_ == kEpiStoreStats || EPI_ == kEpiGelu ||
                                      EPI_ == kEpiMulGeluGrad || EPI_ == kEpiF32);
    // boxes of staging per epilogue warp: one per stored plane; fp32 results alternate between two
    static constexpr int WARP_BOXES = (EPI_ == kEpiF32) ? 2 : (EPI_ == kEpiGelu) ? 2 : 1;
    static constexpr int OUT_BOX_ROWS = WARP_EPI ? 32 : kBlockM;
    static constexpr uint32_t BIAS_BYTES = (WARP_EPI ? 2 : 1) * BLOCK_N * 4;
    static constexpr uint32_t OFF_BAR = OFF_BIAS + BIAS_BYTES;
    static constexpr uint32_t BAR_BYTES = WARP_EPI ? 512 : 256;
    static constexpr uint32_t SMEM_BYTES = OFF_BAR + BAR_BYTES;
    static constexpr uint32_t TMEM_COLS = (2 * BLOCK_N <= 32) ? 32
                                          : (2 * BLOCK_N <= 64) ? 64
                                          : (2 * BLOCK_N <= 128) ? 128
                                          : (2 * BLOCK_N <= 256) ? 256 : 512;
    // staging buffers used by one epilogue step, and steps per tile
    static constexpr int BUFS_PER_STEP = (EPI == kEpiGelu) ? 2 : (EPI == kEpiSwiglu) ? 3 : 1;
    static constexpr int SLOTS = NSTG / BUFS_PER_STEP;
    static constexpr int STEPS = (EPI == kEpiF32) ? BLOCK_N / 32
                                 : (EPI == kEpiSwiglu) ? BLOCK_N / 128 : BLOCK_N / 64;
    static_assert(CG_ == 1 || CG_ == 2, "CTAs per tile");
    static_assert(BLOCK_N % (64 * CG_) == 0 && BLOCK_N >= 64 && BLOCK_N <= 256, "BLOCK_N");
    static_assert(2 * BLOCK_N <= 512, "two accumulators must fit in TMEM");
    static_assert(NSTG % BUFS_PER_STEP == 0 && SLOTS >= 1, "staging ring");
    static_assert(EPI != kEpiMulGeluGrad || SLOTS >= 2, "staging ring");
    static_assert(EPI != kEpiSwiglu || BLOCK_N == 256, "SwiGLU tiles pair 128 gate + 128 up cols");
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(!WARP_EPI || NSTG * kStgBytes >= 8u * WARP_BOXES * 4096u, "staging boxes per warp");
    static_assert(!WARP_EPI || EPI_ != kEpiMulGeluGrad || NAUX * kStgBytes >= 8u * 2u * 4096u,
                  "two pre-activation boxes per warp");
    static_assert(!DBIAS_ || (A_MN_ && EPI_ == kEpiF32), "the fused bias gradient belongs to wgrad");
};

// barrier slots inside the 256-byte barrier region (8 bytes each)
//   [0, S)      full[s]     TMA -> MMA
//   [S, 2S)     empty[s]    MMA -> TMA
//   2S, 2S+1    tmem_full   MMA -> epilogue
//   2S+2, 2S+3  tmem_empty  epilogue -> MMA
//   byte 256 + 8 (2 w + b): kEpiMulGeluGrad, pre-activation box b (0 / 1) of epilogue warp w has landed
//   byte 240: TMEM base address, 244: abort flag (any role), 248: epilogue abort flag

struct WaitCtx {
    uint32_t abort_addr;
    int *status;
    unsigned long long timeout_ns;
};

__device__ __forceinline__ bool wait_barrier(const WaitCtx &w, uint32_t bar, uint32_t parity,
                                             int where)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t it = 0;
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((++it & 15u) == 0) {
            if (ptx::ld_shared_u32_volatile(w.abort_addr) != 0) return false;
            if (ptx::globaltimer_ns() - t0 > w.timeout_ns) {
                ptx::st_shared_u32_volatile(w.abort_addr, 1);
                if (atomicCAS(w.status, 0, kStatusTimeout) == 0) {
                    w.status[1] = where;
                    w.status[2] = static_cast<int>(blockIdx.x);
                }
                return false;
            }
        }
    }
}

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes,
                                                   uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);         // start address
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;  // leading byte offset
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;  // stride byte offset
    d |= static_cast<uint64_t>(1) << 46;                         // descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                         // 128-byte swizzle
    return d;
}

__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool a_mn, bool b_mn)
{
    return (1u << 4)                               // accumulator fp32
           | (1u << 7) | (1u << 10)                // A, B bf16
           | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16)
           | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

__device__ __forceinline__ void decode_unit(const GemmParams &p, int u, int &m_blk, int &n_blk,
                                            int &split)
{
    const int tiles = p.tiles_m * p.tiles_n;
    split = u / tiles;
    const int t = u - split * tiles;
    const int per_group = p.group_m * p.tiles_n;
    const int g = t / per_group;
    const int r = t - g * per_group;
    const int first_m = g * p.group_m;
    const int gsz = min(p.group_m, p.tiles_m - first_m);
    m_blk = first_m + r % gsz;
    n_blk = r / gsz;
}

__device__ __forceinline__ float gelu_fwd(float z)
{
    const float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
    return 0.5f * z * (1.0f + ptx::tanh_approx(u));
}
__device__ __forceinline__ float gelu_bwd(float x)
{
    const float x2 = x * x;
    const float u = 0.7978845608028654f * (x + 0.044715f * x * x2);
    const float t = ptx::tanh_approx(u);
    const float du = 0.7978845608028654f * (1.0f + 3.0f * 0.044715f * x2);
    return 0.5f * (1.0f + t) + 0.5f * x * (1.0f - t * t) * du;
}
// The same two functions on pairs (packed fp32): tanh-GELU of z, and acc * gelu'(x).
__device__ __forceinline__ ptx::f2 gelu_fwd2(ptx::f2 z)
{
    const ptx::f2 c0 = ptx::make_f2(0.7978845608028654f, 0.7978845608028654f);
    const ptx::f2 c01 = ptx::make_f2(0.7978845608028654f * 0.044715f, 0.7978845608028654f * 0.044715f);
    const ptx::f2 half = ptx::make_f2(0.5f, 0.5f);
    const ptx::f2 z2 = ptx::mul2(z, z);
    const ptx::f2 u = ptx::mul2(z, ptx::fma2(z2, c01, c0));
    float u0, u1;
    ptx::split_f2(u, u0, u1);
    const ptx::f2 t = ptx::make_f2(ptx::tanh_approx(u0), ptx::tanh_approx(u1));
    const ptx::f2 hz = ptx::mul2(z, half);
    return ptx::fma2(hz, t, hz);
}
__device__ __forceinline__ ptx::f2 mul_gelu_bwd2(ptx::f2 acc, ptx::f2 x)
{
    const ptx::f2 c0 = ptx::make_f2(0.7978845608028654f, 0.7978845608028654f);
    const ptx::f2 c01 = ptx::make_f2(0.7978845608028654f * 0.044715f, 0.7978845608028654f * 0.044715f);
    const ptx::f2 c03 = ptx::make_f2(3.0f * 0.7978845608028654f * 0.044715f,
                                     3.0f * 0.7978845608028654f * 0.044715f);
    const ptx::f2 half = ptx::make_f2(0.5f, 0.5f);
    const ptx::f2 one = ptx::make_f2(1.0f, 1.0f);
    const ptx::f2 neg1 = ptx::make_f2(-1.0f, -1.0f);
    const ptx::f2 x2 = ptx::mul2(x, x);
    const ptx::f2 u = ptx::mul2(x, ptx::fma2(x2, c01, c0));
    float u0, u1;
    ptx::split_f2(u, u0, u1);
    const ptx::f2 t = ptx::make_f2(ptx::tanh_approx(u0), ptx::tanh_approx(u1));
    const ptx::f2 du = ptx::fma2(x2, c03, c0);                    // d/dx of the tanh argument
    const ptx::f2 a = ptx::fma2(t, half, half);                   // 0.5 (1 + t)
    const ptx::f2 omt2 = ptx::fma2(ptx::mul2(t, t), neg1, one);   // 1 - t^2
    const ptx::f2 b = ptx::mul2(ptx::mul2(x, half), du);          // 0.5 x du
    return ptx::mul2(acc, ptx::fma2(b, omt2, a));
}
__device__ __forceinline__ uint32_t pack_f2_bf16x2(ptx::f2 v)
{
    float lo, hi;
    ptx::split_f2(v, lo, hi);
    return ptx::pack_bf16x2(lo, hi);
}

__device__ __forceinline__ float silu_fwd(float g) { return __fdividef(g, 1.0f + __expf(-g)); }

__device__ __forceinline__ void atomicAdd_shared_f32(uint32_t addr, float v)
{
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

template <class Cfg>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmE,
            const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
            const GemmParams p)
{
    constexpr int BLOCK_N = Cfg::BLOCK_N;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int EPI = Cfg::EPI;
    constexpr int CG = Cfg::CG;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem = ptx::smem_u32(smem_raw);
    const int warp = static_cast<int>(threadIdx.x >> 5);
    const int lane = static_cast<int>(threadIdx.x & 31);
    // position in the CTA pair; pairs are consecutive blocks along x, so this equals %cluster_ctarank
    // (taken from blockIdx so the compiler can see that it is uniform across the block)
    const uint32_t rank = (CG == 2) ? (blockIdx.x & 1u) : 0u;
    const int first_unit = static_cast<int>(blockIdx.x) / CG;       // units are shared by the pair
    const int unit_stride = static_cast<int>(gridDim.x) / CG;

    // swizzled tiles need 1024-byte alignment; if the base is off, record it and do no work
    const bool smem_ok = (smem & 1023u) == 0;
    if (!smem_ok && threadIdx.x == 0 && atomicCAS(p.status, 0, kStatusBadSmem) == 0)
        p.status[2] = static_cast<int>(blockIdx.x);

    const uint32_t bar0 = smem + Cfg::OFF_BAR;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
    // DBIAS only: a stage is handed MMA -> reducers (empty_bar) -> producer (free_bar)
    auto free_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 8 + s); };
    const uint32_t tmem_slot = bar0 + 240;
    const uint32_t abort_addr = bar0 + 244;
    const uint32_t epi_abort_addr = bar0 + 248;
    static_assert(8 * (3 * STAGES + 8) <= 240, "barrier region");

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);  // MMAs that read the stage are done
            ptx::mbar_init(free_bar(s), 4);   // DBIAS: the four reducer warps have read it too
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), kEpiWarps * CG);  // one arrive per epilogue warp of the tile
        }
        if (Cfg::WARP_EPI && EPI == kEpiMulGeluGrad)  // two per epilogue warp, above the common slots
            for (int b = 0; b < 2 * kEpiWarps; ++b) ptx::mbar_init(bar0 + 256u + 8u * b, 1);
        ptx::st_shared_u32_volatile(abort_addr, 0);
        ptx::st_shared_u32_volatile(epi_abort_addr, 0);
        ptx::fence_barrier_init();
        ptx::prefetch_tmap(&tmA);
        ptx::prefetch_tmap(&tmB);
        ptx::prefetch_tmap(&tmD);
        if (EPI == kEpiGelu || EPI == kEpiSwiglu || EPI == kEpiMulGeluGrad) ptx::prefetch_tmap(&tmE);
    }
    if (warp == 1) {
        ptx::tmem_alloc<CG>(tmem_slot, Cfg::TMEM_COLS);
        ptx::tmem_relinquish<CG>();
    }
    ptx::tc_fence_before();
    if (CG == 2) ptx::cluster_sync();  // the peer's barriers are initialised before anyone signals them
    else __syncthreads();
    ptx::tc_fence_after();
    // Everything above touched only this CTA's shared memory and TMEM, so it may run while the
    // previous kernel of the stream is still draining; global memory is not read or written before
    // that kernel has completed.
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const uint32_t tmem_base = ptx::ld_shared_u32_volatile(tmem_slot);

    const WaitCtx wctx{abort_addr, p.status, p.timeout_ns};
    // The epilogue waits for a whole unit where the issuer waits for one stage: with twice the limit
    // the wait that is closest to the cause of a stall is the one that expires and gets reported.
    const WaitCtx wctx_epi{abort_addr, p.status, 2 * p.timeout_ns};
    const int num_units = p.tiles_m * p.tiles_n * p.splits;

    // one tile load, counted on the leader CTA's barrier
    auto load = [&](uint32_t dst, const CUtensorMap *m, uint32_t bar, int x, int y) {
        if (CG == 2) ptx::tma_load_2d_pair(dst, m, bar, x, y);
        else ptx::tma_load_2d(dst, m, bar, x, y);
    };

    if (!smem_ok) {
        // fall through to the common exit
    } else if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (every CTA)
        // One elected lane; the election sits in a warp-uniform branch, the form in which the
        // compiler hands coordinates to the TMA unit reliably (a thread-index test did not).
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int issued = 0;  // k-blocks loaded so far
            for (int u = first_unit; u < num_units && ok; u += unit_stride) {
                int m_blk, n_blk, split;
                decode_unit(p, u, m_blk, n_blk, split);
                const int kb0 = split * p.kblocks_per_split;
                const int kb1 = min(kb0 + p.kblocks_per_split, p.kblocks);
                const int m0 = m_blk * Cfg::TILE_M + static_cast<int>(rank) * kBlockM;
                const int kb_end = kb1 + p.kblocks_ext;  // the adapter term's k-blocks come last
                for (int kb = kb0; kb < kb_end; ++kb) {
                    // self-test only: leave the rest unloaded, so that the issuer's wait for this
                    // stage runs out and the kernel leaves through its time-out exit
                    if (issued++ == p.debug_stop_kb) {
                        ok = false;
                        break;
                    }
                    const bool ext = kb >= kb1;
                    const CUtensorMap *mapA = ext ? &tmA2 : &tmA;
                    const CUtensorMap *mapB = ext ? &tmB2 : &tmB;
                    ok = wait_barrier(wctx, Cfg::DBIAS ? free_bar(stage) : empty_bar(stage), phase ^ 1u,
                                      100 + stage);
                    if (!ok) break;
                    // the leader's barrier collects the bytes of both CTAs of a pair
                    const uint32_t fb = (CG == 2) ? ptx::mapa(full_bar(stage), 0) : full_bar(stage);
                    if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), CG * (Cfg::A_BYTES + Cfg::B_BYTES));
                    const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES;
                    const uint32_t sb = smem + Cfg::OFF_B + stage * Cfg::B_BYTES;
                    const int k0 = (ext ? kb - kb1 : kb) * kBlockK;
                    if (Cfg::A_MN) {  // tensor [K rows, M cols]: boxes of 64(m) x 64(k)
#pragma unroll
                        for (int j = 0; j < kBlockM / 64; ++j)
                            load(sa + j * 8192u, mapA, fb, m0 + j * 64, k0);
                    } else {          // tensor [M rows, K cols]: boxes of 64(k) x 64(m)
#pragma unroll
                        for (int j = 0; j < kBlockM / 64; ++j)
                            load(sa + j * 8192u, mapA, fb, k0, m0 + j * 64);
                    }
                    // this CTA's share of B's N extent: all of it, or its half of the pair's tile
                    if (Cfg::B_MN) {
                        const int n0 = n_blk * BLOCK_N + static_cast<int>(rank) * Cfg::B_ROWS;
#pragma unroll
                        for (int j = 0; j < Cfg::B_ROWS / 64; ++j)
                            load(sb + j * 8192u, mapB, fb, n0 + j * 64, k0);
                    } else if (EPI == kEpiSwiglu) {  // 128 gate rows, then the matching 128 up rows
                        const int n0 = n_blk * 128;
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            if (CG == 1 || rank == 0)
                                load(sb + j * 8192u, mapB, fb, k0, n0 + j * 64);
                            if (CG == 1 || rank == 1)
                                load(sb + (CG == 1 ? 16384u : 0u) + j * 8192u, mapB, fb, k0,
                                     p.swiglu_h + n0 + j * 64);
                        }
                    } else {                          // boxes of 64(k) x 64(n)
                        const int n0 = n_blk * BLOCK_N + static_cast<int>(rank) * Cfg::B_ROWS;
#pragma unroll
                        for (int j = 0; j < Cfg::B_ROWS / 64; ++j)
                            load(sb + j * 8192u, mapB, fb, k0, n0 + j * 64);
                    }
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0 && ptx::elect_one()) {
            constexpr uint32_t idesc = make_idesc(Cfg::TILE_M, BLOCK_N, Cfg::A_MN, Cfg::B_MN);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int u = first_unit; u < num_units && ok; u += unit_stride) {
                int m_blk, n_blk, split;
                decode_unit(p, u, m_blk, n_blk, split);
                const int kb0 = split * p.kblocks_per_split;
                const int kb1 = min(kb0 + p.kblocks_per_split, p.kblocks);
                ok = wait_barrier(wctx, tempty_bar(acc), acc_phase ^ 1u, 200 + acc);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BLOCK_N);
                const int kb_end = kb1 + p.kblocks_ext;
                for (int kb = kb0; kb < kb_end; ++kb) {
                    ok = wait_barrier(wctx, full_bar(stage), phase, 300 + stage);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES;
                    const uint32_t sb = smem + Cfg::OFF_B + stage * Cfg::B_BYTES;
                    // K-major: 8-row groups 1024 B apart, 16 k = 32 B inside the swizzle row.
                    // MN-major: 64-wide chunks 8192 B apart, 8-k groups 1024 B apart, 16 k = 2048 B.
                    const uint64_t adesc = Cfg::A_MN ? make_smem_desc(sa, 8192, 1024)
                                                     : make_smem_desc(sa, 16, 1024);
                    const uint64_t bdesc = Cfg::B_MN ? make_smem_desc(sb, 8192, 1024)
                                                     : make_smem_desc(sb, 16, 1024);
                    constexpr uint32_t a_step = Cfg::A_MN ? (2048u >> 4) : (32u >> 4);
                    constexpr uint32_t b_step = Cfg::B_MN ? (2048u >> 4) : (32u >> 4);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        ptx::umma_bf16<CG>(d_tmem, adesc + static_cast<uint64_t>(k * a_step),
                                       bdesc + static_cast<uint64_t>(k * b_step), idesc,
                                       (kb > kb0 || k > 0) ? 1u : 0u);
                    }
                    ptx::umma_commit<CG>(empty_bar(stage));  // stage may be refilled once these finish
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::umma_commit<CG>(tfull_bar(acc));  // accumulator complete
                if (++acc == 2) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
        }
    } else if (Cfg::DBIAS && warp >= 10) {
        // ------------------------------------------------------------ bias-gradient reducers (warps 10..13)
        // They read a stage after the tensor core has, and only then is it handed back to the
        // producer. A tile of a stage (MN-major): two boxes of 64 k-rows x 128 bytes (64 m values), swizzled.
        // Thread t sums chunk (t & 15) (8 consecutive m) over k rows (t >> 4) + 8 i. Only the units
        // of the first n-tile do the arithmetic; every unit takes part in the stage hand-shake.
        const int rt = static_cast<int>(threadIdx.x) - 320;  // 0..127
        const int cc = rt & 15;
        const int kbase = rt >> 4;
        const uint32_t part_s = smem + Cfg::OFF_BIAS;  // 128 floats, unused by the fp32 epilogue
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        if (rt < kBlockM) ptx::st_shared_f32(part_s + 4u * rt, 0.0f);
        ptx::named_bar_sync(2, 128);
        for (int u = first_unit; u < num_units; u += unit_stride) {
            int m_blk, n_blk, split;
            decode_unit(p, u, m_blk, n_blk, split);
            const int kb0 = split * p.kblocks_per_split;
            const int kb1 = min(kb0 + p.kblocks_per_split, p.kblocks);
            const bool mine = (n_blk == 0) && p.dbias != nullptr;
            float sum[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) sum[k] = 0.0f;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (ok) {
                    // wait until the tensor core is done with the stage: its completion is multicast
                    // to both CTAs of a pair, so no CTA has to watch the other's barriers, and the
                    // tile is still intact because the producer waits for the reducers
                    bool w = true;
                    if (lane == 0) w = wait_barrier(wctx, empty_bar(stage), phase, 600 + stage);
                    ok = __shfl_sync(0xffffffffu, w ? 1 : 0, 0) != 0;
                }
                if (ok && mine) {
                    const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES +
                                        static_cast<uint32_t>(cc >> 3) * 8192u;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t kr = static_cast<uint32_t>(kbase + 8 * i);
                        uint32_t x[4];
                        ptx::ld_shared_v4(sa + kr * 128u + (((cc & 7u) ^ (kr & 7u)) << 4), x[0], x[1], x[2], x[3]);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            sum[2 * k] += ptx::bf16_lo(x[k]);
                            sum[2 * k + 1] += ptx::bf16_hi(x[k]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(free_bar(stage));  // this warp is done with the stage
                if (++stage == STAGES) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (mine) {  // uniform across the four warps: same unit, same parameters
#pragma unroll
                for (int k = 0; k < 8; ++k) atomicAdd_shared_f32(part_s + 4u * (cc * 8 + k), sum[k]);
                ptx::named_bar_sync(2, 128);
                const int m = m_blk * Cfg::TILE_M + static_cast<int>(rank) * kBlockM + rt;
                if (ok && rt < kBlockM && m < p.M) atomicAdd(p.dbias + m, ptx::ld_shared_f32(part_s + 4u * rt));
                if (rt < kBlockM) ptx::st_shared_f32(part_s + 4u * rt, 0.0f);
                ptx::named_bar_sync(2, 128);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        // Warp w may read TMEM lanes 32*(w%4)..+31, i.e. rows q*32..q*32+31 of the tile. Two warps
        // share each lane quarter and split every step's columns in halves (hf = 0 / 1).
        const int q = warp & 3;
        const int hf = (warp - 2) >> 2;
        const int row = q * 32 + lane;
      if constexpr (Cfg::WARP_EPI) {
        // ------------------------------------------------------------ epilogue, warp by warp
        // A warp owns 32 rows (its TMEM lane quarter) x 128 columns (its half) of the tile. It issues
        // the TMEM loads of all its columns at once, then, 32 columns at a time, applies the
        // epilogue, stages 32 x 64 boxes in its own 4 KB buffers and stores them with its own TMA
        // copies. No barrier joins the warps: while one waits for TMEM, a proxy fence or a store,
        // the others compute.
        const int ew = warp - 2;                  // 0..7
        constexpr uint32_t kBoxBytes = 32 * 128;  // 32 rows x 64 bf16, 128-byte swizzled
        constexpr uint32_t NBUF = Cfg::WARP_BOXES;  // kEpiGelu: activated + pre-activation; kEpiF32: a ring of two
        const uint32_t stg = smem + Cfg::OFF_STG + static_cast<uint32_t>(ew) * NBUF * kBoxBytes;
        const uint32_t aux0 = smem + Cfg::OFF_AUX + static_cast<uint32_t>(ew) * 2u * kBoxBytes;
        const uint32_t lane_off = static_cast<uint32_t>(lane) * 128u;
        const uint32_t sw = static_cast<uint32_t>(lane & 7);
        auto chunk_pos = [&](int chunk) { return lane_off + ((static_cast<uint32_t>(chunk) ^ sw) << 4); };
        auto waux_bar = [&](uint32_t b) { return bar0 + 256u + 8u * (static_cast<uint32_t>(ew) * 2u + b); };
        const bool has_bias = (EPI == kEpiStore || EPI == kEpiStoreStats || EPI == kEpiGelu) && p.bias != nullptr;
        const ptx::f2 al = ptx::make_f2(p.alpha, p.alpha);
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t tile_i = 0;  // tiles this warp has started: bias buffer parity, position in the aux ring

        // kEpiMulGeluGrad: the 32 x 64 box of the producer's pre-activation for this warp's step g
        // (two steps per tile) lands in buffer g & 1; issued by the elected lane two steps ahead
        auto issue_aux = [&](uint32_t g) {
            const long long u = static_cast<long long>(first_unit) +
                                static_cast<long long>(g >> 1) * unit_stride;
            if (u >= num_units) return;
            int m_blk, n_blk, split;
            decode_unit(p, static_cast<int>(u), m_blk, n_blk, split);
            const uint32_t ab = waux_bar(g & 1u);
            ptx::mbar_expect_tx(ab, kBoxBytes);
            ptx::tma_load_2d(aux0 + (g & 1u) * kBoxBytes, &tmE, ab,
                             n_blk * BLOCK_N + hf * 128 + static_cast<int>(g & 1u) * 64,
                             m_blk * Cfg::TILE_M + static_cast<int>(rank) * kBlockM + q * 32);
        };
        if constexpr (EPI == kEpiMulGeluGrad) {
            if (ptx::elect_one()) {
                issue_aux(0);
                issue_aux(1);
            }
            __syncwarp();
        }
        auto release_acc = [&](int a) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2) ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(a), 0));
                else ptx::mbar_arrive(tempty_bar(a));
            }
            __syncwarp();
        };

        for (int u = first_unit; u < num_units; u += unit_stride, ++tile_i) {
            if (ptx::ld_shared_u32_volatile(epi_abort_addr) != 0) break;
            int m_blk, n_blk, split;
            decode_unit(p, u, m_blk, n_blk, split);
            const int m0 = m_blk * Cfg::TILE_M + static_cast<int>(rank) * kBlockM;
            const int nw = n_blk * BLOCK_N + hf * 128;  // this warp's first column
            // this lane's four of the warp's 128 bias values, fetched while the tile is still in the
            // tensor core
            uint32_t bv[4] = {0u, 0u, 0u, 0u};
            if (has_bias) {
                const int col = nw + lane * 4;
                if (col < p.N) {  // N is a multiple of 8 and col of 4: all four exist
                    // element loads: the bias pointer is only required to be 2-byte aligned
                    const unsigned short *bp = reinterpret_cast<const unsigned short *>(p.bias) + col;
#pragma unroll
                    for (int k = 0; k < 4; ++k) bv[k] = static_cast<uint32_t>(__ldg(bp + k)) << 16;
                }
            }
            bool ok = true;
            if (lane == 0) ok = wait_barrier(wctx_epi, tfull_bar(acc), acc_phase, 400 + acc);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) ptx::st_shared_u32_volatile(epi_abort_addr, 1);
            ptx::tc_fence_after();
            // The bias buffer of this parity was last read for the tile two back, whose accumulator
            // every warp handed over (after issuing its last bias loads) before this tile's MMAs
            // could start. The four warps of a column half write the same values.
            const uint32_t bias_t = smem + Cfg::OFF_BIAS + (tile_i & 1u) * (BLOCK_N * 4u) +
                                    static_cast<uint32_t>(hf) * 512u;
            if (has_bias) {
                ptx::st_shared_v4(bias_t + static_cast<uint32_t>(lane) * 16u, bv[0], bv[1], bv[2], bv[3]);
                __syncwarp();
            }
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                   static_cast<uint32_t>(acc * BLOCK_N + hf * 128);
            // All four loads of the warp's 128 columns are issued at once (a TMEM load takes several
            // hundred cycles while the tensor core is busy; one after the other they would add up),
            // unless the register budget of the kernel only allows two in flight.
            constexpr int LD_DEPTH = Cfg::DBIAS ? 2 : 4;
            uint32_t rr[LD_DEPTH][32];
#pragma unroll
            for (int i = 0; i < LD_DEPTH; ++i)
                ptx::tmem_ld_32x32_issue(t_acc + static_cast<uint32_t>(i * 32), rr[i]);
            float st_m = -INFINITY, st_s = 0.0f;  // kEpiStoreStats: this thread's row statistics
#pragma unroll
            for (int s4 = 0; s4 < 4; ++s4) {  // 32 columns at a time; two make a stored box
                const int step = s4 >> 1, sub = s4 & 1;
                const uint32_t g = tile_i * 2u + static_cast<uint32_t>(step);
                // the bias of 16 columns at a time, ahead of the arithmetic that uses it (the loads
                // cannot be moved by the compiler across the shared-memory stores in between)
                float4 bb[4];
                auto load_bias16 = [&](int half) {
                    if (has_bias) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            ptx::ld_shared_f32x4(bias_t + 4u * static_cast<uint32_t>(s4 * 32 + half * 16 + j * 4),
                                                 bb[j]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) bb[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    }
                };
                load_bias16(0);
                uint32_t (&r)[32] = rr[s4 % LD_DEPTH];
                if (LD_DEPTH == 4) {
                    if (s4 == 0) {  // one wait covers all four loads
                        ptx::tmem_ld_wait_32(rr[0]);
                        ptx::reg_fence_32(rr[1 % LD_DEPTH]);
                        ptx::reg_fence_32(rr[2 % LD_DEPTH]);
                        ptx::reg_fence_32(rr[3 % LD_DEPTH]);
                    }
                } else {
                    // waits for every load issued so far: the one in use and the one after it
                    ptx::tmem_ld_wait_32(r);
                    ptx::reg_fence_32(rr[(s4 + 1) % LD_DEPTH]);
                }
                // The accumulator goes back once its last column is in registers. Where there is a
                // bias, the hand-over also orders the reuse of the bias buffers, so it waits until
                // this tile's last bias loads have been issued (in the loop over j below).
                constexpr bool kBiasEpi = (EPI == kEpiStore || EPI == kEpiStoreStats || EPI == kEpiGelu);
                constexpr int kReleaseAt = (LD_DEPTH == 4) ? 0 : 3;
                if (!kBiasEpi && s4 == kReleaseAt) release_acc(acc);
                if constexpr (EPI == kEpiF32) {
                    // 32 fp32 columns are a box of their own; two boxes alternate, so a box is
                    // rewritten only after the copy issued two boxes ago has read it
                    const uint32_t fb = stg + static_cast<uint32_t>(s4 & 1) * kBoxBytes;
                    ptx::bulk_wait_group_read<1>();  // every lane: only the one that issued copies has any to wait for
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        ptx::st_shared_v4(fb + chunk_pos(j), r[j * 4], r[j * 4 + 1], r[j * 4 + 2], r[j * 4 + 3]);
                    if (LD_DEPTH == 2 && s4 + 2 < 4)  // these registers are free again
                        ptx::tmem_ld_32x32_issue(t_acc + static_cast<uint32_t>((s4 + 2) * 32), rr[s4 % LD_DEPTH]);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (ptx::elect_one()) {
                        const int x = nw + s4 * 32;
                        const int y = m0 + q * 32;
                        if (ok && x < p.N && y < p.M) {
                            if (p.reduce) ptx::tma_reduce_add_2d(&tmD, fb, x, y);
                            else ptx::tma_store_2d(&tmD, fb, x, y);
                        }
                        ptx::bulk_commit_group();
                    }
                    __syncwarp();
                    continue;
                }
                if (sub == 0) {
                    // the staging box is free once the previous step's store has read it
                    ptx::bulk_wait_group_read<0>();  // every lane: only the one that issued copies has any to wait for
                    __syncwarp();
                    if (EPI == kEpiMulGeluGrad) {
                        bool aok = true;
                        if (lane == 0)
                            aok = wait_barrier(wctx_epi, waux_bar(g & 1u), (g >> 1) & 1u, 500 + ew);
                        aok = __shfl_sync(0xffffffffu, aok ? 1 : 0, 0) != 0;
                        if (!aok) {
                            ptx::st_shared_u32_volatile(epi_abort_addr, 1);
                            ok = false;
                        }
                    }
                }
                float sv[EPI == kEpiStoreStats ? 32 : 1];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t pos = chunk_pos(sub * 4 + j);
                    if (EPI == kEpiMulGeluGrad) {
                        uint32_t x[4], w[4];
                        ptx::ld_shared_v4(aux0 + (g & 1u) * kBoxBytes + pos, x[0], x[1], x[2], x[3]);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const ptx::f2 a2 = ptx::make_f2_bits(r[j * 8 + 2 * k], r[j * 8 + 2 * k + 1]);
                            const ptx::f2 x2 = ptx::make_f2_bits(x[k] << 16, x[k] & 0xffff0000u);
                            w[k] = pack_f2_bf16x2(mul_gelu_bwd2(a2, x2));
                        }
                        ptx::st_shared_v4(stg + pos, w[0], w[1], w[2], w[3]);
                    } else {
                        if (j == 2) {
                            load_bias16(1);
                            if (s4 == 3) release_acc(acc);  // kBiasEpi: the tile's last bias loads are out
                        }
                        const float4 b0 = bb[2 * (j & 1)], b1 = bb[2 * (j & 1) + 1];
                        ptx::f2 z[4];  // eight columns as four packed pairs
                        z[0] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 0], r[j * 8 + 1]), al, ptx::make_f2(b0.x, b0.y));
                        z[1] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 2], r[j * 8 + 3]), al, ptx::make_f2(b0.z, b0.w));
                        z[2] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 4], r[j * 8 + 5]), al, ptx::make_f2(b1.x, b1.y));
                        z[3] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 6], r[j * 8 + 7]), al, ptx::make_f2(b1.z, b1.w));
                        if (EPI == kEpiGelu) {
                            ptx::st_shared_v4(stg + kBoxBytes + pos, pack_f2_bf16x2(z[0]), pack_f2_bf16x2(z[1]),
                                              pack_f2_bf16x2(z[2]), pack_f2_bf16x2(z[3]));
#pragma unroll
                            for (int k = 0; k < 4; ++k) z[k] = gelu_fwd2(z[k]);
                        }
                        const uint32_t w0 = pack_f2_bf16x2(z[0]), w1 = pack_f2_bf16x2(z[1]),
                                       w2 = pack_f2_bf16x2(z[2]), w3 = pack_f2_bf16x2(z[3]);
                        ptx::st_shared_v4(stg + pos, w0, w1, w2, w3);
                        if (EPI == kEpiStoreStats) {  // keep the eight stored (rounded) values
                            sv[j * 8 + 0] = ptx::bf16_lo(w0); sv[j * 8 + 1] = ptx::bf16_hi(w0);
                            sv[j * 8 + 2] = ptx::bf16_lo(w1); sv[j * 8 + 3] = ptx::bf16_hi(w1);
                            sv[j * 8 + 4] = ptx::bf16_lo(w2); sv[j * 8 + 5] = ptx::bf16_hi(w2);
                            sv[j * 8 + 6] = ptx::bf16_lo(w3); sv[j * 8 + 7] = ptx::bf16_hi(w3);
                        }
                    }
                }
                if (EPI == kEpiStoreStats) {
                    // online softmax statistics of this thread's 32 stored values: running
                    // maximum st_m and sum of exp(value - st_m), columns >= v_real left out
                    const int g0 = nw + s4 * 32;
                    float mx = -INFINITY;
                    if (g0 + 32 > p.v_real) {  // only the tile that straddles v_real masks
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if (g0 + k >= p.v_real) sv[k] = -INFINITY;
                    }
#pragma unroll
                    for (int k = 0; k < 32; ++k) mx = fmaxf(mx, sv[k]);
                    if (mx > st_m) {
                        st_s *= exp2f((st_m - mx) * 1.4426950408889634f);  // 0 while st_m = -inf
                        st_m = mx;
                    }
                    if (st_m > -INFINITY) {
                        const float ms = st_m * 1.4426950408889634f;
                        float acc_s = 0.0f;
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            acc_s += ptx::ex2_approx(fmaf(sv[k], 1.4426950408889634f, -ms));
                        st_s += acc_s;
                    }
                }
                if (sub == 1) {
                    // the box is complete: make it visible to the TMA engine and store it
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (ptx::elect_one()) {
                        const int x = nw + step * 64;
                        const int y = m0 + q * 32;
                        if (ok && x < p.N && y < p.M) {
                            ptx::tma_store_2d(&tmD, stg, x, y);
                            if (EPI == kEpiGelu) ptx::tma_store_2d(&tmE, stg + kBoxBytes, x, y);
                        }
                        ptx::bulk_commit_group();
                        // every lane has read this step's pre-activation box (__syncwarp above)
                        if (EPI == kEpiMulGeluGrad) issue_aux(g + 2u);
                    }
                    __syncwarp();
                }
            }
            if (EPI == kEpiStoreStats) {
                const long long grow = static_cast<long long>(m0) + row;
                if (ok && grow < p.M)
                    p.stats[grow * p.stats_ld + n_blk * 2 + hf] = make_float2(st_m, st_s);
            }
            if (++acc == 2) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
        ptx::bulk_wait_group<0>();  // all stores have reached global memory (every lane waits for its own)
        __syncwarp();
      } else {
        // ------------------------------------------------------------ epilogue, eight warps in step
        // The form the 64-wide narrow tiles (plain store, fp32) and the SwiGLU epilogue use: two
        // warps share each lane quarter and split every step's columns in halves (hf = 0 / 1); a
        // named barrier joins the eight warps at every step and warp 2 stores the 128-row chunk.
        // TMA stores and the bulk-group bookkeeping are issued by one elected lane of warp 2, always
        // from a warp-uniform branch with the election at the point of use
        static_assert(EPI == kEpiStore || EPI == kEpiSwiglu || EPI == kEpiF32,
                      "the other epilogues exist only in the warp-by-warp form");
        const bool store_warp = (warp == 2);
        const int et = static_cast<int>(threadIdx.x) - 64;  // 0..255
        const uint32_t stg0 = smem + Cfg::OFF_STG;
        const uint32_t bias_s = smem + Cfg::OFF_BIAS;
        const uint32_t row_off = static_cast<uint32_t>(row) * 128u;
        const uint32_t sw = static_cast<uint32_t>(row & 7);
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t gstep = 0;  // epilogue steps done so far (drives the staging ring)
        constexpr int SLOTS = Cfg::SLOTS;
        constexpr int STEPS = Cfg::STEPS;
        // the accumulator is handed back on the leader CTA's barrier
        auto release_acc = [&](int a) {
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2) ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(a), 0));
                else ptx::mbar_arrive(tempty_bar(a));
            }
            __syncwarp();
        };
        // 8 bf16 columns (one 16-byte chunk) of this thread's row in a staging buffer
        auto chunk_pos = [&](int chunk) { return row_off + ((static_cast<uint32_t>(chunk) ^ sw) << 4); };

        for (int u = first_unit; u < num_units; u += unit_stride) {
            // uniform exit: the flag is only written by epilogue threads inside a unit, and
            // only read here, between the last barrier of one unit and the first of the next
            if (ptx::ld_shared_u32_volatile(epi_abort_addr) != 0) break;
            int m_blk, n_blk, split;
            decode_unit(p, u, m_blk, n_blk, split);
            const int m0 = m_blk * Cfg::TILE_M + static_cast<int>(rank) * kBlockM;
            const int n0 = (EPI == kEpiSwiglu) ? n_blk * 128 : n_blk * BLOCK_N;
            if (EPI == kEpiStore || EPI == kEpiSwiglu) {
                for (int i = et; i < BLOCK_N; i += kEpiThreads) {
                    int col;
                    if (EPI == kEpiSwiglu) col = (i < 128) ? (n0 + i) : (p.swiglu_h + n0 + i - 128);
                    else col = n0 + i;
                    float b = 0.0f;
                    if (p.bias != nullptr && col < p.N) b = __bfloat162float(p.bias[col]);
                    ptx::st_shared_f32(bias_s + 4u * i, b);
                }
            }
            ptx::named_bar_sync(1, kEpiThreads);

            bool ok = true;
            if (lane == 0) ok = wait_barrier(wctx_epi, tfull_bar(acc), acc_phase, 400 + acc);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) ptx::st_shared_u32_volatile(epi_abort_addr, 1);
            ptx::tc_fence_after();
            const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                   static_cast<uint32_t>(acc * BLOCK_N);

#pragma unroll 1
            for (int c = 0; c < STEPS; ++c, ++gstep) {
                const uint32_t slot = gstep % SLOTS;
                const uint32_t buf = stg0 + slot * Cfg::BUFS_PER_STEP * kStgBytes;

                if (EPI == kEpiStore) {
                    // this thread: columns [c*64 + hf*32, +32) of its row
                    const int col0 = c * 64 + hf * 32;
                    uint32_t r[32];
                    ptx::tmem_ld_32x32_wait(t_acc + col0, r);
                    if (c == STEPS - 1) release_acc(acc);  // accumulator fully read
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float4 b0, b1;
                        ptx::ld_shared_f32x4(bias_s + 4u * (col0 + j * 8), b0);
                        ptx::ld_shared_f32x4(bias_s + 4u * (col0 + j * 8 + 4), b1);
                        ptx::f2 z[4];  // eight columns as four packed pairs
                        const ptx::f2 al = ptx::make_f2(p.alpha, p.alpha);
                        z[0] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 0], r[j * 8 + 1]), al, ptx::make_f2(b0.x, b0.y));
                        z[1] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 2], r[j * 8 + 3]), al, ptx::make_f2(b0.z, b0.w));
                        z[2] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 4], r[j * 8 + 5]), al, ptx::make_f2(b1.x, b1.y));
                        z[3] = ptx::fma2(ptx::make_f2_bits(r[j * 8 + 6], r[j * 8 + 7]), al, ptx::make_f2(b1.z, b1.w));
                        ptx::st_shared_v4(buf + chunk_pos(hf * 4 + j), pack_f2_bf16x2(z[0]), pack_f2_bf16x2(z[1]),
                                          pack_f2_bf16x2(z[2]), pack_f2_bf16x2(z[3]));
                    }
                } else if (EPI == kEpiSwiglu) {
                    // step c covers out columns [c*64, +64): gate TMEM cols c*64.., up cols 128 + c*64..
                    const int col0 = c * 64 + hf * 32;
                    uint32_t rg[32], ru[32];
                    ptx::tmem_ld_32x32_x2_wait(t_acc + col0, t_acc + 128 + col0, rg, ru);
                    if (c == STEPS - 1) release_acc(acc);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float g[8], uu[8], o[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int cc = col0 + j * 8 + k;
                            g[k] = __uint_as_float(rg[j * 8 + k]) + ptx::ld_shared_f32(bias_s + 4u * cc);
                            uu[k] = __uint_as_float(ru[j * 8 + k]) +
                                    ptx::ld_shared_f32(bias_s + 4u * (128 + cc));
                            o[k] = silu_fwd(g[k]) * uu[k];
                        }
                        const uint32_t pos = chunk_pos(hf * 4 + j);
                        ptx::st_shared_v4(buf + pos, ptx::pack_bf16x2(o[0], o[1]),
                                          ptx::pack_bf16x2(o[2], o[3]), ptx::pack_bf16x2(o[4], o[5]),
                                          ptx::pack_bf16x2(o[6], o[7]));
                        ptx::st_shared_v4(buf + kStgBytes + pos, ptx::pack_bf16x2(g[0], g[1]),
                                          ptx::pack_bf16x2(g[2], g[3]), ptx::pack_bf16x2(g[4], g[5]),
                                          ptx::pack_bf16x2(g[6], g[7]));
                        ptx::st_shared_v4(buf + 2 * kStgBytes + pos, ptx::pack_bf16x2(uu[0], uu[1]),
                                          ptx::pack_bf16x2(uu[2], uu[3]), ptx::pack_bf16x2(uu[4], uu[5]),
                                          ptx::pack_bf16x2(uu[6], uu[7]));
                    }
                } else {  // kEpiF32: 32 fp32 columns per step, 16 per thread
                    uint32_t r[16];
                    ptx::tmem_ld_32x16_wait(t_acc + c * 32 + hf * 16, r);
                    if (c == STEPS - 1) release_acc(acc);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        ptx::st_shared_v4(buf + chunk_pos(hf * 4 + j), r[j * 4], r[j * 4 + 1],
                                          r[j * 4 + 2], r[j * 4 + 3]);
                }

                // make the staged tile visible to the TMA engine, then one thread stores it
                ptx::fence_proxy_async_smem();
                if (store_warp && SLOTS >= 2) {
                    // the slot the NEXT step writes was last stored SLOTS-1 groups ago
                    if (ptx::elect_one()) ptx::bulk_wait_group_read<(SLOTS >= 2 ? SLOTS - 2 : 0)>();
                }
                __syncwarp();
                ptx::named_bar_sync(1, kEpiThreads);
                if (store_warp) {
                  if (ptx::elect_one()) {
                    const int y = m0;
                    if (ok && y < p.M) {
                        if (EPI == kEpiStore) {
                            const int x = n0 + c * 64;
                            if (x < p.N) ptx::tma_store_2d(&tmD, buf, x, y);
                        } else if (EPI == kEpiSwiglu) {
                            const int x = n0 + c * 64;
                            if (x < p.swiglu_h) {
                                ptx::tma_store_2d(&tmD, buf, x, y);
                                ptx::tma_store_2d(&tmE, buf + kStgBytes, x, y);
                                ptx::tma_store_2d(&tmE, buf + 2 * kStgBytes, p.swiglu_h + x, y);
                            }
                        } else {
                            const int x = n0 + c * 32;
                            if (x < p.N) {
                                if (p.reduce) ptx::tma_reduce_add_2d(&tmD, buf, x, y);
                                else ptx::tma_store_2d(&tmD, buf, x, y);
                            }
                        }
                    }
                    ptx::bulk_commit_group();
                    if (SLOTS == 1) ptx::bulk_wait_group_read<0>();
                  }
                }
                __syncwarp();  // the single-lane block above rejoins its warp before collective ops
                if (SLOTS == 1) ptx::named_bar_sync(1, kEpiThreads);
            }
            if (++acc == 2) {
                acc = 0;
                acc_phase ^= 1u;
            }
        }
        if (store_warp) {
            if (ptx::elect_one()) ptx::bulk_wait_group<0>();  // all stores have reached global memory
        }
      }
    }

    // ---------------------------------------------------------------- common exit
    if (ptx::ld_shared_u32_volatile(abort_addr) != 0 ||
        ptx::ld_shared_u32_volatile(epi_abort_addr) != 0) {
        // a wait expired somewhere: give copies and MMAs still in flight time to land
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    __syncwarp();
    ptx::tc_fence_before();
    if (CG == 2) ptx::cluster_sync();  // neither CTA of a pair leaves while the other may still signal it
    else __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<CG>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace nb
