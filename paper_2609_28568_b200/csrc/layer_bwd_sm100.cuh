// Backward of one linear layer as ONE persistent launch for sm_100a:
//
//     dinp[BT, C]     = dz[BT, OC] . W[OC, C]        (x gelu'(inp_pre) in the epilogue, optional)
//     dweight[OC, C] += dz^T[OC, BT] . inp[BT, C]    fp32, reduce-added
//     dbias[OC]      += column sums of dz            fp32, optional
//
// Both products read dz, and neither depends on the other, so their work units share one list:
// 256 x 256 tiles of dinp over the whole K = OC ("D units"), and 256 x 256 tiles of dweight over
// a range of 64-row k-blocks of K = BT ("W units"; partial sums meet in memory through TMA
// reduce-adds, so a W tile may be cut anywhere along K). A launch of its own for each product
// runs its last wave partly empty (16384 x 768 outputs are 192 tiles for 74 CTA pairs: 2.59
// waves run as 3) and pays a start and an end; here the weight-gradient k-blocks fill what the
// input-gradient tiles leave, every CTA pair gets the same amount of tensor-core work, and the
// long epilogue of a D unit (gelu') runs under the long main loop of a W unit.
//
// Schedule (computed on the host, see plan_layer_bwd): "rounds" of one unit per CTA pair, D rounds
// and W rounds interleaved in the order given by a bit mask, so that at any time all pairs work on
// neighbouring tiles of the same product (operand reuse in L2); then the last, partial D round;
// then the remaining W k-blocks, cut into contiguous ranges whose lengths make up for what a pair
// got more or less than the others before.
//
// Roles (four warpgroups, registers re-divided with setmaxnreg):
//   warp 0        TMA producer            warp 1   MMA issuer (leader CTA of the pair)
//   warp 2        TMEM allocation         warp 3   idle
//   warps 4..11   epilogue, warp-private: 32 rows x 128 columns of the tile each
//   warps 12..15  bias-gradient reducers (sum the dz^T tiles of the W units of column tile 0 from
//                 shared memory once the tensor core is done with them)
#pragma once
#include "gemm_sm100.cuh"

namespace nb {

constexpr int kMaxPairs = 80;
constexpr int kLbThreads = 512;
constexpr int kLbMaxRounds = 64;

struct LayerBwdParams {
    int BT, C, OC;
    int num_pairs;
    // D units: tiles of dinp, K = OC
    int d_tiles_m, d_tiles_n, d_tiles, d_group_m, d_kblocks;
    int d_rounds;  // full rounds (num_pairs tiles each)
    int d_tail;    // tiles of the partial round: pairs [0, d_tail) take one more
    // W units: tiles of dweight, K = BT cut into chunks of w_kbc k-blocks; unit j = chunk j / w_tiles
    // of tile j % w_tiles
    int w_tiles_m, w_tiles_n, w_tiles, w_kblocks, w_kbc, w_units;
    int w_rounds;  // full rounds (num_pairs units each)
    unsigned long long round_is_w;  // order of the d_rounds + w_rounds full rounds, bit r: W round
    // what is left of the W units after the full rounds, as one line of k-blocks: w_kbc per unit for
    // the first w_tail_full k-blocks, then w_last_len per unit (the units of the last chunk, when K
    // does not divide evenly); pair p takes [w_tail_begin[p], w_tail_begin[p + 1])
    int w_tail_full, w_last_len;
    int w_tail_begin[kMaxPairs + 1];
    float *dbias;  // [OC] or nullptr
    int *status;
    unsigned long long timeout_ns;
};

struct LbUnit {
    int is_w;
    int m_blk, n_blk;
    int kb0, kb1;
};

// The sequence of units of one CTA pair; every role of both CTAs walks the same sequence.
struct LbIter {
    int r, iD, iW, part, x, x_end, pair;  // part: 0 whole rounds, 1 last D round, 2 W tail, 3 done
    static __host__ __device__ __forceinline__ int imin(int a, int b) { return a < b ? a : b; }
    __host__ __device__ __forceinline__ LbIter(const LayerBwdParams &p, int pair_)
        : r(0), iD(0), iW(0), part(0), x(p.w_tail_begin[pair_]), x_end(p.w_tail_begin[pair_ + 1]),
          pair(pair_)
    {
    }
    static __host__ __device__ __forceinline__ void d_tile(const LayerBwdParams &p, int t, LbUnit &u)
    {
        const int per_group = p.d_group_m * p.d_tiles_n;
        const int g = t / per_group;
        const int rr = t - g * per_group;
        const int first_m = g * p.d_group_m;
        const int gsz = imin(p.d_group_m, p.d_tiles_m - first_m);
        u.is_w = 0;
        u.m_blk = first_m + rr % gsz;
        u.n_blk = rr / gsz;
        u.kb0 = 0;
        u.kb1 = p.d_kblocks;
    }
    static __host__ __device__ __forceinline__ void w_unit(const LayerBwdParams &p, int j, int ko0, int ko1,
                                                  LbUnit &u)
    {
        const int s = j / p.w_tiles;
        const int t = j - s * p.w_tiles;
        u.is_w = 1;
        u.m_blk = t / p.w_tiles_n;
        u.n_blk = t - u.m_blk * p.w_tiles_n;
        u.kb0 = imin(s * p.w_kbc + ko0, p.w_kblocks);
        u.kb1 = imin(s * p.w_kbc + ko1, p.w_kblocks);
    }
    // the i-th D tile of this pair, or -1
    static __host__ __device__ __forceinline__ int d_ordinal(const LayerBwdParams &p, int pair, int i)
    {
        if (i < p.d_rounds) return i * p.num_pairs + pair;
        if (i == p.d_rounds && pair < p.d_tail) return p.d_rounds * p.num_pairs + pair;
        return -1;
    }
    __host__ __device__ __forceinline__ bool next(const LayerBwdParams &p, LbUnit &u)
    {
        while (true) {
            if (part == 0) {
                if (r < p.d_rounds + p.w_rounds) {
                    const bool w = ((p.round_is_w >> r) & 1ull) != 0;
                    ++r;
                    if (w) {
                        w_unit(p, iW * p.num_pairs + pair, 0, p.w_kbc, u);
                        ++iW;
                        if (u.kb0 >= u.kb1) continue;  // a chunk beyond the ragged end of K
                    } else {
                        d_tile(p, iD * p.num_pairs + pair, u);
                        ++iD;
                    }
                    return true;
                }
                part = 1;
            }
            if (part == 1) {
                part = 2;
                if (pair < p.d_tail) {
                    d_tile(p, p.d_rounds * p.num_pairs + pair, u);
                    return true;
                }
            }
            if (part == 2) {
                if (x < x_end) {
                    int j = p.w_rounds * p.num_pairs, ko, ulen;
                    if (x < p.w_tail_full) {
                        j += x / p.w_kbc;
                        ko = x % p.w_kbc;
                        ulen = p.w_kbc;
                    } else {
                        const int xr = x - p.w_tail_full;
                        j += p.w_tail_full / p.w_kbc + xr / p.w_last_len;
                        ko = xr % p.w_last_len;
                        ulen = p.w_last_len;
                    }
                    const int len = imin(ulen - ko, x_end - x);
                    x += len;
                    w_unit(p, j, ko, ko + len, u);
                    if (u.kb0 >= u.kb1) continue;
                    return true;
                }
                part = 3;
            }
            return false;
        }
    }
};

template <bool GELU_GRAD_, bool DBIAS_>
struct LbCfg {
    static constexpr bool GELU_GRAD = GELU_GRAD_;
    static constexpr bool DBIAS = DBIAS_;
    static constexpr int STAGES = GELU_GRAD_ ? 4 : 5;
    static constexpr uint32_t A_BYTES = kBlockM * kBlockK * 2;  // 128 rows of the pair's 256
    static constexpr uint32_t B_BYTES = 128 * kBlockK * 2;      // this CTA's half of the 256 columns
    static constexpr uint32_t OFF_A = 0;
    static constexpr uint32_t OFF_B = STAGES * A_BYTES;
    static constexpr uint32_t OFF_STG = STAGES * (A_BYTES + B_BYTES);
    // staging boxes (4 KB: 32 rows x 128 bytes, 128B-swizzled) per epilogue warp:
    //   box 0       bf16 result of a D unit / first fp32 box of a W unit
    //   GELU_GRAD:  boxes 1, 2 receive the pre-activation boxes of the next two D steps, so the
    //               fp32 results of a W unit go through box 0 alone
    //   otherwise:  box 1 is the second fp32 box (two reduce-adds in flight)
    static constexpr int F32_RING = GELU_GRAD_ ? 1 : 2;
    static constexpr int WARP_BOXES = GELU_GRAD_ ? 3 : 2;
    static constexpr uint32_t kBoxBytes = 4096;
    static constexpr uint32_t STG_BYTES = kEpiWarps * WARP_BOXES * kBoxBytes;
    static constexpr uint32_t OFF_PART = OFF_STG + STG_BYTES;  // 128 floats: dbias partial sums
    static constexpr uint32_t OFF_BAR = OFF_PART + 512;
    static constexpr uint32_t BAR_BYTES = 512;
    static constexpr uint32_t SMEM_BYTES = OFF_BAR + BAR_BYTES;
    static constexpr uint32_t TMEM_COLS = 512;  // two 256-column accumulators
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

template <class Cfg>
__global__ void __launch_bounds__(kLbThreads, 1)
layer_bwd_kernel(const __grid_constant__ CUtensorMap tmDz,    // dz   [BT, OC] bf16, 64 x 64 boxes
                 const __grid_constant__ CUtensorMap tmW,     // W    [OC, C]  bf16, 64 x 64 boxes
                 const __grid_constant__ CUtensorMap tmInp,   // inp  [BT, C]  bf16, 64 x 64 boxes
                 const __grid_constant__ CUtensorMap tmDinp,  // dinp [BT, C]  bf16, 32-row boxes
                 const __grid_constant__ CUtensorMap tmPre,   // inp_pre [BT, C] bf16, 32-row boxes
                 const __grid_constant__ CUtensorMap tmDw,    // dweight [OC, C] fp32, 32 x 32 boxes
                 const __grid_constant__ LayerBwdParams p)
{
    constexpr int STAGES = Cfg::STAGES;
    constexpr bool GELU_GRAD = Cfg::GELU_GRAD;
    constexpr bool DBIAS = Cfg::DBIAS;
    constexpr uint32_t kBoxBytes = Cfg::kBoxBytes;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem = ptx::smem_u32(smem_raw);
    const int warp = static_cast<int>(threadIdx.x >> 5);
    const int lane = static_cast<int>(threadIdx.x & 31);
    const uint32_t rank = blockIdx.x & 1u;  // position in the CTA pair (pairs are consecutive blocks)
    const int pair = static_cast<int>(blockIdx.x >> 1);

    const bool smem_ok = (smem & 1023u) == 0;
    if (!smem_ok && threadIdx.x == 0 && atomicCAS(p.status, 0, kStatusBadSmem) == 0)
        p.status[2] = static_cast<int>(blockIdx.x);

    // barrier slots (8 bytes each): full[S], empty[S], free[S], tmem_full[2], tmem_empty[2],
    // then 16 pre-activation barriers (two per epilogue warp); bytes 480.. hold the TMEM base
    // address and the two abort flags
    const uint32_t bar0 = smem + Cfg::OFF_BAR;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto free_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (3 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (3 * STAGES + 2 + b); };
    auto aux_bar = [&](uint32_t i) { return bar0 + 8u * (3 * STAGES + 4 + i); };
    static_assert(8 * (3 * STAGES + 4 + 16) <= 480, "barrier region");
    const uint32_t tmem_slot = bar0 + 480;
    const uint32_t abort_addr = bar0 + 484;
    const uint32_t epi_abort_addr = bar0 + 488;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
            ptx::mbar_init(free_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), kEpiWarps * 2);
        }
        for (uint32_t b = 0; b < 16; ++b) ptx::mbar_init(aux_bar(b), 1);
        ptx::st_shared_u32_volatile(abort_addr, 0);
        ptx::st_shared_u32_volatile(epi_abort_addr, 0);
        ptx::fence_barrier_init();
        ptx::prefetch_tmap(&tmDz);
        ptx::prefetch_tmap(&tmW);
        ptx::prefetch_tmap(&tmInp);
        ptx::prefetch_tmap(&tmDinp);
        ptx::prefetch_tmap(&tmDw);
        if (GELU_GRAD) ptx::prefetch_tmap(&tmPre);
    }
    if (warp == 2) {
        ptx::tmem_alloc<2>(tmem_slot, Cfg::TMEM_COLS);
        ptx::tmem_relinquish<2>();
    }
    ptx::tc_fence_before();
    ptx::cluster_sync();  // the peer's barriers are initialised before anyone signals them
    ptx::tc_fence_after();
    // nothing above touched global memory: it may overlap the previous kernel's tail
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const uint32_t tmem_base = ptx::ld_shared_u32_volatile(tmem_slot);
    const WaitCtx wctx{abort_addr, p.status, p.timeout_ns};
    // The epilogue waits for a whole unit where the issuer waits for one stage: with twice the limit
    // the wait that is closest to the cause of a stall is the one that expires and gets reported.
    const WaitCtx wctx_epi{abort_addr, p.status, 2 * p.timeout_ns};

    if (warp < 4) {
        ptx::setmaxnreg_dec<56>();
        if (!smem_ok) {
            // fall through to the common exit
        } else if (warp == 0) {
            // -------------------------------------------------------- TMA producer (both CTAs)
            if (ptx::elect_one()) {
                LbIter it(p, pair);
                LbUnit u;
                int stage = 0;
                uint32_t phase = 0;
                bool ok = true;
                while (ok && it.next(p, u)) {
                    const int m0 = u.m_blk * 256 + static_cast<int>(rank) * 128;
                    const int n0 = u.n_blk * 256 + static_cast<int>(rank) * 128;
                    const CUtensorMap *mapB = u.is_w ? &tmInp : &tmW;
                    for (int kb = u.kb0; kb < u.kb1; ++kb) {
                        ok = wait_barrier(wctx, DBIAS ? free_bar(stage) : empty_bar(stage), phase ^ 1u,
                                          100 + stage);
                        if (!ok) break;
                        // the leader's barrier collects the bytes of both CTAs of the pair
                        const uint32_t fb = ptx::mapa(full_bar(stage), 0);
                        if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), 2 * (Cfg::A_BYTES + Cfg::B_BYTES));
                        const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES;
                        const uint32_t sb = smem + Cfg::OFF_B + stage * Cfg::B_BYTES;
                        const int k0 = kb * kBlockK;
                        if (u.is_w) {  // A = dz^T: m runs along dz's columns, k along its rows
                            ptx::tma_load_2d_pair(sa, &tmDz, fb, m0, k0);
                            ptx::tma_load_2d_pair(sa + 8192u, &tmDz, fb, m0 + 64, k0);
                        } else {       // A = dz: m along its rows, k along its columns
                            ptx::tma_load_2d_pair(sa, &tmDz, fb, k0, m0);
                            ptx::tma_load_2d_pair(sa + 8192u, &tmDz, fb, k0, m0 + 64);
                        }
                        // B (W for a D unit, inp for a W unit): n along the columns, k along the rows
                        ptx::tma_load_2d_pair(sb, mapB, fb, n0, k0);
                        ptx::tma_load_2d_pair(sb + 8192u, mapB, fb, n0 + 64, k0);
                        if (++stage == STAGES) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------- MMA issuer (leader CTA only)
            if (rank == 0 && ptx::elect_one()) {
                constexpr uint32_t idesc_d = make_idesc(256, 256, false, true);
                constexpr uint32_t idesc_w = make_idesc(256, 256, true, true);
                LbIter it(p, pair);
                LbUnit u;
                int stage = 0;
                uint32_t phase = 0;
                int acc = 0;
                uint32_t acc_phase = 0;
                bool ok = true;
                while (ok && it.next(p, u)) {
                    ok = wait_barrier(wctx, tempty_bar(acc), acc_phase ^ 1u, 200 + acc);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * 256);
                    const uint32_t idesc = u.is_w ? idesc_w : idesc_d;
                    // K-major A (D unit): 16 k = 32 B inside the swizzle row; MN-major: 16 k = 2048 B
                    const uint32_t a_step = u.is_w ? (2048u >> 4) : (32u >> 4);
                    const bool mine = DBIAS && u.is_w && u.n_blk == 0;
                    for (int kb = u.kb0; kb < u.kb1; ++kb) {
                        ok = wait_barrier(wctx, full_bar(stage), phase, 300 + stage);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES;
                        const uint32_t sb = smem + Cfg::OFF_B + stage * Cfg::B_BYTES;
                        const uint64_t adesc = u.is_w ? make_smem_desc(sa, 8192, 1024)
                                                      : make_smem_desc(sa, 16, 1024);
                        const uint64_t bdesc = make_smem_desc(sb, 8192, 1024);
#pragma unroll
                        for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                            ptx::umma_bf16<2>(d_tmem, adesc + static_cast<uint64_t>(k * a_step),
                                              bdesc + static_cast<uint64_t>(k * (2048u >> 4)), idesc,
                                              (kb > u.kb0 || k > 0) ? 1u : 0u);
                        }
                        // Without reducers the producer waits on empty[s]. With them it waits on
                        // free[s], which a stage they do not read gets from here and a stage they
                        // read gets from them; empty[s] then counts only the uses they read.
                        if (!DBIAS || mine) ptx::umma_commit<2>(empty_bar(stage));
                        else ptx::umma_commit<2>(free_bar(stage));
                        if (++stage == STAGES) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    ptx::umma_commit<2>(tfull_bar(acc));
                    if (++acc == 2) {
                        acc = 0;
                        acc_phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp >= 12) {
        ptx::setmaxnreg_dec<64>();
        if (DBIAS && smem_ok) {
            // -------------------------------------------------------- bias-gradient reducers
            // A tile of a W unit (MN-major): two boxes of 64 k-rows x 128 bytes (64 m values),
            // swizzled. Thread t sums chunk (t & 15) (8 consecutive m) over k rows (t >> 4) + 8 i.
            const int rt = static_cast<int>(threadIdx.x) - 384;  // 0..127
            const int cc = rt & 15;
            const int kbase = rt >> 4;
            const uint32_t part_s = smem + Cfg::OFF_PART;
            ptx::st_shared_f32(part_s + 4u * rt, 0.0f);
            ptx::named_bar_sync(2, 128);
            LbIter it(p, pair);
            LbUnit u;
            // Only the stages of the W units of column tile 0 are read here. The position in the
            // ring follows from the unit sequence; empty[s] completes one phase per use of stage s
            // that is read here (the issuer commits to it for those uses only), so its parity is
            // kept per stage. The reducers can neither fall behind nor run ahead of it: the next
            // use of a stage they read waits for their arrive on free[s].
            int stage = 0;
            uint32_t mphase = 0;  // bit s: parity of the next use of stage s that is read here
            bool ok = true;
            while (it.next(p, u)) {
                const int nkb = u.kb1 - u.kb0;
                if (!(u.is_w && u.n_blk == 0)) {
                    stage = (stage + nkb) % STAGES;
                    continue;
                }
                float sum[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) sum[k] = 0.0f;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (ok) {
                        bool w = true;
                        if (lane == 0) w = wait_barrier(wctx, empty_bar(stage), (mphase >> stage) & 1u, 600 + stage);
                        ok = __shfl_sync(0xffffffffu, w ? 1 : 0, 0) != 0;
                    }
                    if (ok) {
                        const uint32_t sa = smem + Cfg::OFF_A + stage * Cfg::A_BYTES +
                                            static_cast<uint32_t>(cc >> 3) * 8192u;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const uint32_t kr = static_cast<uint32_t>(kbase + 8 * i);
                            uint32_t x[4];
                            ptx::ld_shared_v4(sa + kr * 128u + (((cc & 7u) ^ (kr & 7u)) << 4), x[0], x[1],
                                              x[2], x[3]);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                sum[2 * k] += ptx::bf16_lo(x[k]);
                                sum[2 * k + 1] += ptx::bf16_hi(x[k]);
                            }
                        }
                    }
                    // all four warps have read the stage: one arrive hands it back to the producer
                    ptx::named_bar_sync(2, 128);
                    if (rt == 0) ptx::mbar_arrive(free_bar(stage));
                    mphase ^= 1u << stage;
                    if (++stage == STAGES) stage = 0;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) atomicAdd_shared_f32(part_s + 4u * (cc * 8 + k), sum[k]);
                ptx::named_bar_sync(2, 128);
                const int m = u.m_blk * 256 + static_cast<int>(rank) * 128 + rt;
                if (ok && m < p.OC) atomicAdd(p.dbias + m, ptx::ld_shared_f32(part_s + 4u * rt));
                ptx::st_shared_f32(part_s + 4u * rt, 0.0f);
                ptx::named_bar_sync(2, 128);
            }
        }
    } else {
        ptx::setmaxnreg_inc<192>();
        if (smem_ok) {
            // -------------------------------------------------------- epilogue (warps 4..11)
            // Warp w reads TMEM lanes 32 (w % 4) .. +31: rows q*32.. of the CTA's 128; two warps
            // share a lane quarter and take 128 columns each (hf = 0 / 1).
            const int ew = warp - 4;
            const int q = warp & 3;
            const int hf = ew >> 2;
            const uint32_t stg = smem + Cfg::OFF_STG + static_cast<uint32_t>(ew) * Cfg::WARP_BOXES * kBoxBytes;
            const uint32_t aux0 = stg + kBoxBytes;  // GELU_GRAD: two pre-activation boxes
            const uint32_t lane_off = static_cast<uint32_t>(lane) * 128u;
            const uint32_t sw = static_cast<uint32_t>(lane & 7);
            auto chunk_pos = [&](int chunk) { return lane_off + ((static_cast<uint32_t>(chunk) ^ sw) << 4); };
            auto waux_bar = [&](uint32_t b) { return aux_bar(static_cast<uint32_t>(ew) * 2u + b); };
            int acc = 0;
            uint32_t acc_phase = 0;
            uint32_t d_ord = 0;  // D units this warp has started

            // the 32 x 64 pre-activation box of D step g of this pair (two steps per D unit) lands
            // in box g & 1, issued two steps ahead by the elected lane
            auto issue_aux = [&](uint32_t g) {
                const int t = LbIter::d_ordinal(p, pair, static_cast<int>(g >> 1));
                if (t < 0) return;
                LbUnit du;
                LbIter::d_tile(p, t, du);
                const uint32_t ab = waux_bar(g & 1u);
                ptx::mbar_expect_tx(ab, kBoxBytes);
                ptx::tma_load_2d(aux0 + (g & 1u) * kBoxBytes, &tmPre, ab,
                                 du.n_blk * 256 + hf * 128 + static_cast<int>(g & 1u) * 64,
                                 du.m_blk * 256 + static_cast<int>(rank) * 128 + q * 32);
            };
            if constexpr (GELU_GRAD) {
                if (ptx::elect_one()) {
                    issue_aux(0);
                    issue_aux(1);
                }
                __syncwarp();
            }
            auto release_acc = [&](int a) {
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(a), 0));
                __syncwarp();
            };

            LbIter it(p, pair);
            LbUnit u;
            while (it.next(p, u)) {
                if (ptx::ld_shared_u32_volatile(epi_abort_addr) != 0) break;
                const int m0 = u.m_blk * 256 + static_cast<int>(rank) * 128;
                const int nw = u.n_blk * 256 + hf * 128;  // this warp's first column
                bool ok = true;
                if (lane == 0) ok = wait_barrier(wctx_epi, tfull_bar(acc), acc_phase, 400 + acc);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) ptx::st_shared_u32_volatile(epi_abort_addr, 1);
                ptx::tc_fence_after();
                const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       static_cast<uint32_t>(acc * 256 + hf * 128);
                uint32_t rr[4][32];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    ptx::tmem_ld_32x32_issue(t_acc + static_cast<uint32_t>(i * 32), rr[i]);
                // the previous unit's last copy has read box 0 (and box 1) by now; every lane
                // waits, only the one that issued copies has any to wait for
                ptx::bulk_wait_group_read<0>();
                ptx::tmem_ld_wait_32(rr[0]);
                ptx::reg_fence_32(rr[1]);
                ptx::reg_fence_32(rr[2]);
                ptx::reg_fence_32(rr[3]);
                release_acc(acc);  // the accumulator is in registers

                if (u.is_w) {
                    // ---------------- fp32 tile of dweight: 32-column boxes, reduce-added
#pragma unroll
                    for (int s4 = 0; s4 < 4; ++s4) {
                        uint32_t (&r)[32] = rr[s4];
                        const uint32_t fb = stg + (Cfg::F32_RING == 2 ? static_cast<uint32_t>(s4 & 1) * kBoxBytes : 0u);
                        ptx::bulk_wait_group_read<Cfg::F32_RING - 1>();
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            ptx::st_shared_v4(fb + chunk_pos(j), r[j * 4], r[j * 4 + 1], r[j * 4 + 2], r[j * 4 + 3]);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (ptx::elect_one()) {
                            const int x = nw + s4 * 32;
                            const int y = m0 + q * 32;
                            if (ok && x < p.C && y < p.OC) ptx::tma_reduce_add_2d(&tmDw, fb, x, y);
                            ptx::bulk_commit_group();
                        }
                        __syncwarp();
                    }
                } else {
                    // ---------------- bf16 tile of dinp: 64-column boxes
#pragma unroll
                    for (int s4 = 0; s4 < 4; ++s4) {
                        const int step = s4 >> 1, sub = s4 & 1;
                        const uint32_t g = d_ord * 2u + static_cast<uint32_t>(step);
                        uint32_t (&r)[32] = rr[s4];
                        // without pre-activation boxes the two steps of a tile alternate between
                        // boxes 0 and 1, so a step waits only for the store before the previous one
                        const uint32_t ob = stg + (GELU_GRAD ? 0u : static_cast<uint32_t>(step) * kBoxBytes);
                        if (sub == 0) {
                            ptx::bulk_wait_group_read<GELU_GRAD ? 0 : 1>();
                            __syncwarp();
                            if (GELU_GRAD) {
                                bool aok = true;
                                if (lane == 0) aok = wait_barrier(wctx_epi, waux_bar(g & 1u), (g >> 1) & 1u, 500 + ew);
                                aok = __shfl_sync(0xffffffffu, aok ? 1 : 0, 0) != 0;
                                if (!aok) {
                                    ptx::st_shared_u32_volatile(epi_abort_addr, 1);
                                    ok = false;
                                }
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t pos = chunk_pos(sub * 4 + j);
                            uint32_t w[4];
                            if (GELU_GRAD) {
                                uint32_t x[4];
                                ptx::ld_shared_v4(aux0 + (g & 1u) * kBoxBytes + pos, x[0], x[1], x[2], x[3]);
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const ptx::f2 a2 = ptx::make_f2_bits(r[j * 8 + 2 * k], r[j * 8 + 2 * k + 1]);
                                    const ptx::f2 x2 = ptx::make_f2_bits(x[k] << 16, x[k] & 0xffff0000u);
                                    w[k] = pack_f2_bf16x2(mul_gelu_bwd2(a2, x2));
                                }
                            } else {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    w[k] = ptx::pack_bf16x2(__uint_as_float(r[j * 8 + 2 * k]),
                                                            __uint_as_float(r[j * 8 + 2 * k + 1]));
                            }
                            ptx::st_shared_v4(ob + pos, w[0], w[1], w[2], w[3]);
                        }
                        if (sub == 1) {
                            ptx::fence_proxy_async_smem();
                            __syncwarp();
                            if (ptx::elect_one()) {
                                const int x = nw + step * 64;
                                const int y = m0 + q * 32;
                                if (ok && x < p.C && y < p.BT) ptx::tma_store_2d(&tmDinp, ob, x, y);
                                ptx::bulk_commit_group();
                                // every lane has read this step's pre-activation box (__syncwarp above)
                                if (GELU_GRAD) issue_aux(g + 2u);
                            }
                            __syncwarp();
                        }
                    }
                    ++d_ord;
                }
                if (++acc == 2) {
                    acc = 0;
                    acc_phase ^= 1u;
                }
            }
            ptx::bulk_wait_group<0>();  // all stores and reduce-adds have reached global memory
            __syncwarp();
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
    ptx::cluster_sync();  // neither CTA of a pair leaves while the other may still signal it
    if (warp == 2) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<2>(tmem_base, Cfg::TMEM_COLS);
    }
}

}  // namespace nb
