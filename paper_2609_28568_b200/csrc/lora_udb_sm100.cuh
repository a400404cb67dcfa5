// Two skinny products of an adapted projection's backward from ONE pass over dy, for sm_100a:
//
//     u [BT, r]   = bf16( scale * dy[BT, OC] . B[OC, r] )     (contracts OC)
//     dB[OC, r] (+)= dy^T[OC, BT] . t[BT, r]                   (contracts BT; fp32, reduce-added)
//
// Both are bound by reading dy (r is 8..64, dy is tens of megabytes), and as launches of their own
// each reads it once. Here a CTA owns a panel of 128 rows of dy and streams it in tiles of
// 128 rows x 128 columns; every tile feeds two MMAs from the same shared-memory bytes:
//   - as a K-major A operand (M = the 128 rows, K = the 128 columns) against B's rows of those
//     columns: the panel's u, accumulated in TMEM over all tiles of the panel;
//   - as an MN-major A operand (M = the 128 columns, K = the 128 rows) against the panel's rows of
//     t: this panel's whole contribution to 128 rows of dB, which the epilogue reduce-adds into
//     dB at once (four TMEM buffers, so the next tiles' MMAs do not wait for it).
// A tile is fetched as four 64 x 64 boxes with 128-byte rows and the 128-byte swizzle; "row r,
// 64 columns" is at the same place whether the tensor core walks the tile by rows or by columns,
// which is what lets one copy serve both products. The panels walk the column tiles in rotated
// orders (panel pn starts at tile pn mod tiles), so that at any moment the CTAs work on different
// rows of B and dB.
//
// Optionally a third product rides on the same launch: the panel's contribution to the A gradient,
//     dA[r, C] (+)= u^T[r, BT] . x[BT, C]                     (contracts BT; fp32, reduce-added)
// Once a panel's u is final, the epilogue also leaves it (scaled, bf16: the same values it stores) in
// shared memory in the layout of the t tile, and the CTA streams the panel's rows of x through the
// same stage ring: each 128 x 128 tile of x, read MN-major exactly like a dy tile in the dB product,
// times the panel's u gives 128 columns of dA (transposed in TMEM: lanes = columns of x), which the
// epilogue turns while staging and reduce-adds. The launch of the dA product and its start and end
// are saved; x is read once, as before.
//
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 epilogue (TMEM lane quarter = warp % 4).
// Every wait is bounded as in gemm_kernel; on expiry the kernel records it and leaves.
#pragma once
#include "gemm_sm100.cuh"

namespace nb {

constexpr int kUdbThreads = 192;
constexpr int kUdbStages = 3;
constexpr uint32_t kUdbABytes = 32768;  // dy tile: 128 rows x 128 columns bf16
constexpr uint32_t kUdbBBytes = 16384;  // 128 rows of B (or of t) x 64 columns (r real, the rest zero)
constexpr uint32_t kUdbOffA = 0;
constexpr uint32_t kUdbOffB = kUdbStages * kUdbABytes;
constexpr uint32_t kUdbOffT = kUdbOffB + kUdbStages * kUdbBBytes;
constexpr uint32_t kUdbOffU = kUdbOffT + kUdbBBytes;            // the panel's u, bf16, laid out like the t tile
constexpr uint32_t kUdbOffStg = kUdbOffU + kUdbBBytes;          // 4 warps x 2 boxes of 4 KB
constexpr uint32_t kUdbOffBar = kUdbOffStg + 4 * 2 * 4096;
constexpr uint32_t kUdbSmemBytes = kUdbOffBar + 256;
constexpr int kUdbDbBufs = 4;
constexpr uint32_t kUdbTmemCols = 512;  // u: 64 columns; four dB buffers of 64

struct UdbParams {
    int BT, OC, r;
    int panels;    // ceil(BT / 128)
    int tiles;     // ceil(OC / 128)
    int want_db;   // 0: only u
    int want_da;   // 1: also dA (+)= u^T . x, x [BT, C]
    int C;         // columns of x
    int xtiles;    // ceil(C / 128)
    float alpha;
    __nv_bfloat16 *u;  // first element of this adapter's column slice of u
    int u_ld;          // elements from one row of u to the next
    int *status;
    unsigned long long timeout_ns;
};

__global__ void __launch_bounds__(kUdbThreads, 1)
lora_udb_kernel(const __grid_constant__ CUtensorMap tmDy,  // dy [BT, OC] bf16, 64 x 64 boxes
                const __grid_constant__ CUtensorMap tmB,   // lora_b [OC, r] bf16, 64 x 64 boxes
                const __grid_constant__ CUtensorMap tmT,   // t slice [BT, r] bf16, 64 x 64 boxes
                const __grid_constant__ CUtensorMap tmDb,  // dB [OC, r] fp32, 32 x 32 boxes
                const __grid_constant__ CUtensorMap tmX,   // x [BT, C] bf16, 64 x 64 boxes (want_da)
                const __grid_constant__ CUtensorMap tmDa,  // dA [r, C] fp32, 32 x 32 boxes (want_da)
                const UdbParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem = ptx::smem_u32(smem_raw);
    const int warp = static_cast<int>(threadIdx.x >> 5);
    const int lane = static_cast<int>(threadIdx.x & 31);
    const bool smem_ok = (smem & 1023u) == 0;
    if (!smem_ok && threadIdx.x == 0 && atomicCAS(p.status, 0, kStatusBadSmem) == 0)
        p.status[2] = static_cast<int>(blockIdx.x);

    // barriers: full[S], empty[S], t_full, t_empty, u_full, u_empty, db_full[NB], db_empty[NB]
    constexpr int S = kUdbStages;
    constexpr int NB = kUdbDbBufs;
    const uint32_t bar0 = smem + kUdbOffBar;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    const uint32_t t_full = bar0 + 8u * (2 * S), t_empty = bar0 + 8u * (2 * S + 1);
    const uint32_t u_full = bar0 + 8u * (2 * S + 2), u_empty = bar0 + 8u * (2 * S + 3);
    auto dbfull_bar = [&](int b) { return bar0 + 8u * (2 * S + 4 + b); };
    auto dbempty_bar = [&](int b) { return bar0 + 8u * (2 * S + 4 + NB + b); };
    // the panel's u in shared memory: written by the four epilogue warps, read by the dA MMAs
    const uint32_t us_full = bar0 + 8u * (2 * S + 4 + 2 * NB), us_empty = bar0 + 8u * (2 * S + 5 + 2 * NB);
    const uint32_t tmem_slot = bar0 + 240, abort_addr = bar0 + 244;
    static_assert(8 * (2 * S + 6 + 2 * NB) <= 240, "barrier region");

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        ptx::mbar_init(t_full, 1);
        ptx::mbar_init(t_empty, 1);   // the issuer's commit after a panel's last tile
        ptx::mbar_init(u_full, 1);
        ptx::mbar_init(u_empty, 4);   // one arrive per epilogue warp
        for (int b = 0; b < NB; ++b) {
            ptx::mbar_init(dbfull_bar(b), 1);
            ptx::mbar_init(dbempty_bar(b), 4);
        }
        ptx::mbar_init(us_full, 4);   // one arrive per epilogue warp
        ptx::mbar_init(us_empty, 1);  // the issuer's commit after a panel's last dA MMA
        ptx::st_shared_u32_volatile(abort_addr, 0);
        ptx::fence_barrier_init();
        if (p.want_da) {
            ptx::prefetch_tmap(&tmX);
            ptx::prefetch_tmap(&tmDa);
        }
        ptx::prefetch_tmap(&tmDy);
        ptx::prefetch_tmap(&tmB);
        ptx::prefetch_tmap(&tmT);
        ptx::prefetch_tmap(&tmDb);
    }
    if (warp == 1) {
        ptx::tmem_alloc<1>(tmem_slot, kUdbTmemCols);
        ptx::tmem_relinquish<1>();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const uint32_t tmem_base = ptx::ld_shared_u32_volatile(tmem_slot);
    const WaitCtx wctx{abort_addr, p.status, p.timeout_ns};
    const WaitCtx wctx_epi{abort_addr, p.status, 2 * p.timeout_ns};
    const int first = static_cast<int>(blockIdx.x), stride = static_cast<int>(gridDim.x);

    if (!smem_ok) {
        // fall through to the common exit
    } else if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0, pphase = 0;
            bool ok = true;
            for (int pn = first; pn < p.panels && ok; pn += stride, pphase ^= 1u) {
                const int m0 = pn * 128;
                if (p.want_db) {  // this panel's rows of t, once
                    ok = wait_barrier(wctx, t_empty, pphase ^ 1u, 150);
                    if (!ok) break;
                    ptx::mbar_expect_tx(t_full, kUdbBBytes);
                    ptx::tma_load_2d(smem + kUdbOffT, &tmT, t_full, 0, m0);
                    ptx::tma_load_2d(smem + kUdbOffT + 8192u, &tmT, t_full, 0, m0 + 64);
                }
                for (int j = 0; j < p.tiles; ++j) {
                    ok = wait_barrier(wctx, empty_bar(stage), phase ^ 1u, 100 + stage);
                    if (!ok) break;
                    ptx::mbar_expect_tx(full_bar(stage), kUdbABytes + kUdbBBytes);
                    const uint32_t sa = smem + kUdbOffA + stage * kUdbABytes;
                    const uint32_t sb = smem + kUdbOffB + stage * kUdbBBytes;
                    // Panel pn starts at column tile pn % tiles and wraps around: with every CTA on
                    // tile 0 at the same time, all of them fetched the same rows of B and reduce-added
                    // into the same rows of dB at once (a quarter of the kernel's time went there).
                    const int c0 = ((j + pn) % p.tiles) * 128;
                    // dy tile: columns c0..+63 for rows 0..127 (16 KB), then columns c0+64..+127
                    ptx::tma_load_2d(sa, &tmDy, full_bar(stage), c0, m0);
                    ptx::tma_load_2d(sa + 8192u, &tmDy, full_bar(stage), c0, m0 + 64);
                    ptx::tma_load_2d(sa + 16384u, &tmDy, full_bar(stage), c0 + 64, m0);
                    ptx::tma_load_2d(sa + 24576u, &tmDy, full_bar(stage), c0 + 64, m0 + 64);
                    // B's rows c0..+127 (the k index of the u product), r columns
                    ptx::tma_load_2d(sb, &tmB, full_bar(stage), 0, c0);
                    ptx::tma_load_2d(sb + 8192u, &tmB, full_bar(stage), 0, c0 + 64);
                    if (++stage == S) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                // the panel's rows of x, tile by tile, through the same ring (no B rows: the panel's
                // u in shared memory is the other operand)
                for (int i = 0; i < (p.want_da ? p.xtiles : 0) && ok; ++i) {
                    ok = wait_barrier(wctx, empty_bar(stage), phase ^ 1u, 110 + stage);
                    if (!ok) break;
                    ptx::mbar_expect_tx(full_bar(stage), kUdbABytes);
                    const uint32_t sa = smem + kUdbOffA + stage * kUdbABytes;
                    const int c0 = ((i + pn) % p.xtiles) * 128;
                    ptx::tma_load_2d(sa, &tmX, full_bar(stage), c0, m0);
                    ptx::tma_load_2d(sa + 8192u, &tmX, full_bar(stage), c0, m0 + 64);
                    ptx::tma_load_2d(sa + 16384u, &tmX, full_bar(stage), c0 + 64, m0);
                    ptx::tma_load_2d(sa + 24576u, &tmX, full_bar(stage), c0 + 64, m0 + 64);
                    if (++stage == S) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (ptx::elect_one()) {
            constexpr uint32_t idesc_u = make_idesc(128, 64, false, true);   // A K-major, B MN-major
            constexpr uint32_t idesc_db = make_idesc(128, 64, true, true);   // both MN-major
            int stage = 0;
            uint32_t phase = 0, pphase = 0;
            int buf = 0;
            uint32_t bphase = 0;
            bool ok = true;
            const uint32_t u_tmem = tmem_base;
            for (int pn = first; pn < p.panels && ok; pn += stride, pphase ^= 1u) {
                ok = wait_barrier(wctx, u_empty, pphase ^ 1u, 250);  // the previous panel's u has been read
                if (!ok) break;
                if (p.want_db) {
                    ok = wait_barrier(wctx, t_full, pphase, 260);
                    if (!ok) break;
                }
                ptx::tc_fence_after();
                const uint32_t st = smem + kUdbOffT;
                for (int j = 0; j < p.tiles; ++j) {
                    ok = wait_barrier(wctx, full_bar(stage), phase, 300 + stage);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t sa = smem + kUdbOffA + stage * kUdbABytes;
                    const uint32_t sb = smem + kUdbOffB + stage * kUdbBBytes;
                    // u += dy_tile . B_rows: A K-major, 64 k per 16 KB half; B MN-major, 16 k = 2048 B
                    const uint64_t bdesc = make_smem_desc(sb, 8192, 1024);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint64_t adesc = make_smem_desc(sa + static_cast<uint32_t>(k >> 2) * 16384u, 16, 1024) +
                                               static_cast<uint64_t>((k & 3) * (32u >> 4));
                        ptx::umma_bf16<1>(u_tmem, adesc, bdesc + static_cast<uint64_t>(k * (2048u >> 4)), idesc_u,
                                          (j > 0 || k > 0) ? 1u : 0u);
                    }
                    if (p.want_db) {
                        // dB_tile = dy_tile^T . t_rows: the same bytes as an MN-major A (two 64-column
                        // chunks 16 KB apart, 16 k = 16 rows = 2048 B); the partial sum is complete
                        // after these eight MMAs
                        ok = wait_barrier(wctx, dbempty_bar(buf), bphase ^ 1u, 270 + buf);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t d_tmem = tmem_base + 64u + static_cast<uint32_t>(buf) * 64u;
                        const uint64_t adesc = make_smem_desc(sa, 16384, 1024);
                        const uint64_t tdesc = make_smem_desc(st, 8192, 1024);
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            ptx::umma_bf16<1>(d_tmem, adesc + static_cast<uint64_t>(k * (2048u >> 4)),
                                              tdesc + static_cast<uint64_t>(k * (2048u >> 4)), idesc_db, k > 0 ? 1u : 0u);
                    }
                    ptx::umma_commit<1>(empty_bar(stage));
                    if (p.want_db) {
                        ptx::umma_commit<1>(dbfull_bar(buf));
                        if (++buf == NB) {
                            buf = 0;
                            bphase ^= 1u;
                        }
                    }
                    if (++stage == S) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                ptx::umma_commit<1>(u_full);
                if (p.want_db) ptx::umma_commit<1>(t_empty);  // t's rows may be replaced once these MMAs are done
                if (p.want_da) {
                    // dA_tile^T = x_tile^T . u_panel: the x tile as an MN-major A (as the dy tile in
                    // the dB product), the panel's u from shared memory as an MN-major B
                    ok = wait_barrier(wctx, us_full, pphase, 280);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint64_t udesc = make_smem_desc(smem + kUdbOffU, 8192, 1024);
                    for (int i = 0; i < p.xtiles; ++i) {
                        ok = wait_barrier(wctx, full_bar(stage), phase, 310 + stage);
                        if (!ok) break;
                        ok = wait_barrier(wctx, dbempty_bar(buf), bphase ^ 1u, 290 + buf);
                        if (!ok) break;
                        ptx::tc_fence_after();
                        const uint32_t sa = smem + kUdbOffA + stage * kUdbABytes;
                        const uint32_t d_tmem = tmem_base + 64u + static_cast<uint32_t>(buf) * 64u;
                        const uint64_t adesc = make_smem_desc(sa, 16384, 1024);
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            ptx::umma_bf16<1>(d_tmem, adesc + static_cast<uint64_t>(k * (2048u >> 4)),
                                              udesc + static_cast<uint64_t>(k * (2048u >> 4)), idesc_db, k > 0 ? 1u : 0u);
                        ptx::umma_commit<1>(empty_bar(stage));
                        ptx::umma_commit<1>(dbfull_bar(buf));
                        if (++buf == NB) {
                            buf = 0;
                            bphase ^= 1u;
                        }
                        if (++stage == S) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    ptx::umma_commit<1>(us_empty);  // the panel's u in shared memory may be replaced
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;  // TMEM lanes 32 q .. 32 q + 31
        const int ew = warp - 2;
        const uint32_t stg = smem + kUdbOffStg + static_cast<uint32_t>(ew) * 2u * 4096u;
        const uint32_t lane_off = static_cast<uint32_t>(lane) * 128u;
        const uint32_t sw = static_cast<uint32_t>(lane & 7);
        auto chunk_pos = [&](int chunk) { return lane_off + ((static_cast<uint32_t>(chunk) ^ sw) << 4); };
        int buf = 0;
        uint32_t bphase = 0, pphase = 0;
        uint32_t box = 0;
        bool ok = true;
        for (int pn = first; pn < p.panels && ok; pn += stride, pphase ^= 1u) {
            if (p.want_db) {
                for (int j = 0; j < p.tiles; ++j) {
                    bool w = true;
                    if (lane == 0) w = wait_barrier(wctx_epi, dbfull_bar(buf), bphase, 400 + buf);
                    ok = __shfl_sync(0xffffffffu, w ? 1 : 0, 0) != 0;
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + 64u +
                                           static_cast<uint32_t>(buf) * 64u;
                    // rows = 32 of the tile's 128 columns of dy (rows of dB), columns = r (<= 64)
                    for (int c = 0; c < p.r; c += 32) {
                        uint32_t r32[32];
                        if (p.r <= 16) {  // half the columns are enough; the rest of the box is clipped by the copy
                            uint32_t r16[16];
                            ptx::tmem_ld_32x16_wait(t_acc, r16);
#pragma unroll
                            for (int i = 0; i < 16; ++i) r32[i] = r16[i];
#pragma unroll
                            for (int i = 16; i < 32; ++i) r32[i] = 0u;
                        } else {
                            ptx::tmem_ld_32x32_wait(t_acc + static_cast<uint32_t>(c), r32);
                        }
                        const uint32_t fb = stg + (box & 1u) * 4096u;
                        ++box;
                        ptx::bulk_wait_group_read<1>();
                        __syncwarp();
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            ptx::st_shared_v4(fb + chunk_pos(i), r32[i * 4], r32[i * 4 + 1], r32[i * 4 + 2], r32[i * 4 + 3]);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (ptx::elect_one()) {
                            const int y = ((j + pn) % p.tiles) * 128 + q * 32;  // the producer's tile order
                            if (y < p.OC) ptx::tma_reduce_add_2d(&tmDb, fb, c, y);
                            ptx::bulk_commit_group();
                        }
                        __syncwarp();
                    }
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(dbempty_bar(buf));
                    __syncwarp();
                    if (++buf == NB) {
                        buf = 0;
                        bphase ^= 1u;
                    }
                }
                if (!ok) break;
            }
            // the panel's u: rows = 32 of its 128 rows, r columns, scaled and rounded once
            bool w = true;
            if (lane == 0) w = wait_barrier(wctx_epi, u_full, pphase, 450);
            ok = __shfl_sync(0xffffffffu, w ? 1 : 0, 0) != 0;
            if (!ok) break;
            ptx::tc_fence_after();
            const long long row = static_cast<long long>(pn) * 128 + q * 32 + lane;
            if (p.want_da) {  // the previous panel's dA MMAs have read the shared copy of its u
                bool w2 = true;
                if (lane == 0) w2 = wait_barrier(wctx_epi, us_empty, pphase ^ 1u, 460);
                ok = __shfl_sync(0xffffffffu, w2 ? 1 : 0, 0) != 0;
                if (!ok) break;
            }
            for (int c = 0; c < (p.want_da ? 64 : p.r); c += 32) {
                uint32_t r32[32];
                ptx::tmem_ld_32x32_wait(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(c), r32);
                if (p.want_da) {
                    // row q*32 + lane of the u tile: 64 bf16 = eight 16-byte pieces, 128-byte swizzle
                    // (columns beyond r are the zeros the TMA filled B with)
                    const uint32_t urow = smem + kUdbOffU + static_cast<uint32_t>(q * 32 + lane) * 128u;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t piece = static_cast<uint32_t>((c >> 3) + i);
                        ptx::st_shared_v4(urow + ((piece ^ sw) << 4),
                                          ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 0]), p.alpha * __uint_as_float(r32[i * 8 + 1])),
                                          ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 2]), p.alpha * __uint_as_float(r32[i * 8 + 3])),
                                          ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 4]), p.alpha * __uint_as_float(r32[i * 8 + 5])),
                                          ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 6]), p.alpha * __uint_as_float(r32[i * 8 + 7])));
                    }
                }
                if (c >= p.r) continue;
                if (row < p.BT) {
                    __nv_bfloat16 *dst = p.u + row * p.u_ld + c;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (c + i * 8 < p.r) {  // r is a multiple of 8: whole 16-byte pieces
                            uint4 v;
                            v.x = ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 0]), p.alpha * __uint_as_float(r32[i * 8 + 1]));
                            v.y = ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 2]), p.alpha * __uint_as_float(r32[i * 8 + 3]));
                            v.z = ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 4]), p.alpha * __uint_as_float(r32[i * 8 + 5]));
                            v.w = ptx::pack_bf16x2(p.alpha * __uint_as_float(r32[i * 8 + 6]), p.alpha * __uint_as_float(r32[i * 8 + 7]));
                            *reinterpret_cast<uint4 *>(dst + i * 8) = v;
                        }
                    }
                }
            }
            if (p.want_da) ptx::fence_proxy_async_smem();  // the MMAs read the shared copy through the async proxy
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (p.want_da) ptx::mbar_arrive(us_full);
                ptx::mbar_arrive(u_empty);
            }
            __syncwarp();
            if (p.want_da) {
                // 128 columns of dA per x tile, transposed in TMEM: this warp's lanes are 32 columns c of
                // x, its registers the rows j of dA. Staged as box row j, column lane (a warp-wide store
                // fills one 128-byte row: no bank conflicts), then reduce-added as a 32 x 32 box.
                for (int i = 0; i < p.xtiles; ++i) {
                    bool w3 = true;
                    if (lane == 0) w3 = wait_barrier(wctx_epi, dbfull_bar(buf), bphase, 470 + buf);
                    ok = __shfl_sync(0xffffffffu, w3 ? 1 : 0, 0) != 0;
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + 64u +
                                           static_cast<uint32_t>(buf) * 64u;
                    for (int jb = 0; jb < p.r; jb += 32) {
                        uint32_t r32[32];
                        ptx::tmem_ld_32x32_wait(t_acc + static_cast<uint32_t>(jb), r32);
                        const uint32_t fb = stg + (box & 1u) * 4096u;
                        ++box;
                        ptx::bulk_wait_group_read<1>();
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            ptx::st_shared_u32(fb + static_cast<uint32_t>(j) * 128u +
                                                   (((static_cast<uint32_t>(lane) >> 2) ^ static_cast<uint32_t>(j & 7)) << 4) +
                                                   (static_cast<uint32_t>(lane) & 3u) * 4u,
                                               r32[j]);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (ptx::elect_one()) {
                            const int x = ((i + pn) % p.xtiles) * 128 + q * 32;
                            if (x < p.C) ptx::tma_reduce_add_2d(&tmDa, fb, x, jb);
                            ptx::bulk_commit_group();
                        }
                        __syncwarp();
                    }
                    ptx::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(dbempty_bar(buf));
                    __syncwarp();
                    if (++buf == NB) {
                        buf = 0;
                        bphase ^= 1u;
                    }
                }
                if (!ok) break;
            }
        }
        ptx::bulk_wait_group<0>();
        __syncwarp();
    }

    // ---------------------------------------------------------------- common exit
    if (ptx::ld_shared_u32_volatile(abort_addr) != 0) {
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    __syncwarp();
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<1>(tmem_base, kUdbTmemCols);
    }
}

}  // namespace nb
