// Pair GEMM: the tensor-core kernel behind gq_objective (Eq. 7) and behind the panel products of the
// coordinate-descent cycles (Appendix B.2, Algorithm 4).  Both are sums over a contraction index of
// products of MN-major bf16 operands (rows = contraction index, contiguous columns = the output index),
//
//     D[a][b] = sum_terms sum_r  A_term[r][a] * B_term[r][b],
//
// with fp32 values carried as two bf16 matrices (hi + lo) and the three terms hi hi + hi lo + lo hi
// accumulated into the same tensor-memory tile.  CTA pairs, 256 x 256 tiles and the work distribution are
// described in gq_pipeline.cuh.  Roles inside a CTA:
//   warp 0 (one lane)  TMA producer: 64-row x 64-feature boxes, 128-byte swizzle, ring of OBJ_STAGES stages;
//                      byte counts of both CTAs are collected on the first CTA's "full" barriers
//   warp 1 (one lane)  MMA issuer (first CTA of the pair only); its commits signal both CTAs
//   warp 2             TMEM allocation / release (all 512 columns: two 256-column accumulators)
//   warps 4..7         epilogue: tcgen05.ld the finished accumulator while the next tile is computed into
//                      the other accumulator
//
// MODE_OBJECTIVE   loss_k = <H_k, Delta_k^T Delta_k>: A, B = Delta = W - W_hat of group k (rows = output
//                  channels), upper-triangular tiles only, epilogue
//                  sum_{a <= b} (2 - [a == b]) * D[a][b] * H_k[a][b] as one fp64 partial per (unit, CTA, warp);
//                  whole units only, so the result is reproducible.
// MODE_PANEL       P[r][ch] += sum_{c outside the block} H_k[c][s0 + r] * E[c][ch] for the 256 rows of one
//                  coordinate block: A = H_k (rows = contraction index c, by symmetry H[c][r] = H[r][c]),
//                  B = E = (What - W)^T (rows = input coordinates c, columns = output channels); work unit =
//                  (group, tile of 256 channels, piece of the contraction range); the pieces of a tile are
//                  added into P with red.global.add.
// MODE_FULL        C[r][col] = sum_c A[c][r] * B[c][col], a plain product of MN-major operands (used by the
//                  LNQ codebook step: A = H_k split three ways, B = W^T or one-hot assignment columns); work
//                  unit = (256-row block, 256-column tile), each unit stores its tile.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_pipeline.cuh"

namespace gq {

constexpr int OBJ_STAGES = 6;
constexpr int OBJ_A_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;
constexpr int OBJ_B_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;
constexpr int OBJ_STAGE_BYTES = OBJ_A_BYTES + OBJ_B_BYTES;
constexpr int OBJ_THREADS = 256;
constexpr int OBJ_SMEM_BYTES = OBJ_STAGES * OBJ_STAGE_BYTES + 1024;   // + slack to align the ring to 1024 B
constexpr int MAX_TERMS = 6;
constexpr int MAX_MAPS = 6;
constexpr int PARTIALS_PER_UNIT = 8;                   // one fp64 per (CTA of the pair, epilogue warp)

constexpr int MODE_OBJECTIVE = 0;
constexpr int MODE_PANEL = 1;
constexpr int MODE_FULL = 2;

struct PairGemmParams {
    int d;                   // number of features (d_in)
    int rows;                // MODE_OBJECTIVE: contraction length of every term
    int g;                   // groups
    int nj;                  // ceil(d / 256): tile blocks per side
    int raster;              // edge (in tiles) of the super-blocks of the tile order
    int n_terms;
    int term_a[MAX_TERMS];   // which of the six tensor maps feeds A / B in each term
    int term_b[MAX_TERMS];
    int map_grouped[MAX_MAPS];   // 1: the map's third coordinate is the group index; 0: always 0
    Schedule sched;          // units = (number of upper-triangular 256 x 256 tiles) * g,
                             // ksteps = n_terms * ceil(rows / 64)
    const float *H;          // MODE_OBJECTIVE: [g][d][d], only a <= b is read
    double *partials;        // MODE_OBJECTIVE: [units][PARTIALS_PER_UNIT]
    // MODE_PANEL
    int s0;                  // first coordinate of the block
    int blk_ksteps;          // 64-row k-steps covered by the block itself (left out of the contraction)
    int nk;                  // 64-row k-steps outside the block (per term)
    int ch_tiles;            // tiles of 256 channels per group
    int pieces;              // pieces of the contraction range per (group, channel tile); sched.ksteps each
    int mk;                  // channels per group
    int d_out;
    float *P;                // [256][d_out]
    // MODE_FULL: C[r][col - col0] = sum over all `rows` contraction rows, r < d, col0 <= col < col0 + cols
    int full_k;              // group index given to the grouped maps
    int col0, cols;          // B columns of this launch
    int col_tiles;           // ceil(cols / 256)
    float *C;                // output, row stride ldc (floats), written (not added)
    long long ldc;
    uint32_t *status;        // device status word (4 x u32)
    unsigned long long wait_budget_ns;
};

// Where a work item's operands start and which k-steps it covers.
struct ItemGeom {
    int ti, tj;      // MODE_OBJECTIVE: tile
    int k;           // group
    int a0, b0;      // first A / B column this CTA loads
    int ks0, ks1;    // k-steps [ks0, ks1) of the flattened (term, row block) range
};

template <int MODE>
__device__ __forceinline__ bool item_geom(const PairGemmParams &p, const WorkItem &w, uint32_t rank, ItemGeom &ge)
{
    if (MODE == MODE_OBJECTIVE) {
        tile_of_slot_blocked(w.unit / p.g, p.nj, p.raster, ge.ti, ge.tj);
        ge.k = w.unit % p.g;
        ge.a0 = ge.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS;
        ge.b0 = ge.tj * TILE_N + static_cast<int>(rank) * CTA_ROWS;
        ge.ks0 = w.ks0;
        ge.ks1 = w.ks1;
        return true;
    }
    if (MODE == MODE_FULL) {
        ge.ti = w.unit / p.col_tiles;
        ge.tj = w.unit % p.col_tiles;
        ge.k = p.full_k;
        ge.a0 = ge.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS;
        ge.b0 = p.col0 + ge.tj * TILE_N + static_cast<int>(rank) * CTA_ROWS;
        ge.ks0 = w.ks0;
        ge.ks1 = w.ks1;
        return true;
    }
    const int piece = w.unit % p.pieces;
    const int t = (w.unit / p.pieces) % p.ch_tiles;
    ge.k = w.unit / (p.pieces * p.ch_tiles);
    ge.ti = 0;
    ge.tj = t;
    ge.a0 = p.s0 + static_cast<int>(rank) * CTA_ROWS;
    ge.b0 = ge.k * p.mk + t * TILE_N + static_cast<int>(rank) * CTA_ROWS;
    ge.ks0 = piece * p.sched.ksteps;
    const int total = p.n_terms * p.nk;
    ge.ks1 = (ge.ks0 + p.sched.ksteps < total) ? ge.ks0 + p.sched.ksteps : total;
    return ge.ks1 > ge.ks0;          // a piece beyond the end of the range has nothing to do: every role skips it
}

// Term and first contraction row of flattened k-step ks.
template <int MODE>
__device__ __forceinline__ void kstep_coords(const PairGemmParams &p, int ks, int kblocks, int &term, int &row)
{
    if (MODE != MODE_PANEL) {
        term = ks / kblocks;
        row = (ks - term * kblocks) * TILE_K;
    } else {
        term = ks / p.nk;
        const int kb = ks - term * p.nk;
        row = (kb < p.s0 / TILE_K ? kb : kb + p.blk_ksteps) * TILE_K;
    }
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(OBJ_THREADS, 1)
pair_gemm_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
                 const __grid_constant__ CUtensorMap map2, const __grid_constant__ CUtensorMap map3,
                 const __grid_constant__ CUtensorMap map4, const __grid_constant__ CUtensorMap map5,
                 const PairGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[OBJ_STAGES];      // used in the pair's first CTA only
    __shared__ __align__(8) uint64_t bar_empty[OBJ_STAGES];     // signalled in both CTAs by the MMA commits
    __shared__ __align__(8) uint64_t bar_acc_full[2];       // signalled in both CTAs by the MMA commits
    __shared__ __align__(8) uint64_t bar_acc_empty[2];      // first CTA only: 8 epilogue warps arrive
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile uint32_t abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                // 0: issues the MMAs; 1: its peer
    const int pair = static_cast<int>(blockIdx.x >> 1);
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < OBJ_STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 8);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&map0);
        prefetch_tensormap(&map1);
        prefetch_tensormap(&map2);
        prefetch_tensormap(&map3);
        prefetch_tensormap(&map4);
        prefetch_tensormap(&map5);
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(&tmem_base_smem), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    cluster_sync_all();          // barriers initialised and TMEM allocated in both CTAs before any remote access
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_smem;

    const WaitCtx wc{&abort_flag, p.status, p.wait_budget_ns};
    const int kblocks = (p.rows + TILE_K - 1) / TILE_K;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        int s = 0;
        uint32_t ph = 0;
        uint32_t issued = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            ItemGeom ge;
            if (!item_geom<MODE>(p, w, rank, ge)) continue;
            const void *maps[MAX_MAPS] = {&map0, &map1, &map2, &map3, &map4, &map5};
            for (int ks = ge.ks0; ks < ge.ks1; ++ks) {
                int term, row;
                kstep_coords<MODE>(p, ks, kblocks, term, row);
                const int ma = p.term_a[term], mb = p.term_b[term];
                const void *amap = maps[ma];
                const void *bmap = maps[mb];
                const int ka = p.map_grouped[ma] ? ge.k : 0;
                const int kb = p.map_grouped[mb] ? ge.k : 0;
                if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, w.unit)) { ok = false; break; }
                const uint32_t full_local = smem_u32(&bar_full[s]);
                if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * OBJ_STAGE_BYTES);   // both CTAs' bytes
                const uint32_t full = map_to_cta(full_local, 0);
                const uint32_t sa = ring + s * OBJ_STAGE_BYTES;
                const uint32_t sb = sa + OBJ_A_BYTES;
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sa + q * BOX_BYTES, amap, full, ge.a0 + q * BOX_FEATURES, row, ka);
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sb + q * BOX_BYTES, bmap, full, ge.b0 + q * BOX_FEATURES, row, kb);
                ++issued;
                if (++s == OBJ_STAGES) { s = 0; ph ^= 1u; }
            }
        }
        // Stay until every stage that was filled has been released again: the release is an arrival on
        // this CTA's barriers, which must not come after the CTA has gone.
        // (Stages that were never filled pass at once.)
        for (int q = 0; ok && issued != 0u && q < OBJ_STAGES; ++q) {
            if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 5u, 0u)) ok = false;
            if (++s == OBJ_STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) spin_ns(1000000ull);      // copies already issued land well within this time
    } else if (warp == 1 && lane == 0 && rank == 0) {
        // ------------------------------------------------------------------ MMA issuer (first CTA)
        constexpr uint32_t idesc = umma_idesc_bf16_mn(TILE_M, TILE_N);
        int s = 0;
        uint32_t ph = 0;
        int buf = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            ItemGeom ge;
            if (!item_geom<MODE>(p, w, rank, ge)) continue;
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[buf]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * TILE_N);
            for (int ks = ge.ks0; ks < ge.ks1; ++ks) {
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t sa = ring + s * OBJ_STAGE_BYTES;
                const uint32_t sb = sa + OBJ_A_BYTES;
#pragma unroll
                for (int kk = 0; kk < TILE_K / 16; ++kk) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + kk * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + kk * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != ge.ks0 || kk != 0) ? 1u : 0u);
                }
                umma_commit_pair(smem_u32(&bar_empty[s]));   // stage reusable in both CTAs once these MMAs have read it
                if (++s == OBJ_STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
            umma_commit_pair(smem_u32(&bar_acc_full[buf]));
            buf ^= 1;
            if (buf == 0) acc_ph ^= 1u;
        }
        if (!ok) {
            // Make sure no MMA is still writing TMEM when it is released.
            umma_commit_local(smem_u32(&bar_drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&bar_drain), 0u) && global_timer_ns() - t0 < 5000000ull) {}
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue (128 threads, both CTAs)
        const int q = warp & 3;                 // TMEM lane quarter this warp may access
        int buf = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            ItemGeom ge;
            if (!item_geom<MODE>(p, w, rank, ge)) continue;
            if (MODE == MODE_OBJECTIVE) {
                // The H values this warp needs do not depend on the accumulator: the first block's are requested
                // before the wait for the MMAs, every other block's while the block before it is being used.
                const int ti = ge.ti, tj = ge.tj, k = ge.k;
                const int row0 = ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
                const int row = row0 + lane;
                const bool row_ok = row < p.d;
                const float *hrow = p.H + (static_cast<size_t>(k) * p.d + (row_ok ? row : 0)) * static_cast<size_t>(p.d);
                auto block_active = [&](int cc) {
                    const int col0 = tj * TILE_N + cc * 32;
                    return col0 < p.d && row0 < p.d && col0 + 32 > row0;      // inside the matrix, not below the diagonal
                };
                auto load_block = [&](int cc, float4 (&h)[8]) {
                    const int col0 = tj * TILE_N + cc * 32;
                    const bool act = row_ok && block_active(cc);
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const int c = col0 + v * 4;
                        h[v] = (act && c < p.d && c + 3 >= row) ? __ldg(reinterpret_cast<const float4 *>(hrow + c))
                                                                : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                };
                float4 hq[2][8];
                load_block(0, hq[0]);
                ok = bounded_wait(smem_u32(&bar_acc_full[buf]), acc_ph, wc, 4u, w.unit);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                double dsum = 0.0;
#pragma unroll
                for (int cc = 0; cc < TILE_N / 32; ++cc) {
                    if (cc + 1 < TILE_N / 32) load_block(cc + 1, hq[(cc + 1) & 1]);
                    if (!block_active(cc)) continue;           // uniform over the warp
                    const int col0 = tj * TILE_N + cc * 32;
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                      static_cast<uint32_t>(buf * TILE_N + cc * 32), r);
                    tmem_ld_wait();
                    float part = 0.0f;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const int c = col0 + v * 4;
                        const float4 h = hq[cc & 1][v];        // zero where it was not loaded
                        const float hv[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float wgt = (c + e > row) ? 2.0f : ((c + e == row) ? 1.0f : 0.0f);
                            part = fmaf(wgt * __uint_as_float(r[v * 4 + e]), hv[e], part);
                        }
                    }
                    dsum += static_cast<double>(part);
                }
                // This warp has read all it needs from the accumulator: tell the MMA issuer (first CTA).
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                if (lane == 0)
                    p.partials[static_cast<size_t>(w.unit) * PARTIALS_PER_UNIT + rank * 4 + q] = dsum;
                buf ^= 1;
                if (buf == 0) acc_ph ^= 1u;
                continue;
            }
            ok = bounded_wait(smem_u32(&bar_acc_full[buf]), acc_ph, wc, 4u, w.unit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            if (MODE == MODE_OBJECTIVE) {
            } else if (MODE == MODE_FULL) {
                const int row0 = ge.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
                const int row = row0 + lane;
                float *crow = p.C + static_cast<size_t>(row < p.d ? row : 0) * p.ldc;
#pragma unroll 1
                for (int cc = 0; cc < TILE_N / 32; ++cc) {
                    const int c0 = ge.tj * TILE_N + cc * 32;                           // column relative to col0
                    if (c0 >= p.cols || row0 >= p.d) break;
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                      static_cast<uint32_t>(buf * TILE_N + cc * 32), r);
                    tmem_ld_wait();
                    if (row >= p.d) continue;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        if (c0 + v * 4 < p.cols)
                            *reinterpret_cast<float4 *>(crow + c0 + v * 4) =
                                make_float4(__uint_as_float(r[v * 4 + 0]), __uint_as_float(r[v * 4 + 1]),
                                            __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
            } else {
                const int rl = static_cast<int>(rank) * CTA_ROWS + q * 32 + lane;      // row inside the block
                const bool row_ok = p.s0 + rl < p.d;
                const int ch_end = (ge.k + 1) * p.mk;                                  // channels of this group only
                float *prow = p.P + static_cast<size_t>(rl) * p.d_out;
#pragma unroll 1
                for (int cc = 0; cc < TILE_N / 32; ++cc) {
                    const int ch0 = ge.k * p.mk + ge.tj * TILE_N + cc * 32;
                    if (ch0 >= ch_end) break;
                    if (p.s0 + static_cast<int>(rank) * CTA_ROWS + q * 32 >= p.d) break;
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                      static_cast<uint32_t>(buf * TILE_N + cc * 32), r);
                    tmem_ld_wait();
                    if (!row_ok) continue;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        if (ch0 + v * 4 < ch_end)
                            red_add_f32x4(prow + ch0 + v * 4, __uint_as_float(r[v * 4 + 0]), __uint_as_float(r[v * 4 + 1]),
                                          __uint_as_float(r[v * 4 + 2]), __uint_as_float(r[v * 4 + 3]));
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
            }
            buf ^= 1;
            if (buf == 0) acc_ph ^= 1u;
        }
    }

    // Both CTAs stay until neither can touch the other's shared memory, barriers or tensor memory any more.
    __syncwarp();
    tc_fence_before_sync();
    cluster_sync_all();
    if (warp == 2) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace gq
