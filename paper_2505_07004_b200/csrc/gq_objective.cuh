// Objective of Eq. 7 on the tensor cores:  loss_k = <H_k, Delta_k^T Delta_k>  with
//
//     D_k[a][b] = sum_terms sum_j  A_term[k][j][a] * B_term[k][j][b]        (j: output channels of group k)
//
// where Delta = W - W_hat is held as two bf16 matrices (hi + lo) and the three terms hi^T hi + hi^T lo +
// lo^T hi are accumulated into the same tensor-memory tile, and with the symmetry of H_k
//
//     loss_k = sum_{a <= b} (2 - [a == b]) * D_k[a][b] * H_k[a][b].
//
// Operands are row-major bf16 matrices whose rows are the contraction index (output channels) and whose
// columns are the d_in input features, so both MMA operands are "MN-major" (feature-contiguous).
// CTA pairs, 256 x 256 tiles and the work distribution are described in gq_pipeline.cuh; work unit =
// (upper-triangular tile, group), whole units only (each unit writes its own partial sums, so the result is
// reproducible).  Roles inside a CTA:
//   warp 0 (one lane)  TMA producer: 64-row x 64-feature boxes, 128-byte swizzle, ring of OBJ_STAGES stages;
//                      byte counts of both CTAs are collected on the first CTA's "full" barriers
//   warp 1 (one lane)  MMA issuer (first CTA of the pair only); its commits signal both CTAs
//   warp 2             TMEM allocation / release (all 512 columns: two 256-column accumulators)
//   warps 4..7         epilogue: tcgen05.ld the finished accumulator, multiply with the H_k tile read from
//                      global memory, fp64 partial sum per (unit, CTA, warp); runs while the next tile is
//                      computed into the other accumulator
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
constexpr int MAX_TERMS = 3;
constexpr int PARTIALS_PER_UNIT = 8;                   // one fp64 per (CTA of the pair, epilogue warp)

struct ObjectiveParams {
    int d;                   // number of features (d_in)
    int rows;                // contraction length of every term
    int g;                   // groups
    int nj;                  // ceil(d / 256): tile blocks per side
    int raster;              // edge (in tiles) of the super-blocks of the tile order
    int n_terms;
    int term_a[MAX_TERMS];   // which tensor map (0/1) feeds A / B in each term
    int term_b[MAX_TERMS];
    int map_grouped[2];      // 1: the map's third coordinate is the group index; 0: always 0
    Schedule sched;          // units = (number of upper-triangular 256 x 256 tiles) * g,
                             // ksteps = n_terms * ceil(rows / 64)
    const float *H;          // [g][d][d], only a <= b is read
    double *partials;        // [units][PARTIALS_PER_UNIT]
    uint32_t *status;        // device status word (4 x u32)
    unsigned long long wait_budget_ns;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(OBJ_THREADS, 1)
objective_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1, const ObjectiveParams p)
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
            int ti, tj;
            tile_of_slot_blocked(w.unit / p.g, p.nj, p.raster, ti, tj);
            const int k = w.unit % p.g;
            const int a0 = ti * TILE_M + static_cast<int>(rank) * CTA_ROWS;
            const int b0 = tj * TILE_N + static_cast<int>(rank) * CTA_ROWS;
            for (int ks = w.ks0; ks < w.ks1; ++ks) {
                const int term = ks / kblocks;
                const int r = ks - term * kblocks;
                const int ma = p.term_a[term], mb = p.term_b[term];
                const void *amap = ma ? static_cast<const void *>(&map1) : static_cast<const void *>(&map0);
                const void *bmap = mb ? static_cast<const void *>(&map1) : static_cast<const void *>(&map0);
                const int ka = p.map_grouped[ma] ? k : 0;
                const int kb = p.map_grouped[mb] ? k : 0;
                if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, w.unit)) { ok = false; break; }
                const uint32_t full_local = smem_u32(&bar_full[s]);
                if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * OBJ_STAGE_BYTES);   // both CTAs' bytes
                const uint32_t full = map_to_cta(full_local, 0);
                const uint32_t sa = ring + s * OBJ_STAGE_BYTES;
                const uint32_t sb = sa + OBJ_A_BYTES;
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sa + q * BOX_BYTES, amap, full, a0 + q * BOX_FEATURES, r * TILE_K, ka);
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sb + q * BOX_BYTES, bmap, full, b0 + q * BOX_FEATURES, r * TILE_K, kb);
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
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[buf]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * TILE_N);
            for (int ks = w.ks0; ks < w.ks1; ++ks) {
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t sa = ring + s * OBJ_STAGE_BYTES;
                const uint32_t sb = sa + OBJ_A_BYTES;
#pragma unroll
                for (int kk = 0; kk < TILE_K / 16; ++kk) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + kk * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + kk * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != w.ks0 || kk != 0) ? 1u : 0u);
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
            int ti, tj;
            tile_of_slot_blocked(w.unit / p.g, p.nj, p.raster, ti, tj);
            const int k = w.unit % p.g;
            ok = bounded_wait(smem_u32(&bar_acc_full[buf]), acc_ph, wc, 4u, w.unit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int row0 = ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
            const int row = row0 + lane;
            const bool row_ok = row < p.d;
            const float *hrow = p.H + (static_cast<size_t>(k) * p.d + (row_ok ? row : 0)) * static_cast<size_t>(p.d);
            double dsum = 0.0;
#pragma unroll 1
            for (int cc = 0; cc < TILE_N / 32; ++cc) {
                const int col0 = tj * TILE_N + cc * 32;
                if (col0 >= p.d) break;                    // right of the matrix
                if (col0 + 32 <= row0) continue;           // 32 x 32 block strictly below the diagonal
                if (row0 >= p.d) break;                    // below the matrix
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                  static_cast<uint32_t>(buf * TILE_N + cc * 32), r);
                tmem_ld_wait();
                if (!row_ok) continue;
                {
                    float part = 0.0f;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const int c = col0 + v * 4;
                        if (c < p.d && c + 3 >= row) {
                            const float4 h = __ldg(reinterpret_cast<const float4 *>(hrow + c));
                            const float hv[4] = {h.x, h.y, h.z, h.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float wgt = (c + e > row) ? 2.0f : ((c + e == row) ? 1.0f : 0.0f);
                                part = fmaf(wgt * __uint_as_float(r[v * 4 + e]), hv[e], part);
                            }
                        }
                    }
                    dsum += static_cast<double>(part);
                }
            }
            // This warp has read all it needs from the accumulator: tell the MMA issuer (first CTA).
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
            {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                if (lane == 0)
                    p.partials[static_cast<size_t>(w.unit) * PARTIALS_PER_UNIT + rank * 4 + q] = dsum;
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
