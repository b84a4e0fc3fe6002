// Wide pair GEMM: C[r][col] = sum_terms sum_c A_term[c][r] * B_term[c][col] for MN-major bf16 operands, the
// large product of the LNQ codebook step (Section 4.2, Eq. 8: H_k times the one-hot assignment columns).
//
// pair_gemm_kernel<MODE_FULL> computes one 256 x 256 tile per unit and loads 128 A rows and 128 B columns per
// CTA and k-step for four MMAs: 64 bytes from L2 per SM and tensor-core clock, more than the L2 delivers to 148
// SMs at once.  Here a unit is a 256-row block times TWO neighbouring 256-column tiles, as in the guided-Hessian
// kernel's wide units: the stage holds [B(tile 0) | A | B(tile 1)], the A block serves both accumulators, and
// the traffic per MMA drops by a quarter.  The two accumulators fill tensor memory, so the read-out is not
// hidden behind the next unit except for its first k-steps (same scheme as in gq_hessian.cuh), which the long
// contraction (all of d_in, two terms) makes affordable.
//
// (The objective of Eq. 7 runs on units of the same shape in a kernel of its own, gq_gram_dot.cuh.)
//
// Roles: warp 0 (one lane) TMA producer, warp 1 (one lane, first CTA) MMA issuer, warp 2 TMEM allocation,
// warps 4..11 epilogue (tcgen05.ld, plain 16-byte stores; whole units only, one writer per element).
// Every mbarrier wait is bounded (gq_pipeline.cuh).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_objective.cuh"
#include "gq_pipeline.cuh"

namespace gq {

constexpr int WG_STAGES = 4;
constexpr int WG_SLOT_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;      // one operand block: 16 KB
constexpr int WG_STAGE_BYTES = 3 * WG_SLOT_BYTES;                         // [B0 | A | B1]
constexpr int WG_EPI_WARPS = 8;
constexpr int WG_THREADS = 32 * (4 + WG_EPI_WARPS);
constexpr int WG_SMEM_BYTES = WG_STAGES * WG_STAGE_BYTES + 1024;
constexpr int WG_FULL = 0;

struct WideUnit {
    int ti;          // row block
    int tj[2];       // column tile of accumulator 0 / 1
    bool use[2];
    int k;           // third coordinate of the grouped maps
};

// Uses the MODE_FULL fields of PairGemmParams (d, rows, n_terms, term_a/b, map_grouped, full_k, col0, cols,
// col_tiles, C, ldc), units = row blocks * ceil(col_tiles / 2), sched.ksteps = n_terms * ceil(rows / 64).
template <int WMODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(WG_THREADS, 1)
wide_gemm_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1,
                 const __grid_constant__ CUtensorMap map2, const __grid_constant__ CUtensorMap map3,
                 const __grid_constant__ CUtensorMap map4, const __grid_constant__ CUtensorMap map5,
                 const PairGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[WG_STAGES];     // first CTA: bytes of both CTAs
    __shared__ __align__(8) uint64_t bar_empty[WG_STAGES];    // both CTAs: signalled by the MMA commits
    __shared__ __align__(8) uint64_t bar_acc_full;            // both CTAs: signalled by the MMA commit
    __shared__ __align__(8) uint64_t bar_acc_empty[2];        // first CTA, one per accumulator: 16 epilogue warps arrive
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile uint32_t abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = static_cast<int>(blockIdx.x >> 1);
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < WG_STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc_full), 1);
        for (int kk = 0; kk < 2; ++kk) mbar_init(smem_u32(&bar_acc_empty[kk]), 2 * WG_EPI_WARPS);
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
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_smem;
    const WaitCtx wc{&abort_flag, p.status, p.wait_budget_ns};
    const int kblocks = (p.rows + TILE_K - 1) / TILE_K;
    const int col_pairs = (p.col_tiles + 1) / 2;

    auto decode = [&](int unit) {
        WideUnit u;
        u.ti = unit / col_pairs;
        u.tj[0] = 2 * (unit - u.ti * col_pairs);
        u.tj[1] = u.tj[0] + 1;
        u.use[0] = true;
        u.use[1] = u.tj[1] < p.col_tiles;
        u.k = p.full_k;
        return u;
    };
    const int col_base = p.col0;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        int s = 0;
        uint32_t ph = 0;
        uint32_t issued = 0;
        bool ok = true;
        WorkItem w;
        const void *maps[MAX_MAPS] = {&map0, &map1, &map2, &map3, &map4, &map5};
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const WideUnit u = decode(w.unit);
            const int a0 = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS;
            const int n_ops = 1 + (u.use[0] ? 1 : 0) + (u.use[1] ? 1 : 0);
            for (int ks = w.ks0; ks < w.ks1; ++ks) {
                const int term = ks / kblocks;
                const int row = (ks - term * kblocks) * TILE_K;
                const int ma = p.term_a[term], mb = p.term_b[term];
                const int ka = p.map_grouped[ma] ? u.k : 0;
                const int kb = p.map_grouped[mb] ? u.k : 0;
                if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, w.unit)) { ok = false; break; }
                const uint32_t full_local = smem_u32(&bar_full[s]);
                if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * n_ops * WG_SLOT_BYTES);   // both CTAs' bytes
                const uint32_t full = map_to_cta(full_local, 0);
                const uint32_t stage = ring + s * WG_STAGE_BYTES;
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q) {
                    tma_load_3d_pair(stage + WG_SLOT_BYTES + q * BOX_BYTES, maps[ma], full, a0 + q * BOX_FEATURES, row, ka);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk)
                        if (u.use[kk])
                            tma_load_3d_pair(stage + (kk ? 2 * WG_SLOT_BYTES : 0) + q * BOX_BYTES, maps[mb], full,
                                             col_base + u.tj[kk] * TILE_N + static_cast<int>(rank) * CTA_ROWS + q * BOX_FEATURES,
                                             row, kb);
                }
                ++issued;
                if (++s == WG_STAGES) { s = 0; ph ^= 1u; }
            }
        }
        // Stay until every stage has been released again: the release is an arrival on this CTA's barriers,
        // which must not come after the CTA has gone.
        for (int q = 0; ok && issued != 0u && q < WG_STAGES; ++q) {
            if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 5u, 0u)) ok = false;
            if (++s == WG_STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) spin_ns(1000000ull);
    } else if (warp == 1 && lane == 0 && rank == 0) {
        // ------------------------------------------------------------------ MMA issuer (first CTA)
        constexpr uint32_t idesc = umma_idesc_bf16_mn(TILE_M, TILE_N);
        int s = 0;
        uint32_t ph = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const WideUnit u = decode(w.unit);
            auto issue = [&](int kk, int stage_idx, int ks) {
                if (!u.use[kk]) return;
                const uint32_t stage = ring + stage_idx * WG_STAGE_BYTES;
                const uint32_t sa = stage + WG_SLOT_BYTES;
                const uint32_t sb = stage + (kk ? 2 * WG_SLOT_BYTES : 0);
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(kk * TILE_N);
#pragma unroll
                for (int k16 = 0; k16 < TILE_K / 16; ++k16) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + k16 * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + k16 * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != w.ks0 || k16 != 0) ? 1u : 0u);
                }
            };
            // Accumulator 0 is emptied first: the first k-steps (as many as the ring holds) go to it as soon as
            // it is free, then to accumulator 1; afterwards two k-steps at a time per accumulator.
            const int n_head = (w.ks1 - w.ks0 < WG_STAGES) ? (w.ks1 - w.ks0) : WG_STAGES;
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[0]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            {
                int s_h = s;
                uint32_t ph_h = ph;
                for (int q = 0; q < n_head; ++q) {
                    if (!bounded_wait_hot(smem_u32(&bar_full[s_h]), ph_h, wc, 3u, w.unit)) { ok = false; break; }
                    tc_fence_after_sync();
                    issue(0, s_h, w.ks0 + q);
                    if (++s_h == WG_STAGES) { s_h = 0; ph_h ^= 1u; }
                }
            }
            if (!ok) break;
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[1]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            for (int q = 0; q < n_head; ++q) {
                issue(1, s, w.ks0 + q);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                if (++s == WG_STAGES) { s = 0; ph ^= 1u; }
            }
            int ks = w.ks0 + n_head;
            for (; ks + 1 < w.ks1; ks += 2) {
                const int s2 = (s + 1 == WG_STAGES) ? 0 : s + 1;
                const uint32_t ph2 = (s + 1 == WG_STAGES) ? (ph ^ 1u) : ph;
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                if (!bounded_wait_hot(smem_u32(&bar_full[s2]), ph2, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                issue(0, s, ks);
                issue(0, s2, ks + 1);
                issue(1, s, ks);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                issue(1, s2, ks + 1);
                umma_commit_pair(smem_u32(&bar_empty[s2]));
                s = (s2 + 1 == WG_STAGES) ? 0 : s2 + 1;
                ph = (s2 + 1 == WG_STAGES) ? (ph2 ^ 1u) : ph2;
            }
            for (; ok && ks < w.ks1; ++ks) {
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                issue(0, s, ks);
                issue(1, s, ks);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                if (++s == WG_STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
            umma_commit_pair(smem_u32(&bar_acc_full));
            acc_ph ^= 1u;
        }
        if (!ok) {
            // Make sure no MMA is still writing TMEM when it is released.
            umma_commit_local(smem_u32(&bar_drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&bar_drain), 0u) && global_timer_ns() - t0 < 5000000ull) {}
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue: C = accumulators
        const int ew = warp - 4;                        // 0..7
        const int q = warp & 3;                         // TMEM lane quarter this warp may access
        const int half = ew >> 2;                       // which 128 of the 256 accumulator columns
        uint32_t acc_ph = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const WideUnit u = decode(w.unit);
            const int row0 = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
            const int row = row0 + lane;
            if (lane == 0) ok = bounded_wait(smem_u32(&bar_acc_full), acc_ph, wc, 4u, w.unit);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            (void)mbar_try_wait(smem_u32(&bar_acc_full), acc_ph);     // every lane observes the completed phase
            tc_fence_after_sync();
            float *crow = p.C + static_cast<size_t>(row < p.d ? row : 0) * p.ldc;
            for (int kk = 0; kk < 2; ++kk) {
#pragma unroll 1
                for (int c4 = 0; u.use[kk] && c4 < 4; ++c4) {
                    const int cc = half * 4 + c4;
                    const int c0 = u.tj[kk] * TILE_N + cc * 32;            // column relative to col0
                    if (c0 >= p.cols || row0 >= p.d) break;
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                      static_cast<uint32_t>(kk * TILE_N + cc * 32), r);
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
                // This warp has read all it needs from accumulator kk: tell the MMA issuer (first CTA).
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[kk]), 0));
            }
            acc_ph ^= 1u;
        }
    }

    __syncwarp();
    tc_fence_before_sync();
    cluster_sync_all();
    if (warp == 2) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace gq
