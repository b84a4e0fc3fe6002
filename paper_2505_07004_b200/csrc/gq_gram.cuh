// Tensor-core core of libgq: upper-triangular tiles of batched Gram-type products
//
//     D_k[a][b] = sum_terms sum_r  A_term[k][r][a] * B_term[k][r][b]        (a in tile rows, b in tile columns)
//
// where every operand is a row-major bf16 matrix whose rows are the contraction index r (tokens for the
// guided Hessian of Algorithm 1 line 4, output channels for the objective of Eq. 7) and whose columns are
// the d_in input features.  Both MMA operands are therefore "MN-major" (feature-contiguous).
//
// The kernel runs as clusters of two CTAs (one CTA pair per two SMs).  A pair owns one 256 x 256 tile at a
// time: each CTA loads 128 of the tile's A rows and 128 of its B columns per 64-row k-step (32 KB instead
// of the 48 KB a lone CTA would need for a 128 x 256 tile), the first CTA of the pair issues
// tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16) for both, and each CTA holds the 128 x 256 fp32
// accumulator of its own rows in its tensor memory.  Roles inside a CTA:
//   warp 0 (one lane)  TMA producer: 64-row x 64-feature boxes, 128-byte swizzle, ring of STAGES stages;
//                      byte counts of both CTAs are collected on the first CTA's "full" barriers
//   warp 1 (one lane)  MMA issuer (first CTA of the pair only); its commits signal both CTAs
//   warp 2             TMEM allocation / release (all 512 columns: two 256-column accumulators)
//   warps 4..7         epilogue: tcgen05.ld the finished accumulator while the next tile is computed
// Epilogues:
//   EPI_ACCUM  H_k[tile] += D      (Hessian streaming)
//   EPI_DOT    partial = sum_{a<=b} (2 - [a==b]) * D[a][b] * H_k[a][b]     (objective)
//
// Work distribution: work unit = (tile, group), group fastest so that pairs that run at the same time
// share tiles of X in L2.  Units are dealt round-robin to the pairs for `full_waves` rounds; what is left
// (fewer units than pairs) is cut along the contraction index into equal pieces, one per pair, and the
// pieces of a unit are added to H with red.global.add (EPI_ACCUM only).
//
// Every wait on an mbarrier is bounded by a time budget; when it runs out the kernel records
// STATUS_TIMEOUT in the status word, all roles of that CTA leave their loops (the peer CTA's own waits
// then run out as well), in-flight copies and MMAs are given a bounded time to land, both CTAs meet at
// the final cluster barrier, TMEM is released and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_ptx.cuh"

namespace gq {

constexpr int TILE_M = 256;                            // rows of a pair's tile
constexpr int TILE_N = 256;                            // columns of a pair's tile
constexpr int CTA_ROWS = 128;                          // A rows (and B columns) one CTA loads and owns
constexpr int TILE_K = 64;
constexpr int STAGES = 6;
constexpr int BOX_FEATURES = 64;                       // 128 bytes of bf16
constexpr int BOX_BYTES = TILE_K * 128;                // one TMA box: 64 rows x 128 B
constexpr int A_STAGE_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;
constexpr int B_STAGE_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int GRAM_THREADS = 256;
constexpr int GRAM_SMEM_BYTES = STAGES * STAGE_BYTES + 1024;   // + slack to align the ring to 1024 B
constexpr uint32_t TMEM_COLS = 512;
constexpr int MAX_TERMS = 3;
constexpr int MIN_PIECE_KSTEPS = 8;                    // smallest k-range worth an epilogue of its own
constexpr int PARTIALS_PER_UNIT = 8;                   // EPI_DOT: one fp64 per (CTA of the pair, epilogue warp)

constexpr int EPI_ACCUM = 0;
constexpr int EPI_DOT = 1;

constexpr uint32_t STATUS_TIMEOUT = 6;   // stored in the status word; the host maps it to GQ_ERR_TIMEOUT

// How the work units of a launch are dealt to the CTA pairs.
struct Schedule {
    int units;               // work units of the launch
    int ksteps;              // k-steps (of 64 contraction rows) of one whole unit
    int pairs;               // CTA pairs in the grid
    int full_waves;          // rounds of whole units dealt round-robin
    int tail_units;          // units after the full rounds (0 <= tail_units < pairs), cut into pieces
    int tail_pairs;          // pairs that take a piece of the tail
};

struct GramParams {
    int d;                   // number of features (d_in)
    int rows;                // contraction length of every term
    int g;                   // groups
    int n_terms;
    int term_a[MAX_TERMS];   // which tensor map (0/1) feeds A / B in each term
    int term_b[MAX_TERMS];
    int map_grouped[2];      // 1: the map's third coordinate is the group index; 0: always 0
    Schedule sched;          // units = (number of upper-triangular 256 x 256 tiles) * g,
                             // ksteps = n_terms * ceil(rows / 64)
    float *H;                // [g][d][d]
    double *partials;        // EPI_DOT: [units][PARTIALS_PER_UNIT]
    uint32_t *status;        // device status word (4 x u32)
    unsigned long long wait_budget_ns;
};

// Host side: fills the distribution fields.  `balanced` cuts the last, incomplete round into pieces.
inline Schedule plan_schedule(int units, int ksteps, int pairs, bool balanced)
{
    Schedule p;
    p.units = units;
    p.ksteps = ksteps;
    p.pairs = pairs;
    p.full_waves = (units + pairs - 1) / pairs;
    p.tail_units = 0;
    p.tail_pairs = 0;
    if (balanced && units % pairs != 0) {
        p.full_waves = units / pairs;
        p.tail_units = units - p.full_waves * pairs;
        const long long total = static_cast<long long>(p.tail_units) * ksteps;
        long long tp = total / MIN_PIECE_KSTEPS;
        if (tp < 1) tp = 1;
        if (tp > pairs) tp = pairs;
        p.tail_pairs = static_cast<int>(tp);
    }
    return p;
}

// Slot t of the triangular enumeration -> (row block i, column block j) of 256 x 256 tiles with i <= j,
// column blocks outermost.
__device__ __forceinline__ void tile_of_slot(int t, int &i, int &j)
{
    int jj = static_cast<int>((sqrtf(8.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
    while (jj * (jj + 1) / 2 > t) --jj;
    while ((jj + 1) * (jj + 2) / 2 <= t) ++jj;
    j = jj;
    i = t - jj * (jj + 1) / 2;
}

struct WorkItem {
    int unit;      // (tile slot) * g + group
    int ks0, ks1;  // k-step range [ks0, ks1) of the unit's `ksteps`
    bool piece;    // true: other pairs hold the rest of this unit
};

// The `it`-th work item of pair `pair`; false when the pair has no more work.  Every role of both CTAs of
// a pair walks the same list.
__device__ __forceinline__ bool work_item(const Schedule &p, int pair, int it, WorkItem &w)
{
    if (it < p.full_waves) {
        w.unit = it * p.pairs + pair;
        w.ks0 = 0;
        w.ks1 = p.ksteps;
        w.piece = false;
        return w.unit < p.units;
    }
    if (pair >= p.tail_pairs) return false;
    const long long total = static_cast<long long>(p.tail_units) * p.ksteps;
    const long long begin = total * pair / p.tail_pairs;
    const long long end = total * (pair + 1) / p.tail_pairs;
    long long cur = begin;
    for (int q = p.full_waves; q < it && cur < end; ++q) cur = (cur / p.ksteps + 1) * p.ksteps;
    if (cur >= end) return false;
    const int tu = static_cast<int>(cur / p.ksteps);
    w.unit = p.full_waves * p.pairs + tu;
    w.ks0 = static_cast<int>(cur - static_cast<long long>(tu) * p.ksteps);
    const long long left = end - cur;
    w.ks1 = (left < p.ksteps - w.ks0) ? w.ks0 + static_cast<int>(left) : p.ksteps;
    w.piece = !(w.ks0 == 0 && w.ks1 == p.ksteps);
    return true;
}

struct WaitCtx {
    volatile uint32_t *abort_flag;   // shared memory
    uint32_t *status;                // global memory
    unsigned long long budget_ns;
};

__device__ __forceinline__ bool wait_gave_up(const WaitCtx &w, uint64_t t0, uint32_t site, uint32_t unit)
{
    if (*w.abort_flag) return true;
    if (global_timer_ns() - t0 > w.budget_ns) {
        *w.abort_flag = 1u;
        if (atomicCAS(&w.status[0], 0u, STATUS_TIMEOUT) == 0u) {
            w.status[1] = site;
            w.status[2] = blockIdx.x;
            w.status[3] = unit;
        }
        __threadfence();
        return true;
    }
    return false;
}

// Slow path of bounded_wait: the thread sleeps inside try_wait (woken when the phase completes) and looks at
// the clock and the abort flag between sleeps.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site, uint32_t unit)
{
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        if (mbar_try_wait_suspend(bar, parity, 2000u)) return true;
        if (wait_gave_up(w, t0, site, unit)) return false;
    }
}

// Wait for roles that are ahead of the tensor core (producer, scalers, epilogue).
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site,
                                             uint32_t unit)
{
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, w, site, unit);
}

// Wait for the MMA issuer, the one thread whose reaction time is on the critical path: polls without pause.
__device__ __noinline__ bool bounded_wait_hot(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site,
                                             uint32_t unit)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u && wait_gave_up(w, t0, site, unit)) return false;
    }
}

__device__ __forceinline__ void spin_ns(unsigned long long ns)
{
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < ns) {}
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GRAM_THREADS, 1)
gram_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1, const GramParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[STAGES];      // used in the pair's first CTA only
    __shared__ __align__(8) uint64_t bar_empty[STAGES];     // signalled in both CTAs by the MMA commits
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
        for (int s = 0; s < STAGES; ++s) {
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
            tile_of_slot(w.unit / p.g, ti, tj);
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
                if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * STAGE_BYTES);   // both CTAs' bytes
                const uint32_t full = map_to_cta(full_local, 0);
                const uint32_t sa = ring + s * STAGE_BYTES;
                const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sa + q * BOX_BYTES, amap, full, a0 + q * BOX_FEATURES, r * TILE_K, ka);
#pragma unroll
                for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                    tma_load_3d_pair(sb + q * BOX_BYTES, bmap, full, b0 + q * BOX_FEATURES, r * TILE_K, kb);
                ++issued;
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
        // Stay until every stage that was filled has been released again: the release is an arrival on
        // this CTA's barriers, which must not come after the CTA has gone.
        // (Stages that were never filled pass at once.)
        for (int q = 0; ok && issued != 0u && q < STAGES; ++q) {
            if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 5u, 0u)) ok = false;
            if (++s == STAGES) { s = 0; ph ^= 1u; }
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
                const uint32_t sa = ring + s * STAGE_BYTES;
                const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
                for (int kk = 0; kk < TILE_K / 16; ++kk) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + kk * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + kk * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != w.ks0 || kk != 0) ? 1u : 0u);
                }
                umma_commit_pair(smem_u32(&bar_empty[s]));   // stage reusable in both CTAs once these MMAs have read it
                if (++s == STAGES) { s = 0; ph ^= 1u; }
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
            tile_of_slot(w.unit / p.g, ti, tj);
            const int k = w.unit % p.g;
            ok = bounded_wait(smem_u32(&bar_acc_full[buf]), acc_ph, wc, 4u, w.unit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int row0 = ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
            const int row = row0 + lane;
            const bool row_ok = row < p.d;
            float *hrow = p.H + (static_cast<size_t>(k) * p.d + (row_ok ? row : 0)) * static_cast<size_t>(p.d);
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
                if (EPI == EPI_ACCUM) {
                    if (!w.piece) {
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            if (col0 + v * 4 < p.d) {
                                float4 *hp = reinterpret_cast<float4 *>(hrow + col0 + v * 4);
                                float4 h = *hp;
                                h.x += __uint_as_float(r[v * 4 + 0]);
                                h.y += __uint_as_float(r[v * 4 + 1]);
                                h.z += __uint_as_float(r[v * 4 + 2]);
                                h.w += __uint_as_float(r[v * 4 + 3]);
                                *hp = h;
                            }
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            if (col0 + v * 4 < p.d)
                                red_add_f32x4(hrow + col0 + v * 4, __uint_as_float(r[v * 4 + 0]),
                                              __uint_as_float(r[v * 4 + 1]), __uint_as_float(r[v * 4 + 2]),
                                              __uint_as_float(r[v * 4 + 3]));
                        }
                    }
                } else {
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
            if (EPI == EPI_DOT) {
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
