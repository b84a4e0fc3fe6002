// Tensor-core core of libgq: upper-triangular tiles of batched Gram-type products
//
//     D_k[a][b] = sum_terms sum_r  A_term[k][r][a] * B_term[k][r][b]        (a in tile rows, b in tile columns)
//
// where every operand is a row-major bf16 matrix whose rows are the contraction index r (tokens for the
// guided Hessian of Algorithm 1 line 4, output channels for the objective of Eq. 7) and whose columns are
// the d_in input features.  Both MMA operands are therefore "MN-major" (feature-contiguous).
//
// One persistent CTA per SM walks a static list of work units (tile, group).  Roles inside a CTA:
//   warp 0 (one lane)  TMA producer: 64-row x 64-feature boxes, 128-byte swizzle, 4-stage ring
//   warp 1 (one lane)  tcgen05.mma issuer: 128 x 256 x 16 bf16 MMAs, fp32 accumulator in TMEM
//   warp 2             TMEM allocation / release (all 512 columns: two 256-column accumulators)
//   warps 4..7         epilogue: tcgen05.ld the finished accumulator while the next tile is computed
// Epilogues:
//   EPI_ACCUM  H_k[tile] += D      (Hessian streaming; each element has exactly one writer)
//   EPI_DOT    partial = sum_{a<=b} (2 - [a==b]) * D[a][b] * H_k[a][b]     (objective)
//
// Every wait on an mbarrier is bounded by a time budget; when it runs out the kernel records
// GQ_ERR_TIMEOUT in the status word, all roles leave their loops, in-flight copies and MMAs are
// waited for (bounded again), TMEM is released and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_ptx.cuh"

namespace gq {

constexpr int TILE_M = 128;
constexpr int TILE_N = 256;
constexpr int TILE_K = 64;
constexpr int STAGES = 4;
constexpr int BOX_FEATURES = 64;                       // 128 bytes of bf16
constexpr int BOX_BYTES = TILE_K * 128;                // one TMA box: 64 rows x 128 B
constexpr int A_STAGE_BYTES = (TILE_M / BOX_FEATURES) * BOX_BYTES;
constexpr int B_STAGE_BYTES = (TILE_N / BOX_FEATURES) * BOX_BYTES;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int GRAM_THREADS = 256;
constexpr int GRAM_SMEM_BYTES = STAGES * STAGE_BYTES + 1024;   // + slack to align the ring to 1024 B
constexpr uint32_t TMEM_COLS = 512;
constexpr int MAX_TERMS = 3;

constexpr int EPI_ACCUM = 0;
constexpr int EPI_DOT = 1;

constexpr uint32_t STATUS_TIMEOUT = 6;   // stored in the status word; the host maps it to GQ_ERR_TIMEOUT

struct GramParams {
    int d;                   // number of features (d_in)
    int rows;                // contraction length of every term
    int g;                   // groups
    int n_terms;
    int term_a[MAX_TERMS];   // which tensor map (0/1) feeds A / B in each term
    int term_b[MAX_TERMS];
    int map_grouped[2];      // 1: the map's third coordinate is the group index; 0: always 0
    int tile_slots;          // NJ*NJ + NJ with NJ = ceil(d / 256)
    int units;               // tile_slots * g
    float *H;                // [g][d][d]
    double *partials;        // EPI_DOT: [units][4]
    uint32_t *status;        // device status word (4 x u32)
    unsigned long long wait_budget_ns;
};

// Slot t of the triangular enumeration -> (row block i of 128, column block j of 256) with i <= 2j + 1.
__device__ __forceinline__ void tile_of_slot(int t, int &i, int &j)
{
    int jj = static_cast<int>((sqrtf(4.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
    while (jj * jj + jj > t) --jj;
    while ((jj + 1) * (jj + 1) + (jj + 1) <= t) ++jj;
    j = jj;
    i = t - jj * jj - jj;
}

struct WaitCtx {
    volatile uint32_t *abort_flag;   // shared memory
    uint32_t *status;                // global memory
    unsigned long long budget_ns;
};

__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site, uint32_t unit)
{
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 31u) == 0u) {
            if (*w.abort_flag) return false;
            if (global_timer_ns() - t0 > w.budget_ns) {
                *w.abort_flag = 1u;
                if (atomicCAS(&w.status[0], 0u, STATUS_TIMEOUT) == 0u) {
                    w.status[1] = site;
                    w.status[2] = blockIdx.x;
                    w.status[3] = unit;
                }
                __threadfence();
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site,
                                             uint32_t unit)
{
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, w, site, unit);
}

template <int EPI>
__global__ void __launch_bounds__(GRAM_THREADS, 1)
gram_kernel(const __grid_constant__ CUtensorMap map0, const __grid_constant__ CUtensorMap map1, const GramParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[STAGES];
    __shared__ __align__(8) uint64_t bar_empty[STAGES];
    __shared__ __align__(8) uint64_t bar_acc_full[2];
    __shared__ __align__(8) uint64_t bar_acc_empty[2];
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile uint32_t abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_acc_full[b]), 1);
            mbar_init(smem_u32(&bar_acc_empty[b]), 128);
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
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_smem;

    const WaitCtx wc{&abort_flag, p.status, p.wait_budget_ns};
    const int kblocks = (p.rows + TILE_K - 1) / TILE_K;
    const int ksteps = kblocks * p.n_terms;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        int s = 0;
        uint32_t ph = 0;
        uint32_t issued = 0;
        bool ok = true;
        for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x) {
            int ti, tj;
            tile_of_slot(u / p.g, ti, tj);
            if (ti * TILE_M >= p.d) continue;
            const int k = u % p.g;
            for (int term = 0; ok && term < p.n_terms; ++term) {
                const int ma = p.term_a[term], mb = p.term_b[term];
                const void *amap = ma ? static_cast<const void *>(&map1) : static_cast<const void *>(&map0);
                const void *bmap = mb ? static_cast<const void *>(&map1) : static_cast<const void *>(&map0);
                const int ka = p.map_grouped[ma] ? k : 0;
                const int kb = p.map_grouped[mb] ? k : 0;
                for (int r = 0; r < kblocks; ++r) {
                    if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, u)) { ok = false; break; }
                    const uint32_t full = smem_u32(&bar_full[s]);
                    const uint32_t sa = ring + s * STAGE_BYTES;
                    const uint32_t sb = sa + A_STAGE_BYTES;
                    mbar_arrive_expect_tx(full, STAGE_BYTES);
#pragma unroll
                    for (int q = 0; q < TILE_M / BOX_FEATURES; ++q)
                        tma_load_3d(sa + q * BOX_BYTES, amap, full, ti * TILE_M + q * BOX_FEATURES, r * TILE_K, ka);
#pragma unroll
                    for (int q = 0; q < TILE_N / BOX_FEATURES; ++q)
                        tma_load_3d(sb + q * BOX_BYTES, bmap, full, tj * TILE_N + q * BOX_FEATURES, r * TILE_K, kb);
                    ++issued;
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        if (!ok) {
            // Let the copies that were already issued land before the CTA retires (bounded).
            const uint32_t pending = issued < static_cast<uint32_t>(STAGES) ? issued : STAGES;
            int ss = s;
            uint32_t pp = ph;
            for (uint32_t q = 0; q < pending; ++q) {
                if (--ss < 0) { ss = STAGES - 1; pp ^= 1u; }
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&bar_full[ss]), pp) && global_timer_ns() - t0 < 5000000ull) {}
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16_mn(TILE_M, TILE_N);
        int s = 0;
        uint32_t ph = 0;
        int buf = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x) {
            int ti, tj;
            tile_of_slot(u / p.g, ti, tj);
            if (ti * TILE_M >= p.d) continue;
            if (!bounded_wait(smem_u32(&bar_acc_empty[buf]), acc_ph ^ 1u, wc, 2u, u)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * TILE_N);
            for (int ks = 0; ks < ksteps; ++ks) {
                if (!bounded_wait(smem_u32(&bar_full[s]), ph, wc, 3u, u)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t sa = ring + s * STAGE_BYTES;
                const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
                for (int kk = 0; kk < TILE_K / 16; ++kk) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + kk * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + kk * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks | kk) != 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&bar_empty[s]));   // stage reusable once these MMAs have read it
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
            umma_commit(smem_u32(&bar_acc_full[buf]));
            buf ^= 1;
            if (buf == 0) acc_ph ^= 1u;
        }
        if (!ok) {
            // Make sure no MMA is still writing TMEM when it is released.
            umma_commit(smem_u32(&bar_drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&bar_drain), 0u) && global_timer_ns() - t0 < 5000000ull) {}
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ epilogue (128 threads)
        const int q = warp & 3;                 // TMEM lane quarter this warp may access
        int buf = 0;
        uint32_t acc_ph = 0;
        bool ok = true;
        for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x) {
            int ti, tj;
            tile_of_slot(u / p.g, ti, tj);
            const int k = u % p.g;
            if (ti * TILE_M >= p.d) {
                if (EPI == EPI_DOT && lane == 0) p.partials[static_cast<size_t>(u) * 4 + q] = 0.0;
                continue;
            }
            ok = bounded_wait(smem_u32(&bar_acc_full[buf]), acc_ph, wc, 4u, u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int row0 = ti * TILE_M + q * 32;
            const int row = row0 + lane;
            const bool row_ok = row < p.d;
            float *hrow = p.H + (static_cast<size_t>(k) * p.d + (row_ok ? row : 0)) * static_cast<size_t>(p.d);
            double dsum = 0.0;
#pragma unroll 1
            for (int cc = 0; cc < TILE_N / 32; ++cc) {
                const int col0 = tj * TILE_N + cc * 32;
                if (col0 >= p.d) break;                    // right of the matrix
                if (col0 + 32 <= row0) continue;           // 32 x 32 block strictly below the diagonal
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                  static_cast<uint32_t>(buf * TILE_N + cc * 32), r);
                tmem_ld_wait();
                if (!row_ok) continue;
                if (EPI == EPI_ACCUM) {
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
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&bar_acc_empty[buf]));
            if (EPI == EPI_DOT) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                if (lane == 0) p.partials[static_cast<size_t>(u) * 4 + q] = dsum;
            }
            buf ^= 1;
            if (buf == 0) acc_ph ^= 1u;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace gq
