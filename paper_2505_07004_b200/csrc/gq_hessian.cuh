// Guided Hessian of Algorithm 1, Hessian step with the row scaling fused into the operand path:
//
//     H_k[a][b] += sum_i  (s_k[i] * X[i][a]) * X[i][b]          for a <= b, all groups k
//
// Tokens i are the contraction index, features are contiguous in memory, so both MMA operands are
// MN-major bf16.  The kernel runs as CTA pairs (clusters of two); a pair owns one 256 x 256 tile of H for
// TWO groups at a time (2 x 256 fp32 accumulator columns = all of tensor memory), so that one pass over
// the tile's rows of X serves two groups and no scaled copy of X ever exists in global memory.  (When g is
// odd the last group is processed two neighbouring column tiles at a time instead: see UnitDesc.)
//
//   B operand  raw X[tokens, tile columns]: TMA boxes (64 tokens x 64 features, 128-byte swizzle),
//              16 KB per CTA and k-step, shared by both groups
//   A operand  s_k[token] * X[token, tile rows], one 16 KB block per group and k-step: twelve "scaler" warps
//              in three sets that take k-steps in turn (so three k-steps of loads are in flight) read the raw
//              rows straight from global memory with 128-bit loads, multiply by s_k (carried as two bf16
//              terms, packed bf16 fused multiply-adds, one final rounding to bf16) and store into shared
//              memory in exactly the swizzled layout a TMA load would have produced
//   MMA        the pair's first CTA issues, per k-step and group, four tcgen05.mma.cta_group::2
//              (M = 256, N = 256, K = 16) with fp32 accumulation in tensor memory
//   epilogue   eight warps per CTA move the accumulators to H: tcgen05.ld -> swizzled staging block in
//              shared memory -> TMA reduce-add (cp.reduce.async.bulk.tensor ... .add) of 32 x 32 fp32
//              blocks, so H is never read by the SMs and every access to it is a full 128-byte row segment
//
// Per CTA and k-step (1024 tensor-core clocks for two groups) this moves 32 KB from L2 (half of what a
// per-group pass over pre-scaled operands needs) and 112 KB through shared memory.
//
// Warps: 0 TMA producer (one lane) | 1 MMA issuer (one lane, first CTA) | 2 TMEM allocation | 3 - |
//        4..15 scalers | 16..23 epilogue.  Warps 2 and 3 have nothing to do in the Hessian step; on request
//        (SaliencyAhead) they compute the saliency of the next token chunk meanwhile: 296 warps that stream the
//        next gradient block at a small fraction of the memory bandwidth, hidden behind the tensor-core work.
// Work units are (tile, pair of groups), plus (row block, pair of column tiles) for an odd last group; they are dealt to the CTA pairs as described in gq_pipeline.cuh
// (round-robin rounds, then the incomplete last round cut along the token axis).  Because H is updated
// by reduce-adds only, pieces of a cut unit need no special treatment.
//
// The accumulators are single-buffered: after the last k-step of a unit the MMA issuer waits until the
// epilogue warps have read them out of tensor memory (not until H is updated).  Producer and scalers run
// ahead into the next unit meanwhile, so the pipeline is full again when the MMAs resume.
//
// Every mbarrier wait is bounded (see gq_pipeline.cuh).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_kernels.cuh"
#include "gq_pipeline.cuh"

namespace gq {

constexpr int HS_STAGES = 4;
constexpr int HS_GROUPS = 2;                                   // accumulators resident in tensor memory at once
constexpr int HS_SLOT_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;         // one operand block: 16 KB
constexpr int HS_STAGE_BYTES = 3 * HS_SLOT_BYTES;                            // 48 KB
constexpr int HS_SETS = 3;                                     // independent scaler sets (k-steps in flight)
constexpr int HS_SET_WARPS = 4;                                // warps per set: 128 threads cover 8 tokens x 128 features
constexpr int HS_SCALER_WARPS = HS_SETS * HS_SET_WARPS;
constexpr int HS_EPI_WARPS = 8;
constexpr int HS_STAGING_BYTES = HS_EPI_WARPS * 4096;          // one 32 x 32 fp32 block per epilogue warp
constexpr int HS_THREADS = 32 * (4 + HS_SCALER_WARPS + HS_EPI_WARPS);
constexpr int HS_SMEM_BYTES = HS_STAGES * HS_STAGE_BYTES + HS_STAGING_BYTES + 1024;

// The saliency step of the NEXT token chunk, computed by the two warps per CTA that the Hessian step leaves idle
// (Algorithm 1: the saliency of a chunk depends on nothing the Hessian step of the previous chunk writes).
// grad == nullptr: nothing to do.
struct SaliencyAhead {
    const __nv_bfloat16 *grad;   // [n][ld_grad]
    unsigned n;                  // tokens of the next chunk
    int m;                       // d_out / g
    long long ld_grad;
    float coef;                  // grad_scale^2 / m
    float *s;                    // [g][ld_s]
    long long ld_s;
    uint32_t *words;             // the next call's packed saliency: [ceil(g / 2)][n] pairs of words
};

struct HessianParams {
    const __nv_bfloat16 *X;  // [n][ld_x]
    long long ld_x;
    const uint2 *s2;         // [ceil(g / 2)][n]: split saliency of groups (2 q, 2 q + 1), see split_saliency_kernel
    int n;                   // tokens in this call
    int d;                   // d_in
    int g;
    int nj;                  // ceil(d / 256): tile blocks per side
    int raster;              // edge (in tiles) of the super-blocks of the tile order, see tile_of_slot_blocked
    int full_pairs;          // g / 2: pairs of groups that share a pass over X
    int narrow_units;        // tiles * full_pairs: units (tile, pair of groups)
    Schedule sched;          // units = narrow_units + (g odd ? column-pair slots : 0), ksteps = ceil(n / 64)
    uint32_t *status;
    unsigned long long wait_budget_ns;
    SaliencyAhead ahead;
};

// What a work unit computes.  A unit always fills (up to) two 256-column accumulators from one pass over
// the tile rows of X:
//   pair unit  one tile, two groups: accumulator kk holds group grp[kk]; B (raw columns) is shared, the
//              scalers produce one A block per group;
//   wide unit  (the last group when g is odd) one group, two neighbouring column tiles: accumulator kk
//              holds column tile tj[kk]; the scaled A block is shared, there is one B block per tile.
//              An accumulator whose tile lies below the diagonal or outside the matrix is not used.
// Shared-memory stage = three 16 KB slots: [B | A(g0) | A(g1)] for a pair unit, [B(tj0) | A | B(tj1)] for a
// wide unit.
struct UnitDesc {
    int ti;          // row block of the tile(s)
    int tj[2];       // column block of accumulator 0 / 1
    int grp[2];      // group of accumulator 0 / 1
    bool use[2];
    bool wide;
    __device__ int a_slot(int kk) const { return wide ? 1 : 1 + kk; }
    __device__ int b_slot(int kk) const { return (wide && kk) ? 2 : 0; }
    __device__ int scaled_groups() const { return wide ? 1 : 2; }
};

struct HessianParams;
__device__ __forceinline__ UnitDesc decode_unit(const HessianParams &p, int unit);

__device__ __forceinline__ uint4 ld_stream_16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_shared_16(uint32_t addr, const uint4 &v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Saliency as the scalers use it.  A value a is carried as two bf16 terms packed in one word: low half
// hi = bf16(a), high half lo = bf16(a - hi); hi + lo has 16 significant bits.  The words of groups 2 q and
// 2 q + 1 of a token sit side by side, so a scaler thread fetches both with one 8-byte load and does no
// conversion work in its loop (sixteen threads share a token; converting there would be done sixteen times).
__global__ void __launch_bounds__(256)
split_saliency_kernel(const float *__restrict__ s, long long ld_s, int n, int g, uint2 *__restrict__ out);

__global__ void __launch_bounds__(256)
split_saliency_kernel(const float *__restrict__ s, long long ld_s, int n, int g, uint2 *__restrict__ out)
{
    const int slots = (g + 1) / 2;
    const long long total = static_cast<long long>(slots) * n;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
         idx += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int q = static_cast<int>(idx / n);
        const int i = static_cast<int>(idx - static_cast<long long>(q) * n);
        uint2 v;
        v.x = split_scale(s[static_cast<long long>(2 * q) * ld_s + i]);
        v.y = (2 * q + 1 < g) ? split_scale(s[static_cast<long long>(2 * q + 1) * ld_s + i]) : 0u;
        out[idx] = v;
    }
}

// v (8 bf16) times the split scale `a2`: per element fma(x, hi, x * lo) with packed bf16 fused multiply-adds.
// x * lo is rounded to bf16 (an error of 2^-18 of the product), then x * hi + that is formed exactly and
// rounded to bf16 once; no conversion to fp32 and back is needed.
__device__ __forceinline__ uint4 scale_bf16x8(const uint4 &v, uint32_t a2)
{
    const uint32_t hi_bits = __byte_perm(a2, a2, 0x1010);
    const uint32_t lo_bits = __byte_perm(a2, a2, 0x3232);
    const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162 *>(&hi_bits);
    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162 *>(&lo_bits);
    const __nv_bfloat162 *x = reinterpret_cast<const __nv_bfloat162 *>(&v);
    uint4 o;
    __nv_bfloat162 *oh = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
    for (int e = 0; e < 4; ++e) oh[e] = __hfma2(x[e], hi, __hmul2(x[e], lo));
    return o;
}

__device__ __forceinline__ UnitDesc decode_unit(const HessianParams &p, int unit)
{
    UnitDesc u;
    if (unit < p.narrow_units) {
        int ti, tj;
        tile_of_slot_blocked(unit / p.full_pairs, p.nj, p.raster, ti, tj);
        const int k0 = (unit % p.full_pairs) * 2;
        u.ti = ti;
        u.tj[0] = u.tj[1] = tj;
        u.grp[0] = k0;
        u.grp[1] = k0 + 1;
        u.use[0] = u.use[1] = true;
        u.wide = false;
    } else {
        int i, q;
        colpair_of_slot(unit - p.narrow_units, i, q);
        u.ti = i;
        u.tj[0] = 2 * q;
        u.tj[1] = 2 * q + 1;
        u.grp[0] = u.grp[1] = p.g - 1;
        u.use[0] = 2 * q >= i;
        u.use[1] = 2 * q + 1 < p.nj;
        u.wide = true;
    }
    return u;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(HS_THREADS, 1)
hessian_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapH, const HessianParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[HS_STAGES];    // first CTA: B bytes of both CTAs + all scaler warps
    __shared__ __align__(8) uint64_t bar_empty[HS_STAGES];   // both CTAs: signalled by the MMA commits
    __shared__ __align__(8) uint64_t bar_acc_full;           // both CTAs: signalled by the MMA commit
    __shared__ __align__(8) uint64_t bar_acc_empty[HS_GROUPS];   // first CTA, one per accumulator: 16 epilogue warps arrive
    __shared__ __align__(8) uint64_t bar_drain;
    __shared__ uint32_t tmem_base_smem;
    __shared__ volatile uint32_t abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = static_cast<int>(blockIdx.x >> 1);
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging = ring + HS_STAGES * HS_STAGE_BYTES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < HS_STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1 + 2 * HS_SET_WARPS);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc_full), 1);
        for (int kk = 0; kk < HS_GROUPS; ++kk) mbar_init(smem_u32(&bar_acc_empty[kk]), 2 * HS_EPI_WARPS);
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&mapX);
        prefetch_tensormap(&mapH);
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

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer: raw B columns
        int s = 0;
        uint32_t ph = 0;
        uint32_t issued = 0;
        bool ok = true;
        WorkItem w;
        const uint64_t pol_x = l2_policy_evict_last();      // X is re-read by many units: keep it in L2
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const UnitDesc u = decode_unit(p, w.unit);
            const int n_b = u.wide ? (u.use[0] ? 1 : 0) + (u.use[1] ? 1 : 0) : 1;      // B blocks per stage
            for (int ks = w.ks0; ks < w.ks1; ++ks) {
                if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, w.unit)) { ok = false; break; }
                const uint32_t full_local = smem_u32(&bar_full[s]);
                if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * n_b * HS_SLOT_BYTES);   // both CTAs' bytes
                const uint32_t full = map_to_cta(full_local, 0);
                for (int kk = 0; kk < (u.wide ? 2 : 1); ++kk) {
                    if (!u.use[kk]) continue;
                    const uint32_t sb = ring + s * HS_STAGE_BYTES + u.b_slot(kk) * HS_SLOT_BYTES;
                    const int b0 = u.tj[kk] * TILE_N + static_cast<int>(rank) * CTA_ROWS;
#pragma unroll
                    for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q)
                        tma_load_3d_pair_hint(sb + q * BOX_BYTES, &mapX, full, b0 + q * BOX_FEATURES, ks * TILE_K, 0, pol_x);
                }
                ++issued;
                if (++s == HS_STAGES) { s = 0; ph ^= 1u; }
            }
        }
        // Stay until every stage has been released again: the release is an arrival on this CTA's barriers,
        // which must not come after the CTA has gone.
        for (int q = 0; ok && issued != 0u && q < HS_STAGES; ++q) {
            if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 5u, 0u)) ok = false;
            if (++s == HS_STAGES) { s = 0; ph ^= 1u; }
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
            const UnitDesc u = decode_unit(p, w.unit);
            // The epilogue empties accumulator 0 first.  The first k-steps of the new unit (as many as the ring
            // holds) are therefore issued for accumulator 0 as soon as it is free, while accumulator 1 is still
            // being read out, then for accumulator 1; a stage is released after both.
            auto issue = [&](int kk, int stage_idx, int ks) {
                if (!u.use[kk]) return;
                const uint32_t stage = ring + stage_idx * HS_STAGE_BYTES;
                const uint32_t sa = stage + u.a_slot(kk) * HS_SLOT_BYTES;
                const uint32_t sb = stage + u.b_slot(kk) * HS_SLOT_BYTES;
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(kk * TILE_N);
#pragma unroll
                for (int k16 = 0; k16 < TILE_K / 16; ++k16) {
                    const uint64_t adesc = umma_smem_desc_mn_sw128(sa + k16 * 16 * 128, BOX_BYTES, 1024);
                    const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + k16 * 16 * 128, BOX_BYTES, 1024);
                    umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != w.ks0 || k16 != 0) ? 1u : 0u);
                }
            };
            const int n_head = (w.ks1 - w.ks0 < HS_STAGES) ? (w.ks1 - w.ks0) : HS_STAGES;
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[0]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            {
                int s_h = s;
                uint32_t ph_h = ph;
                for (int q = 0; q < n_head; ++q) {
                    if (!bounded_wait_hot(smem_u32(&bar_full[s_h]), ph_h, wc, 3u, w.unit)) { ok = false; break; }
                    tc_fence_after_sync();
                    issue(0, s_h, w.ks0 + q);
                    if (++s_h == HS_STAGES) { s_h = 0; ph_h ^= 1u; }
                }
            }
            if (!ok) break;
            if (!bounded_wait_hot(smem_u32(&bar_acc_empty[1]), acc_ph ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
            tc_fence_after_sync();
            for (int q = 0; q < n_head; ++q) {
                issue(1, s, w.ks0 + q);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                if (++s == HS_STAGES) { s = 0; ph ^= 1u; }
            }
            int ks = w.ks0 + n_head;
            for (; ks + 1 < w.ks1; ks += 2) {             // two k-steps at a time: eight MMAs in a row per accumulator
                const int s2 = (s + 1 == HS_STAGES) ? 0 : s + 1;
                const uint32_t ph2 = (s + 1 == HS_STAGES) ? (ph ^ 1u) : ph;
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                if (!bounded_wait_hot(smem_u32(&bar_full[s2]), ph2, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                issue(0, s, ks);
                issue(0, s2, ks + 1);
                issue(1, s, ks);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                issue(1, s2, ks + 1);
                umma_commit_pair(smem_u32(&bar_empty[s2]));
                s = (s2 + 1 == HS_STAGES) ? 0 : s2 + 1;
                ph = (s2 + 1 == HS_STAGES) ? (ph2 ^ 1u) : ph2;
            }
            for (; ok && ks < w.ks1; ++ks) {
                if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                issue(0, s, ks);
                issue(1, s, ks);
                umma_commit_pair(smem_u32(&bar_empty[s]));
                if (++s == HS_STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
            umma_commit_pair(smem_u32(&bar_acc_full));
            acc_ph ^= 1u;
        }
        if (!ok) {
            umma_commit_local(smem_u32(&bar_drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&bar_drain), 0u) && global_timer_ns() - t0 < 5000000ull) {}
        }
    } else if (warp >= 4 && warp < 4 + HS_SCALER_WARPS) {
        // ------------------------------------------------------------------ scalers: A_k = s_k (.) X rows
        // The scaler warps form HS_SETS independent sets of four warps; set j produces the k-steps whose
        // running number is j modulo HS_SETS, from the loads to the arrival on the "full" barrier.  A set
        // issues the loads of its next k-step as soon as it has finished the previous one, i.e. HS_SETS - 1
        // k-steps of the other sets' work lie between a load and its use: global-memory latency is hidden by
        // the other sets rather than by a register rotation inside one warp.
        // Inside a set, sixteen threads share a token row (16 x 16 bytes = the 128 features, so a warp reads
        // two whole 256-byte row segments per load) and eight passes cover the 64 tokens of the k-step.  Every
        // thread fetches the (pre-split) saliency words of its eight tokens itself, one broadcast 8-byte load per
        // pass for both groups; shuffles are avoided: like every shared-memory-pipe instruction they compete with the tensor core's
        // operand reads.
        constexpr int TOK_PER_PASS = HS_SET_WARPS * 2;         // tokens a set covers per instruction
        constexpr int PASSES = TILE_K / TOK_PER_PASS;          // 16-byte loads per thread and k-step
        const int set = (warp - 4) / HS_SET_WARPS;
        const int st = static_cast<int>(threadIdx.x) - 128 - set * (HS_SET_WARPS * 32);    // 0..127
        const int c = st & 15;                                 // 16-byte chunk of the 128-feature row
        const int trow = st >> 4;                              // token within a pass
        const uint32_t col_off = static_cast<uint32_t>((c >> 3) * BOX_BYTES);
        const int cb = c & 7;

        KstepCursor cur(p.sched, pair);
        cur.advance(set);
        int cached_it = -1;
        int ng = 0;
        const __nv_bfloat16 *xcol = nullptr;
        const uint2 *s2 = nullptr;
        bool f_ok = false;
        for (int cnt = set; cur.valid; cnt += HS_SETS, cur.advance(HS_SETS)) {
            if (cur.it != cached_it) {
                cached_it = cur.it;
                const UnitDesc u = decode_unit(p, cur.w.unit);
                ng = u.scaled_groups();
                const int f = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + c * 8;
                f_ok = f < p.d;
                xcol = p.X + f;
                s2 = p.s2 + static_cast<long long>(u.grp[0] >> 1) * p.n;
            }
            const int tok0 = cur.ks * TILE_K + trow;
            uint4 buf[PASSES];
            uint2 sv[PASSES];
            {
                const __nv_bfloat16 *src = xcol + static_cast<long long>(tok0) * p.ld_x;
                const long long step = static_cast<long long>(TOK_PER_PASS) * p.ld_x;
                const uint2 *ssrc = s2 + tok0;
                if (f_ok && (cur.ks + 1) * TILE_K <= p.n) {         // whole k-step inside the chunk: no predicates
#pragma unroll
                    for (int j = 0; j < PASSES; ++j) {
                        buf[j] = ld_stream_16(src + j * step);
                        sv[j] = __ldg(ssrc + j * TOK_PER_PASS);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < PASSES; ++j) {
                        const bool t_ok = tok0 + j * TOK_PER_PASS < p.n;
                        buf[j] = (f_ok && t_ok) ? ld_stream_16(src + j * step) : make_uint4(0u, 0u, 0u, 0u);
                        sv[j] = t_ok ? __ldg(ssrc + j * TOK_PER_PASS) : make_uint2(0u, 0u);
                    }
                }
            }

            const int s = cnt % HS_STAGES;
            const uint32_t ph = static_cast<uint32_t>(cnt / HS_STAGES) & 1u;
            bool got = true;
            if (lane == 0) got = bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 6u, cur.w.unit);
            got = __any_sync(0xffffffffu, got && lane == 0);
            if (!got) break;
            (void)mbar_try_wait(smem_u32(&bar_empty[s]), ph ^ 1u);   // every lane observes the completed phase
            const uint32_t sa = ring + s * HS_STAGE_BYTES + HS_SLOT_BYTES + col_off;     // slot 1 (and 2)
#pragma unroll
            for (int j = 0; j < PASSES; ++j) {
                const int tl = j * TOK_PER_PASS + trow;
                const uint32_t dst = sa + static_cast<uint32_t>(tl * 128 + ((cb ^ (tl & 7)) << 4));
                st_shared_16(dst, scale_bf16x8(buf[j], sv[j].x));
                if (ng > 1) st_shared_16(dst + HS_SLOT_BYTES, scale_bf16x8(buf[j], sv[j].y));
            }
            fence_proxy_async_smem();        // make the stores visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_full[s]), 0));
        }
    } else if (warp >= 4 + HS_SCALER_WARPS) {
        // ------------------------------------------------------------------ epilogue: H += accumulators
        const int ew = warp - (4 + HS_SCALER_WARPS);    // 0..7
        const int q = warp & 3;                         // TMEM lane quarter this warp may access
        const int half = ew >> 2;                       // which 128 of the 256 accumulator columns
        const uint32_t stg = staging + static_cast<uint32_t>(ew) * 4096u;
        const uint64_t pol_h = l2_policy_evict_first();     // H is touched once per launch: it should not displace X
        uint32_t acc_ph = 0;
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const UnitDesc u = decode_unit(p, w.unit);
            if (lane == 0) ok = bounded_wait(smem_u32(&bar_acc_full), acc_ph, wc, 4u, w.unit);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            (void)mbar_try_wait(smem_u32(&bar_acc_full), acc_ph);     // every lane observes the completed phase
            tc_fence_after_sync();
            const int row0 = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
            for (int kk = 0; kk < HS_GROUPS; ++kk) {
#pragma unroll 1
                for (int c4 = 0; u.use[kk] && c4 < 4; ++c4) {
                    const int cc = half * 4 + c4;
                    const int col0 = u.tj[kk] * TILE_N + cc * 32;
                    if (col0 >= p.d || row0 >= p.d) break;      // outside the matrix
                    if (col0 + 32 <= row0) continue;            // 32 x 32 block strictly below the diagonal
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                      static_cast<uint32_t>(kk * TILE_N + cc * 32), r);
                    tmem_ld_wait();
                    if (lane == 0) bulk_wait_group_read0();   // the copy engine has read the previous staging block
                    __syncwarp();
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        st_shared_16(stg + static_cast<uint32_t>(lane * 128 + ((v ^ (lane & 7)) << 4)),
                                     make_uint4(r[v * 4 + 0], r[v * 4 + 1], r[v * 4 + 2], r[v * 4 + 3]));
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_reduce_add_3d_hint(&mapH, stg, col0, row0, u.grp[kk], pol_h);
                        bulk_commit_group();
                    }
                }
                // This warp has read all it needs from accumulator kk: tell the MMA issuer (first CTA).
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[kk]), 0));
            }
            acc_ph ^= 1u;
        }
        if (lane == 0) bulk_wait_group_read0();       // shared memory must outlive the last reduce-add's read
    } else if ((warp == 2 || warp == 3) && p.ahead.grad != nullptr) {
        // ------------------------------------------------------------------ saliency of the next chunk
        // Same lane-to-element assignment and the same order of additions as saliency_kernel, so the values are
        // the same bits.  Segment = (token, group); the 2 * gridDim.x warps take segments round-robin, so at any
        // time they read one contiguous window of the gradient block.  Short segments (at most four loads per
        // lane) are taken two at a time, eight loads in flight per lane.
        const SaliencyAhead &a = p.ahead;
        const unsigned g_u = static_cast<unsigned>(p.g);
        const unsigned total = a.n * g_u;
        const unsigned stride = gridDim.x * 2u;
        const int vecs = a.m >> 3;
        unsigned seg = blockIdx.x * 2u + static_cast<unsigned>(warp - 2);
        auto segment_src = [&](unsigned sg, unsigned &i, int &k) {
            i = sg / g_u;
            k = static_cast<int>(sg - i * g_u);
            return reinterpret_cast<const uint4 *>(a.grad + static_cast<long long>(i) * a.ld_grad + static_cast<long long>(k) * a.m);
        };
        if (vecs <= 128) {
            for (; seg < total; seg += 2u * stride) {
                const bool two = seg + stride < total;
                unsigned i0, i1 = 0u;
                int k0, k1 = 0;
                const uint4 *src0 = segment_src(seg, i0, k0);
                const uint4 *src1 = two ? segment_src(seg + stride, i1, k1) : src0;
                uint4 x[8];
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    x[t] = (lane + 32 * t < vecs) ? ld_once_16(src0 + lane + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    x[4 + t] = (two && lane + 32 * t < vecs) ? ld_once_16(src1 + lane + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
                float acc[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) acc[t] = sum_sq_bf16x8(x[t], 0.f);
                const float sum0 = warp_sum_butterfly((acc[0] + acc[1]) + (acc[2] + acc[3]));
                const float sum1 = warp_sum_butterfly((acc[4] + acc[5]) + (acc[6] + acc[7]));
                if (lane == 0) {
                    saliency_store(sum0 * a.coef, i0, k0, a.n, p.g, a.s, a.ld_s, a.words);
                    if (two) saliency_store(sum1 * a.coef, i1, k1, a.n, p.g, a.s, a.ld_s, a.words);
                }
            }
        } else {
            // Long segments: eight loads in flight per lane from the first to the last (saliency_kernel takes
            // the ends of a segment four at a time; element lane + 32 t of every group of eight goes to partial
            // sum t & 3 in ascending order either way, so the sums are the same bits).
            for (; seg < total; seg += stride) {
                unsigned i;
                int k;
                const uint4 *src = segment_src(seg, i, k);
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                for (int v = lane; v < vecs; v += 256) {
                    uint4 x[8];
#pragma unroll
                    for (int t = 0; t < 8; ++t)
                        x[t] = (v + 32 * t < vecs) ? ld_once_16(src + v + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int t = 0; t < 8; ++t) acc[t & 3] = sum_sq_bf16x8(x[t], acc[t & 3]);
                }
                const float sum = warp_sum_butterfly((acc[0] + acc[1]) + (acc[2] + acc[3]));
                if (lane == 0) saliency_store(sum * a.coef, i, k, a.n, p.g, a.s, a.ld_s, a.words);
            }
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
