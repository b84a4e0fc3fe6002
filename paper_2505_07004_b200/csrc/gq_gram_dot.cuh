// The objective of Eq. 7 on the tensor cores:
//
//     loss_k = sum_{j in J_k} delta_j^T H_k delta_j = < H_k , Delta_k^T Delta_k >,     Delta_k = rows J_k of W - W_hat,
//
// evaluated on the upper triangle, sum_{a <= b} (2 - [a == b]) D_k[a][b] H_k[a][b] with D_k = Delta_k^T Delta_k.
// D_k is never written: a CTA pair forms one 256 x 256 tile of it in tensor memory and contracts it with the
// matching entries of H_k straight out of tensor memory.
//
// Operands.  Delta is prepared once per call as ONE fp16 matrix (delta_half_kernel): delta * 2^e with a single
// power of two e for the whole layer, chosen from max |delta| (delta_absmax_kernel) so that the largest entry
// lies in [2^14, 2^15).  fp16 carries 11 significant bits at any magnitude above 2^-14, i.e. down to 2^-28 of
// the largest entry, and the scaling is undone exactly (2^-2e in the final fp64 reduction).  One product at the
// 16-bit rate replaces three bf16 products (hi hi + hi lo + lo hi): the contraction then costs about as much as
// streaming H from HBM, which is what the kernel below is built around.  Rounding: both factors of every
// product carry a relative error of at most 2^-12 (round to nearest), unbiased, so the objective is good to
// 2^-11 = 4.9e-4 in the worst case of all errors aligned and to ~1e-6 for errors of random sign.
//
// Units.  A unit is one 256 x 256 tile (i <= j) of one group; a pair's tensor memory holds two such accumulators,
// so the tile of unit n + 1 is being computed while the tile of unit n is contracted with H: the tensor core
// never waits for a read-out.  (Units of two column tiles sharing their row operand, as in gq_hessian.cuh, need
// a quarter less operand traffic from L2 but fill tensor memory with one unit: measured on the 4096 x 4096 layer
// the tensor core then idled for a third of every unit, waiting for H.)  The stage is [A | B], 16 KB each, 64
// channels of the contraction, six stages.  Units are numbered group-major and, inside a group, in the
// super-block tile order of gq_pipeline.cuh, so that the pairs working at the same time share operand blocks.
//
// H.  The entries of H_k that go with a tile (256 KB per pair) do not depend on the accumulators; what limits
// their delivery is the number of requests an SM can have in flight (a lane needs 32 consecutive floats of ITS
// row, tensor memory dictates lane = row, so a warp's 32-byte load is 32 separate sector requests).  So the
// requests are spread over the whole time the tile is being computed: as soon as an epilogue warp has finished a
// tile it requests the four 32 x 32 blocks of its next tile into registers (128 KB per CTA: with that the eight
// epilogue warps hold all of the CTA's share), and they have a full unit of MMAs (4 - 7 us) to arrive.  (An extra
// warp that asked for the same rows earlier still with bulk L2 prefetches changed nothing measurable on any of
// the layer shapes and was taken out again.)  Once the accumulator is complete the contraction itself takes well
// under a microsecond: tensor-memory columns of block j + 1 are requested before block j is used, blocks above
// the diagonal take a branch without per-entry weights, and the accumulator is handed back as soon as its last
// block sits in registers.
//
// Roles: warp 0 (one lane) TMA producer, warp 1 (one lane, first CTA) MMA issuer, warp 2 TMEM allocation,
// warp 3 idle, warps 4..11 epilogue (registers: the service warpgroup gives up all but 40, the two
// epilogue warpgroups take 232).  Whole units only: one fp64 partial per (unit, CTA, warp), reduced in a fixed
// order, so the result is reproducible.  Every mbarrier wait is bounded (gq_pipeline.cuh).
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gq_pipeline.cuh"

namespace gq {

constexpr int GD_STAGES = 6;
constexpr int GD_SLOT_BYTES = (CTA_ROWS / BOX_FEATURES) * BOX_BYTES;      // one operand block: 16 KB
constexpr int GD_STAGE_BYTES = 2 * GD_SLOT_BYTES;                         // [A | B]
constexpr int GD_EPI_WARPS = 8;
constexpr int GD_THREADS = 32 * (4 + GD_EPI_WARPS);
constexpr int GD_SMEM_BYTES = GD_STAGES * GD_STAGE_BYTES + 1024;
constexpr int GD_PARTIALS_PER_UNIT = 2 * GD_EPI_WARPS;       // one fp64 per (CTA of the pair, epilogue warp)
constexpr int GD_TARGET_EXP = 14;                            // the largest |delta| * 2^e lies in [2^14, 2^15)
constexpr int GD_MAX_SHIFT = 100;                            // |e| is kept below this (the scale stays a normal float)

// Header of the objective workspace, written by the preparation kernels and read by the reduction.
struct GramDotHeader {
    unsigned int absmax_bits;   // bit pattern of max |W - W_hat| (non-negative floats order like unsigned ints)
    int shift;                  // e: the fp16 matrix holds (W - W_hat) * 2^e
    unsigned int blocks_done;   // groups whose loss has been written (the last one forms the total)
};

struct GramDotParams {
    int d;                   // d_in
    int rows;                // channels per group (contraction length)
    int g;
    int nj;                  // ceil(d / 256)
    int tiles;               // nj (nj + 1) / 2: 256 x 256 tiles on the upper triangle
    int raster;              // edge (in tiles) of the super-blocks of the tile order (gq_pipeline.cuh)
    Schedule sched;          // units = tiles * g (group-major: unit = k * tiles + tile slot), ksteps = ceil(rows / 64)
    const float *H;          // [g][d][d], only a <= b is read
    double *partials;        // [units][GD_PARTIALS_PER_UNIT]
    uint32_t *status;
    unsigned long long wait_budget_ns;
};

// Instruction descriptor for kind::f16 with fp16 A and B (both MN-major), fp32 accumulator: as
// umma_idesc_bf16_mn with the operand format fields [7,10) and [10,13) left at 0 (= f16).
__host__ __device__ constexpr uint32_t umma_idesc_f16_mn(uint32_t m, uint32_t n)
{
    return (1u << 4) | (1u << 15) | (1u << 16) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

// Eight consecutive floats (32 bytes, 32-byte aligned) that are read once: no L1 allocation.
__device__ __forceinline__ void ld_stream_f32x8(const float *p, float (&v)[8])
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}

// 16 bytes of fp32 input, loaded by volatile asm so that a thread's loads are all issued before the first use.
__device__ __forceinline__ float4 ld_f32x4(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_f32x4_last_use(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

constexpr int DELTA_VEC_PER_THREAD = 4;      // float4 pairs a thread of the two preparation kernels handles

// ------------------------------------------------------------------------------------------------
// max |W - W_hat| over the layer (the differences are formed in fp32, as everywhere in the objective).
// header->absmax_bits must be 0 before the launch.  One block per 256 * DELTA_VEC_PER_THREAD float4 pairs.
__global__ void __launch_bounds__(256)
delta_absmax_kernel(const float *__restrict__ W, const float *__restrict__ What, unsigned count4, GramDotHeader *header)
{
    const unsigned base = blockIdx.x * (256u * DELTA_VEC_PER_THREAD) + threadIdx.x;
    float4 w[DELTA_VEC_PER_THREAD], q[DELTA_VEC_PER_THREAD];
#pragma unroll
    for (int t = 0; t < DELTA_VEC_PER_THREAD; ++t) {
        const unsigned idx = base + t * 256u;
        const bool in = idx < count4;
        w[t] = in ? ld_f32x4(reinterpret_cast<const float4 *>(W) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        q[t] = in ? ld_f32x4(reinterpret_cast<const float4 *>(What) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float m = 0.0f;
#pragma unroll
    for (int t = 0; t < DELTA_VEC_PER_THREAD; ++t)
        m = fmaxf(m, fmaxf(fmaxf(fabsf(w[t].x - q[t].x), fabsf(w[t].y - q[t].y)),
                           fmaxf(fabsf(w[t].z - q[t].z), fabsf(w[t].w - q[t].w))));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    __shared__ float red[8];
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w8 = 1; w8 < 8; ++w8) m = fmaxf(m, red[w8]);
        // NaN never wins fmaxf; an infinite difference gives 0x7f800000 and the shift below saturates
        if (m > 0.0f) atomicMax(&header->absmax_bits, __float_as_uint(m));
    }
}

// The power of two e for a layer whose largest |delta| has the bit pattern `bits`.
__device__ __forceinline__ int gram_dot_shift(unsigned int bits)
{
    if (bits == 0u) return 0;
    int k = static_cast<int>((bits >> 23) & 0xffu) - 127;          // floor(log2(max)) for normal values
    if (k < -126) k = -126;
    int e = GD_TARGET_EXP - k;
    if (e > GD_MAX_SHIFT) e = GD_MAX_SHIFT;
    if (e < -GD_MAX_SHIFT) e = -GD_MAX_SHIFT;
    return e;
}

// out = fp16((W - W_hat) * 2^e), round to nearest; the chosen e is stored in the header.  Blocks walk the matrices
// from the END towards the start: what the maximum pass read last is still in L2.
__global__ void __launch_bounds__(256)
delta_half_kernel(const float *__restrict__ W, const float *__restrict__ What, unsigned count4, GramDotHeader *header,
                  __half *__restrict__ out)
{
    const unsigned blk = gridDim.x - 1u - blockIdx.x;
    const unsigned base = blk * (256u * DELTA_VEC_PER_THREAD) + threadIdx.x;
    float4 w[DELTA_VEC_PER_THREAD], q[DELTA_VEC_PER_THREAD];
#pragma unroll
    for (int t = 0; t < DELTA_VEC_PER_THREAD; ++t) {
        const unsigned idx = base + t * 256u;
        const bool in = idx < count4;
        w[t] = in ? ld_f32x4_last_use(reinterpret_cast<const float4 *>(W) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        q[t] = in ? ld_f32x4_last_use(reinterpret_cast<const float4 *>(What) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int e = gram_dot_shift(header->absmax_bits);
    if (blockIdx.x == 0 && threadIdx.x == 0) header->shift = e;
    const float scale = __uint_as_float(static_cast<unsigned int>(127 + e) << 23);
#pragma unroll
    for (int t = 0; t < DELTA_VEC_PER_THREAD; ++t) {
        const unsigned idx = base + t * 256u;
        if (idx >= count4) continue;
        uint2 o;
        __half2 *h = reinterpret_cast<__half2 *>(&o);
        h[0] = __floats2half2_rn((w[t].x - q[t].x) * scale, (w[t].y - q[t].y) * scale);
        h[1] = __floats2half2_rn((w[t].z - q[t].z) * scale, (w[t].w - q[t].w) * scale);
        reinterpret_cast<uint2 *>(out)[idx] = o;
    }
}

// loss[k] = 2^(-2e) * sum over the group's partial sums (block k), loss[g] = sum_k loss[k] (formed, in group order,
// by whichever block finishes last).  Every sum is formed in a fixed order (strided per thread, butterfly per warp,
// warp results in order), so the result does not vary from run to run.  partials: [g][slots][per_unit] (units are
// numbered group-major).  header->blocks_done must be 0 before the launch.
__global__ void __launch_bounds__(256)
gram_dot_reduce_kernel(const double *__restrict__ partials, int slots, int g, int per_unit, GramDotHeader *header,
                       double *__restrict__ loss)
{
    __shared__ double warp_sum[8];
    __shared__ bool last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int k = blockIdx.x;
    const double *pk = partials + static_cast<size_t>(k) * slots * per_unit;
    const int count = slots * per_unit;
    double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
    int idx = threadIdx.x;
    for (; idx + 768 < count; idx += 1024) {               // four independent loads in flight
        acc0 += pk[idx];
        acc1 += pk[idx + 256];
        acc2 += pk[idx + 512];
        acc3 += pk[idx + 768];
    }
    for (; idx < count; idx += 256) acc0 += pk[idx];
    double acc = (acc0 + acc1) + (acc2 + acc3);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) warp_sum[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double v = 0.0;
        for (int w8 = 0; w8 < 8; ++w8) v += warp_sum[w8];
        loss[k] = v * ldexp(1.0, -2 * header->shift);
        __threadfence();
        last = atomicAdd(&header->blocks_done, 1u) == static_cast<unsigned int>(g) - 1u;
        if (last) {
            __threadfence();
            double total = 0.0;
            for (int kk = 0; kk < g; ++kk) total += *const_cast<volatile double *>(loss + kk);
            loss[g] = total;
        }
    }
}

struct GramUnit {
    int ti, tj;      // tile (row block, column block), ti <= tj
    int k;           // group
};

__device__ __forceinline__ GramUnit gram_unit(const GramDotParams &p, int unit)
{
    GramUnit u;
    u.k = unit / p.tiles;
    tile_of_slot_blocked(unit - u.k * p.tiles, p.nj, p.raster, u.ti, u.tj);
    return u;
}

// mapD: fp16 [g][rows][d] (64-feature x 64-row boxes, 128-byte swizzle), the prepared Delta of every group.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GD_THREADS, 1)
gram_dot_kernel(const __grid_constant__ CUtensorMap mapD, const GramDotParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[GD_STAGES];     // first CTA: bytes of both CTAs
    __shared__ __align__(8) uint64_t bar_empty[GD_STAGES];    // both CTAs: signalled by the MMA commits
    __shared__ __align__(8) uint64_t bar_acc_full[2];         // both CTAs, one per accumulator: signalled by the MMA commit
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
        for (int s = 0; s < GD_STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int kk = 0; kk < 2; ++kk) {
            mbar_init(smem_u32(&bar_acc_full[kk]), 1);
            mbar_init(smem_u32(&bar_acc_empty[kk]), 2 * GD_EPI_WARPS);
        }
        mbar_init(smem_u32(&bar_drain), 1);
        abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&mapD);
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

    if (warp < 4) {
        // The service warpgroup keeps 40 registers per thread; the rest goes to the epilogue warpgroups.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
        if (warp == 0 && lane == 0) {
            // -------------------------------------------------------------- TMA producer (both CTAs)
            int s = 0;
            uint32_t ph = 0;
            uint32_t issued = 0;
            bool ok = true;
            WorkItem w;
            for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
                const GramUnit u = gram_unit(p, w.unit);
                const int a0 = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS;
                const int b0 = u.tj * TILE_N + static_cast<int>(rank) * CTA_ROWS;
                for (int ks = w.ks0; ks < w.ks1; ++ks) {
                    const int row = ks * TILE_K;
                    if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 1u, w.unit)) { ok = false; break; }
                    const uint32_t full_local = smem_u32(&bar_full[s]);
                    if (rank == 0) mbar_arrive_expect_tx(full_local, 2 * GD_STAGE_BYTES);      // both CTAs' bytes
                    const uint32_t full = map_to_cta(full_local, 0);
                    const uint32_t stage = ring + s * GD_STAGE_BYTES;
#pragma unroll
                    for (int q = 0; q < CTA_ROWS / BOX_FEATURES; ++q) {
                        tma_load_3d_pair(stage + q * BOX_BYTES, &mapD, full, a0 + q * BOX_FEATURES, row, u.k);
                        tma_load_3d_pair(stage + GD_SLOT_BYTES + q * BOX_BYTES, &mapD, full, b0 + q * BOX_FEATURES, row, u.k);
                    }
                    ++issued;
                    if (++s == GD_STAGES) { s = 0; ph ^= 1u; }
                }
            }
            // Stay until every stage has been released again: the release is an arrival on this CTA's barriers,
            // which must not come after the CTA has gone.
            for (int q = 0; ok && issued != 0u && q < GD_STAGES; ++q) {
                if (!bounded_wait(smem_u32(&bar_empty[s]), ph ^ 1u, wc, 5u, 0u)) ok = false;
                if (++s == GD_STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) spin_ns(1000000ull);
        } else if (warp == 1 && lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (first CTA)
            constexpr uint32_t idesc = umma_idesc_f16_mn(TILE_M, TILE_N);
            int s = 0;
            uint32_t ph = 0;
            uint32_t acc_ph[2] = {0u, 0u};
            bool ok = true;
            WorkItem w;
            for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
                const int buf = it & 1;
                // the accumulator of unit it - 2 must have been read out
                if (!bounded_wait_hot(smem_u32(&bar_acc_empty[buf]), acc_ph[buf] ^ 1u, wc, 2u, w.unit)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * TILE_N);
                for (int ks = w.ks0; ks < w.ks1; ++ks) {
                    if (!bounded_wait_hot(smem_u32(&bar_full[s]), ph, wc, 3u, w.unit)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sa = ring + s * GD_STAGE_BYTES;
                    const uint32_t sb = sa + GD_SLOT_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < TILE_K / 16; ++k16) {
                        const uint64_t adesc = umma_smem_desc_mn_sw128(sa + k16 * 16 * 128, BOX_BYTES, 1024);
                        const uint64_t bdesc = umma_smem_desc_mn_sw128(sb + k16 * 16 * 128, BOX_BYTES, 1024);
                        umma_bf16(d_tmem, adesc, bdesc, idesc, (ks != w.ks0 || k16 != 0) ? 1u : 0u);
                    }
                    umma_commit_pair(smem_u32(&bar_empty[s]));
                    if (++s == GD_STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair(smem_u32(&bar_acc_full[buf]));
                acc_ph[buf] ^= 1u;
            }
            if (!ok) {
                // Make sure no MMA is still writing TMEM when it is released.
                umma_commit_local(smem_u32(&bar_drain));
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&bar_drain), 0u) && global_timer_ns() - t0 < 5000000ull) {}
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
        // ------------------------------------------------------------------ epilogue: partial = <accumulator, H>
        const int ew = warp - 4;                        // 0..7
        const int q = warp & 3;                         // TMEM lane quarter this warp may access
        const int half = ew >> 2;                       // which 128 of the 256 accumulator columns
        uint32_t full_ph[2] = {0u, 0u};
        bool ok = true;
        WorkItem w;
        for (int it = 0; ok && work_item(p.sched, pair, it, w); ++it) {
            const int buf = it & 1;
            const GramUnit u = gram_unit(p, w.unit);
            const int row0 = u.ti * TILE_M + static_cast<int>(rank) * CTA_ROWS + q * 32;
            const int row = row0 + lane;
            // sum_{a <= b} (2 - [a == b]) D[a][b] H_k[a][b] over this warp's four 32 x 32 blocks of the tile:
            // block j covers columns tj * 256 + (half * 4 + j) * 32 .. + 31.
            const bool row_ok = row < p.d;
            const float *hrow = p.H + (static_cast<size_t>(u.k) * p.d + (row_ok ? row : 0)) * static_cast<size_t>(p.d);
            const int colw = u.tj * TILE_N + half * 128;
            // uniform over the warp: does block j hold entries on or above the diagonal inside the matrix?
            auto block_active = [&](int j) { return colw + j * 32 < p.d && row0 < p.d && colw + j * 32 + 32 > row0; };
            // All four blocks of H are requested now, while the tensor core is still working on this tile.
            float hq[4][4][8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool act = row_ok && block_active(j);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const int c = colw + j * 32 + v * 8;
                    if (act && c < p.d && c + 7 >= row) {
                        ld_stream_f32x8(hrow + c, hq[j][v]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) hq[j][v][e] = 0.0f;
                    }
                }
            }
            if (lane == 0) ok = bounded_wait(smem_u32(&bar_acc_full[buf]), full_ph[buf], wc, 4u, w.unit);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            (void)mbar_try_wait(smem_u32(&bar_acc_full[buf]), full_ph[buf]);     // every lane observes the completed phase
            full_ph[buf] ^= 1u;
            tc_fence_after_sync();
            const uint32_t tmem_tile = tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                       static_cast<uint32_t>(buf * TILE_N + half * 128);
            double dsum = 0.0;
            uint32_t r[2][32];
            tmem_ld_32x32(tmem_tile, r[0]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                tmem_ld_wait();
                if (j < 3) {
                    tmem_ld_32x32(tmem_tile + static_cast<uint32_t>((j + 1) * 32), r[(j + 1) & 1]);
                } else {
                    // This warp holds all it needs from the accumulator: hand it back to the MMA issuer (first CTA).
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
                }
                if (block_active(j)) {
                    const int col0 = colw + j * 32;
                    float part = 0.0f;
                    if (col0 > row0 + 31) {
                        // the whole block lies above the diagonal: every entry counts twice
#pragma unroll
                        for (int v = 0; v < 4; ++v)
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                part = fmaf(__uint_as_float(r[j & 1][v * 8 + e]), hq[j][v][e], part);
                        part *= 2.0f;
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v)
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int c = col0 + v * 8 + e;
                                const float wgt = (c > row) ? 2.0f : ((c == row) ? 1.0f : 0.0f);
                                part = fmaf(wgt * __uint_as_float(r[j & 1][v * 8 + e]), hq[j][v][e], part);
                            }
                    }
                    dsum += static_cast<double>(part);
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
            if (lane == 0)
                p.partials[static_cast<size_t>(w.unit) * GD_PARTIALS_PER_UNIT + rank * GD_EPI_WARPS + ew] = dsum;
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
