// Cyclic coordinate descent with fixed codebooks on the guided layer objective
// (Section 4.2, Eq. 10; Appendix B.2, Algorithms 3 and 4): the kernels around the tensor-core panel product.
//
// For every group k and channel j in J_k, coordinates i = 0 .. d_in - 1 in order are set to
//     Round_j( W_ij - (1 / H_ii) * sum_{c != i} H_ic * E_cj ),     E = What - W  (current values),
// all channels in parallel.  The coordinates are processed in blocks of CD_BLOCK = 256 (the lazy batch of
// Algorithm 4).  For a block starting at s0 the sum splits into
//   - c outside the block: one tensor-core product per block, P = H[block rows, outside] * E[outside]
//     (pair_gemm_kernel<MODE_PANEL>); rows before the block already hold this cycle's values, rows after it
//     the previous cycle's - exactly what Algorithm 4's B holds for these rows when the block is reached;
//   - c inside the block: done here, sequentially, by cd_block_kernel.
// (Algorithm 4 pushes a finished block's correction to all later rows; here every block pulls the
// contributions of all other rows just before it is processed.  The sums are the same; only their order
// differs, and B never has to exist for more than one block.)
//
// Work arrays are coordinate-major ([d_in][d_out], the paper's orientation) so that one coordinate of all
// channels is contiguous; W, What and the codes are transposed on the way in and out.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace gq {

constexpr int CD_BLOCK = 256;           // coordinates per block
constexpr int CD_CH = 32;               // channels per CTA of the block kernel
constexpr int CD_LANES = 8;             // threads per channel
constexpr int CD_THREADS = CD_CH * CD_LANES;
constexpr int CD_MAX_LEVELS = 16;       // codebook entries per channel (m = 2^b, b <= 4)
constexpr int CD_TILE_LD = CD_CH + 1;   // padded row of the [CD_BLOCK][CD_CH] shared-memory tiles
constexpr int CD_HCHUNK = 32;           // rows of the block's Hessian staged at a time
constexpr int CD_SMEM_BYTES = (3 * CD_BLOCK * CD_TILE_LD + 2 * CD_HCHUNK * CD_BLOCK + CD_BLOCK + 2 * CD_CH * CD_MAX_LEVELS) * 4;

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16 &hi, __nv_bfloat16 &lo)
{
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Wt = W^T, Wht = What^T, E = Wht - Wt (fp32 and as bf16 hi + lo), all [d_in][d_out].  32 x 32 tiles.
__global__ void __launch_bounds__(256)
cd_prepare_kernel(const float *__restrict__ W, const float *__restrict__ What, int d_in, int d_out,
                  float *__restrict__ Wt, float *__restrict__ Wht, float *__restrict__ Et,
                  __nv_bfloat16 *__restrict__ Ehi, __nv_bfloat16 *__restrict__ Elo)
{
    __shared__ float tw[32][33], th[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;          // coordinate / channel origin
    for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, i = i0 + tx;
        const bool ok = j < d_out && i < d_in;
        tw[r][tx] = ok ? W[static_cast<size_t>(j) * d_in + i] : 0.0f;
        th[r][tx] = ok ? What[static_cast<size_t>(j) * d_in + i] : 0.0f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int i = i0 + r, j = j0 + tx;
        if (i < d_in && j < d_out) {
            const float w = tw[tx][r], h = th[tx][r], e = h - w;
            const size_t o = static_cast<size_t>(i) * d_out + j;
            Wt[o] = w;
            Wht[o] = h;
            Et[o] = e;
            __nv_bfloat16 hi, lo;
            split_bf16(e, hi, lo);
            Ehi[o] = hi;
            Elo[o] = lo;
        }
    }
}

// H -> bf16 hi + lo (operands of the panel product) and rdiag[k][i] = 1 / H_k[i][i] (0 where H_ii <= 0).
__global__ void __launch_bounds__(256)
cd_split_h_kernel(const float *__restrict__ H, long long count, int d_in, __nv_bfloat16 *__restrict__ Hhi,
                  __nv_bfloat16 *__restrict__ Hlo, float *__restrict__ rdiag)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < count; idx += stride) {
        const float v = H[idx];
        __nv_bfloat16 hi, lo;
        split_bf16(v, hi, lo);
        Hhi[idx] = hi;
        Hlo[idx] = lo;
        const long long within = idx % (static_cast<long long>(d_in) * d_in);
        const int r = static_cast<int>(within / d_in), c = static_cast<int>(within - static_cast<long long>(r) * d_in);
        if (r == c) rdiag[idx / (static_cast<long long>(d_in) * d_in) * d_in + r] = v > 0.0f ? 1.0f / v : 0.0f;
    }
}

// What = Wht^T, Q = Qt^T back to [d_out][d_in].
__global__ void __launch_bounds__(256)
cd_finish_kernel(const float *__restrict__ Wht, const uint8_t *__restrict__ Qt, int d_in, int d_out,
                 float *__restrict__ What, uint8_t *__restrict__ Q)
{
    __shared__ float th[32][33];
    __shared__ uint8_t tq[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    for (int r = ty; r < 32; r += 8) {
        const int i = i0 + r, j = j0 + tx;
        const bool ok = i < d_in && j < d_out;
        th[r][tx] = ok ? Wht[static_cast<size_t>(i) * d_out + j] : 0.0f;
        tq[r][tx] = ok ? Qt[static_cast<size_t>(i) * d_out + j] : 0;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, i = i0 + tx;
        if (j < d_out && i < d_in) {
            What[static_cast<size_t>(j) * d_in + i] = th[tx][r];
            Q[static_cast<size_t>(j) * d_in + i] = tq[tx][r];
        }
    }
}

struct CdBlockParams {
    const float *H;          // [g][d_in][d_in] full symmetric
    const float *rdiag;      // [g][d_in]
    const float *P;          // [CD_BLOCK][d_out]: contributions of the coordinates outside the block
    const float *Wt;         // [d_in][d_out]
    const float *codebook;   // [d_out][m]
    float *Wht;              // [d_in][d_out]
    float *Et;               // [d_in][d_out]
    __nv_bfloat16 *Ehi, *Elo;
    uint8_t *Qt;             // [d_in][d_out]
    int d_in, d_out, g, mk, m;
    int s0;                  // first coordinate of the block
    int rows;                // coordinates in the block (<= CD_BLOCK)
    int slices;              // ceil(mk / CD_CH): CTAs per group
};

// One block of coordinates for CD_CH channels of one group.  Eight threads share a channel; thread l of
// them owns the rows 32 t + 4 l + e (band t < 8, e < 4) of the running sums
//     Bu[r] = sum_{c != r} H[r][c] * E_c      (current E: this cycle's values for c < r, last cycle's for c > r).
// Pass 1 adds the in-block part of last cycle's values (c > r).  Pass 2 walks the rows in order; per row i:
//   * the owner hands the rounding target W_i - Bu[i] / H_ii to the channel's threads (one shuffle);
//   * Round_j: the channel's levels are kept sorted, thread l holding the thresholds between the sorted levels
//     2l, 2l+1 and 2l+1, 2l+2 (their midpoints, lowered by one ulp where the upper level has the smaller
//     original index, so that an exact tie goes to the smaller index); the nearest level is at sorted position
//     #{q : target > thr_q}: two compares and two warp votes per thread, one table read;
//   * every thread adds H[i][r] * E_i to those of its rows that come after i.
// H[i][.] rows come through shared memory in chunks of 32 (= one band).  The codes are recovered at the end as
// the first level, in the codebook's given order, that equals the chosen value.
__global__ void __launch_bounds__(CD_THREADS, 1)
cd_block_kernel(const CdBlockParams p)
{
    extern __shared__ float smem_f[];
    float *Ws = smem_f;                                  // [CD_BLOCK][CD_TILE_LD]  W of the block
    float *Es = Ws + CD_BLOCK * CD_TILE_LD;              // E of the block, updated in place
    float *Xs = Es + CD_BLOCK * CD_TILE_LD;              // first P (pulled sums), then What of the block
    float *Hs = Xs + CD_BLOCK * CD_TILE_LD;              // [2][CD_HCHUNK][CD_BLOCK]
    float *rds = Hs + 2 * CD_HCHUNK * CD_BLOCK;          // [CD_BLOCK]
    float *cbs = rds + CD_BLOCK;                         // [CD_CH][CD_MAX_LEVELS] codebooks in their given order
    float *srt = cbs + CD_CH * CD_MAX_LEVELS;            // [CD_CH][CD_MAX_LEVELS] the same, sorted

    const int tid = threadIdx.x;
    const int k = blockIdx.x / p.slices;
    const int ch0 = k * p.mk + (blockIdx.x % p.slices) * CD_CH;          // first channel of this CTA
    const int ch_n = min(CD_CH, (k + 1) * p.mk - ch0);                   // valid channels
    const int cidx = tid / CD_LANES, l = tid % CD_LANES;
    const int group_shift = 8 * ((tid >> 3) & 3);                       // where this channel's eight threads sit in a warp vote
    const float *Hk = p.H + static_cast<size_t>(k) * p.d_in * p.d_in;

    // ---- tiles in: 32 channels x 256 coordinates, coalesced over channels
    for (int idx = tid; idx < CD_BLOCK * CD_CH; idx += CD_THREADS) {
        const int r = idx / CD_CH, c = idx % CD_CH;
        const bool ok = r < p.rows && c < ch_n;
        const size_t o = static_cast<size_t>(p.s0 + r) * p.d_out + ch0 + c;
        Ws[r * CD_TILE_LD + c] = ok ? p.Wt[o] : 0.0f;
        Es[r * CD_TILE_LD + c] = ok ? p.Et[o] : 0.0f;
        Xs[r * CD_TILE_LD + c] = ok ? p.P[static_cast<size_t>(r) * p.d_out + ch0 + c] : 0.0f;
    }
    for (int r = tid; r < CD_BLOCK; r += CD_THREADS)
        rds[r] = r < p.rows ? p.rdiag[static_cast<size_t>(k) * p.d_in + p.s0 + r] : 0.0f;

    // rows [c0, c0 + CD_HCHUNK) of the block's H (columns of the block only) into buffer b, zero outside the
    // block; asynchronous copies (cp.async), completed by h_chunk_wait() before the next __syncthreads
    auto load_h_chunk = [&](int c0, int b) {
        float *dst = Hs + b * CD_HCHUNK * CD_BLOCK;
        for (int idx = tid; idx < CD_HCHUNK * CD_BLOCK / 4; idx += CD_THREADS) {
            const int rr = idx / (CD_BLOCK / 4), cc = (idx % (CD_BLOCK / 4)) * 4;
            float *d = dst + rr * CD_BLOCK + cc;
            if (c0 + rr < p.rows && cc < p.rows) {    // rows is a multiple of 8 (d_in % 8 == 0): whole float4 in range
                const float *src = Hk + static_cast<size_t>(p.s0 + c0 + rr) * p.d_in + p.s0 + cc;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(
                                 __cvta_generic_to_shared(d))), "l"(src) : "memory");
            } else {
                *reinterpret_cast<float4 *>(d) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto h_chunk_wait = [&]() { asm volatile("cp.async.wait_group 0;" ::: "memory"); };

    // ---- the channel's levels: given order (cbs), sorted (srt), this thread's two thresholds
    static_assert(CD_MAX_LEVELS == 2 * CD_LANES, "two codebook levels per thread");
    float thr_a = CUDART_INF_F, thr_b = CUDART_INF_F;
    {
        const bool chan = cidx < ch_n;
        const float v0 = (l < p.m && chan) ? p.codebook[static_cast<size_t>(ch0 + cidx) * p.m + l] : CUDART_INF_F;
        const float v1 = (l + 8 < p.m && chan) ? p.codebook[static_cast<size_t>(ch0 + cidx) * p.m + l + 8] : CUDART_INF_F;
        int rank0 = 0, rank1 = 0;                        // positions of (v0, l) and (v1, l + 8) among the 16 pairs
#pragma unroll
        for (int r = 0; r < CD_MAX_LEVELS; ++r) {
            const float vr = __shfl_sync(0xffffffffu, r < 8 ? v0 : v1, r & 7, CD_LANES);
            rank0 += (vr < v0 || (vr == v0 && r < l)) ? 1 : 0;
            rank1 += (vr < v1 || (vr == v1 && r < l + 8)) ? 1 : 0;
        }
        int *sidx = reinterpret_cast<int *>(Hs);         // [CD_CH][CD_MAX_LEVELS] original index by sorted position
        float *mc = cbs + cidx * CD_MAX_LEVELS, *ms = srt + cidx * CD_MAX_LEVELS;
        int *mi = sidx + cidx * CD_MAX_LEVELS;
        mc[l] = v0;
        mc[l + 8] = v1;
        ms[rank0] = v0;
        mi[rank0] = l;
        ms[rank1] = v1;
        mi[rank1] = l + 8;
        __syncwarp();
        auto threshold = [&](int q) {                    // between sorted levels q and q + 1
            const float mid = 0.5f * (ms[q] + ms[q + 1]);
            return (mi[q] < mi[q + 1] || !(fabsf(mid) < CUDART_INF_F)) ? mid : nextafterf(mid, -CUDART_INF_F);
        };
        thr_a = threshold(2 * l);
        if (2 * l + 2 < CD_MAX_LEVELS) thr_b = threshold(2 * l + 1);
    }
    const float *my_levels = srt + cidx * CD_MAX_LEVELS;
    __syncthreads();                                     // sidx (in the H buffer) has been read by everybody

    load_h_chunk(0, 0);
    h_chunk_wait();
    __syncthreads();

    float Bu[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) Bu[t][e] = Xs[(32 * t + 4 * l + e) * CD_TILE_LD + cidx];

    // ---- pass 1: Bu[r] += sum_{c in block, c > r} H[c][r] * E_old[c]
    // (The 32-row bands t are unrolled so that Bu is indexed statically; the rows inside a band are a real
    // loop - unrolling all 256 steps makes the code larger than the instruction cache and ten times slower.)
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        if (t + 1 < 8) load_h_chunk((t + 1) * CD_HCHUNK, (t + 1) & 1);
        const float *hc = Hs + (t & 1) * CD_HCHUNK * CD_BLOCK;
#pragma unroll 1
        for (int ii = 0; ii < 32; ++ii) {
            const float ec = Es[(32 * t + ii) * CD_TILE_LD + cidx];
#pragma unroll
            for (int tp = 0; tp <= t; ++tp) {
                const float4 h = *reinterpret_cast<const float4 *>(hc + ii * CD_BLOCK + 32 * tp + 4 * l);
                if (tp < t) {
                    Bu[tp][0] = fmaf(h.x, ec, Bu[tp][0]);
                    Bu[tp][1] = fmaf(h.y, ec, Bu[tp][1]);
                    Bu[tp][2] = fmaf(h.z, ec, Bu[tp][2]);
                    Bu[tp][3] = fmaf(h.w, ec, Bu[tp][3]);
                } else {                                  // same 32-row band: only rows before c
                    if (4 * l + 0 < ii) Bu[tp][0] = fmaf(h.x, ec, Bu[tp][0]);
                    if (4 * l + 1 < ii) Bu[tp][1] = fmaf(h.y, ec, Bu[tp][1]);
                    if (4 * l + 2 < ii) Bu[tp][2] = fmaf(h.z, ec, Bu[tp][2]);
                    if (4 * l + 3 < ii) Bu[tp][3] = fmaf(h.w, ec, Bu[tp][3]);
                }
            }
        }
        h_chunk_wait();
        __syncthreads();
    }

    // ---- pass 2: the coordinates in order
    load_h_chunk(0, 0);
    h_chunk_wait();
    __syncthreads();
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        if (t + 1 < 8) load_h_chunk((t + 1) * CD_HCHUNK, (t + 1) & 1);
        const float *hc = Hs + (t & 1) * CD_HCHUNK * CD_BLOCK;
#pragma unroll 1
        for (int i4 = 0; i4 < 32; i4 += 4) {
            const int owner = i4 >> 2;                    // the thread that owns rows 32 t + i4 .. + 3
            const bool after = l > owner, mine = l == owner;
            const float4 h4[4] = {*reinterpret_cast<const float4 *>(hc + (i4 + 0) * CD_BLOCK + 32 * t + 4 * l),
                                  *reinterpret_cast<const float4 *>(hc + (i4 + 1) * CD_BLOCK + 32 * t + 4 * l),
                                  *reinterpret_cast<const float4 *>(hc + (i4 + 2) * CD_BLOCK + 32 * t + 4 * l),
                                  *reinterpret_cast<const float4 *>(hc + (i4 + 3) * CD_BLOCK + 32 * t + 4 * l)};
#pragma unroll
            for (int oe = 0; oe < 4; ++oe) {
                const int i = 32 * t + i4 + oe;
                const float w = Ws[i * CD_TILE_LD + cidx];
                const float target = __shfl_sync(0xffffffffu, w - rds[i] * Bu[t][oe], owner, CD_LANES);
                // the thresholds ascend, so the number of thresholds below the target is the level's position
                const unsigned below_a = __ballot_sync(0xffffffffu, target > thr_a);
                const unsigned below_b = __ballot_sync(0xffffffffu, target > thr_b);
                const int pos = __popc((below_a >> group_shift) & 0xffu) + __popc((below_b >> group_shift) & 0xffu);
                const float val = my_levels[pos];
                const float e_new = val - w;
                if (mine) {
                    Es[i * CD_TILE_LD + cidx] = e_new;
                    Xs[i * CD_TILE_LD + cidx] = val;
                }
                // same band: only rows after i (a zero factor instead of a branch)
                const float4 h = h4[oe];
                const float e_after = after ? e_new : 0.0f, e_from = (after || mine) ? e_new : 0.0f;
                Bu[t][0] = fmaf(h.x, 0 > oe ? e_from : e_after, Bu[t][0]);
                Bu[t][1] = fmaf(h.y, 1 > oe ? e_from : e_after, Bu[t][1]);
                Bu[t][2] = fmaf(h.z, 2 > oe ? e_from : e_after, Bu[t][2]);
                Bu[t][3] = fmaf(h.w, 3 > oe ? e_from : e_after, Bu[t][3]);
#pragma unroll
                for (int tp = t + 1; tp < 8; ++tp) {      // later bands: all rows
                    const float4 hh = *reinterpret_cast<const float4 *>(hc + (i4 + oe) * CD_BLOCK + 32 * tp + 4 * l);
                    Bu[tp][0] = fmaf(hh.x, e_new, Bu[tp][0]);
                    Bu[tp][1] = fmaf(hh.y, e_new, Bu[tp][1]);
                    Bu[tp][2] = fmaf(hh.z, e_new, Bu[tp][2]);
                    Bu[tp][3] = fmaf(hh.w, e_new, Bu[tp][3]);
                }
            }
        }
        h_chunk_wait();
        __syncthreads();
    }

    // ---- tiles out
    for (int idx = tid; idx < CD_BLOCK * CD_CH; idx += CD_THREADS) {
        const int r = idx / CD_CH, c = idx % CD_CH;
        if (r < p.rows && c < ch_n) {
            const size_t o = static_cast<size_t>(p.s0 + r) * p.d_out + ch0 + c;
            const float e = Es[r * CD_TILE_LD + c];
            const float val = Xs[r * CD_TILE_LD + c];
            int code = 0;                                 // first level, in the given order, with this value
#pragma unroll
            for (int q = CD_MAX_LEVELS - 1; q >= 0; --q)
                if (cbs[c * CD_MAX_LEVELS + q] == val) code = q;
            p.Et[o] = e;
            p.Wht[o] = val;
            p.Qt[o] = static_cast<uint8_t>(code);
            __nv_bfloat16 hi, lo;
            split_bf16(e, hi, lo);
            p.Ehi[o] = hi;
            p.Elo[o] = lo;
        }
    }
}

}  // namespace gq
