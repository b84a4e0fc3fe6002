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
#include <stdint.h>

namespace gq {

constexpr int CD_BLOCK = 256;           // coordinates per block
constexpr int CD_CH = 32;               // channels per CTA of the block kernel
constexpr int CD_LANES = 8;             // threads per channel
constexpr int CD_THREADS = CD_CH * CD_LANES;
constexpr int CD_MAX_LEVELS = 16;       // codebook entries per channel (m = 2^b, b <= 4)
constexpr int CD_TILE_LD = CD_CH + 1;   // padded row of the [CD_BLOCK][CD_CH] shared-memory tiles
constexpr int CD_HCHUNK = 32;           // rows of the block's Hessian staged at a time
constexpr int CD_SMEM_BYTES = (3 * CD_BLOCK * CD_TILE_LD + 2 * CD_HCHUNK * CD_BLOCK + CD_BLOCK) * 4 + CD_BLOCK * CD_CH;

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
// them owns the rows 32 t + 4 l + e (t < 8, e < 4) of the running sums
//     Bu[r] = sum_{c != r} H[r][c] * E_c      (current E: this cycle's values for c < r, last cycle's for c > r).
// Pass 1 adds the in-block part of last cycle's values (c > r), pass 2 walks the rows in order: the owner of
// row i hands W_i - Bu[i] / H_ii to its seven neighbours, the eight of them find the nearest codebook level
// (ties to the smaller index), and every thread adds H[i][r] * E_i to its rows r > i.  H[i][.] rows come
// through shared memory in chunks of 32.
__global__ void __launch_bounds__(CD_THREADS, 1)
cd_block_kernel(const CdBlockParams p)
{
    extern __shared__ float smem_f[];
    float *Ws = smem_f;                                  // [CD_BLOCK][CD_TILE_LD]  W of the block
    float *Es = Ws + CD_BLOCK * CD_TILE_LD;              // E of the block, updated in place
    float *Xs = Es + CD_BLOCK * CD_TILE_LD;              // first P (pulled sums), then What of the block
    float *Hs = Xs + CD_BLOCK * CD_TILE_LD;              // [2][CD_HCHUNK][CD_BLOCK]
    float *rds = Hs + 2 * CD_HCHUNK * CD_BLOCK;          // [CD_BLOCK]
    uint8_t *Qs = reinterpret_cast<uint8_t *>(rds + CD_BLOCK);   // [CD_BLOCK][CD_CH]

    const int tid = threadIdx.x;
    const int k = blockIdx.x / p.slices;
    const int ch0 = k * p.mk + (blockIdx.x % p.slices) * CD_CH;          // first channel of this CTA
    const int ch_n = min(CD_CH, (k + 1) * p.mk - ch0);                   // valid channels
    const int cidx = tid / CD_LANES, l = tid % CD_LANES;
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

    // codebook levels l and l + 8 of this thread's channel (the eight threads of a channel hold all sixteen)
    static_assert(CD_MAX_LEVELS == 2 * CD_LANES, "two codebook levels per thread");
    const float cb0 = (l < p.m && cidx < ch_n) ? p.codebook[static_cast<size_t>(ch0 + cidx) * p.m + l] : 0.0f;
    const float cb1 = (l + 8 < p.m && cidx < ch_n) ? p.codebook[static_cast<size_t>(ch0 + cidx) * p.m + l + 8] : 0.0f;

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
        for (int ii = 0; ii < 32; ++ii) {
            const int i = 32 * t + ii;
            const int owner = ii >> 2, oe = ii & 3;
            // the owner of row i forms the rounding target; all eight threads of the channel find the nearest
            // codebook level together (two levels each, then a three-step minimum; ties: the smaller index)
            const float bu = oe == 0 ? Bu[t][0] : (oe == 1 ? Bu[t][1] : (oe == 2 ? Bu[t][2] : Bu[t][3]));
            const float w = Ws[i * CD_TILE_LD + cidx];
            const float target = __shfl_sync(0xffffffffu, w - rds[i] * bu, owner, CD_LANES);
            const float d0 = l < p.m ? fabsf(target - cb0) : 3.0e38f;
            const float d1 = l + 8 < p.m ? fabsf(target - cb1) : 3.0e38f;
            float bd = d1 < d0 ? d1 : d0;                 // equal distances keep the smaller index l
            int best = d1 < d0 ? l + 8 : l;
            float val = d1 < d0 ? cb1 : cb0;
#pragma unroll
            for (int off = 1; off < CD_LANES; off <<= 1) {
                const float od = __shfl_xor_sync(0xffffffffu, bd, off, CD_LANES);
                const int ob = __shfl_xor_sync(0xffffffffu, best, off, CD_LANES);
                const float ov = __shfl_xor_sync(0xffffffffu, val, off, CD_LANES);
                if (od < bd || (od == bd && ob < best)) { bd = od; best = ob; val = ov; }
            }
            const float e_new = val - w;
            if (l == owner) {
                Es[i * CD_TILE_LD + cidx] = e_new;
                Xs[i * CD_TILE_LD + cidx] = val;
                Qs[i * CD_CH + cidx] = static_cast<uint8_t>(best);
            }
#pragma unroll
            for (int tp = t; tp < 8; ++tp) {
                const float4 h = *reinterpret_cast<const float4 *>(hc + ii * CD_BLOCK + 32 * tp + 4 * l);
                if (tp > t) {
                    Bu[tp][0] = fmaf(h.x, e_new, Bu[tp][0]);
                    Bu[tp][1] = fmaf(h.y, e_new, Bu[tp][1]);
                    Bu[tp][2] = fmaf(h.z, e_new, Bu[tp][2]);
                    Bu[tp][3] = fmaf(h.w, e_new, Bu[tp][3]);
                } else {                                  // same band: only rows after i
                    if (4 * l + 0 > ii) Bu[tp][0] = fmaf(h.x, e_new, Bu[tp][0]);
                    if (4 * l + 1 > ii) Bu[tp][1] = fmaf(h.y, e_new, Bu[tp][1]);
                    if (4 * l + 2 > ii) Bu[tp][2] = fmaf(h.z, e_new, Bu[tp][2]);
                    if (4 * l + 3 > ii) Bu[tp][3] = fmaf(h.w, e_new, Bu[tp][3]);
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
            p.Et[o] = e;
            p.Wht[o] = Xs[r * CD_TILE_LD + c];
            p.Qt[o] = Qs[r * CD_CH + c];
            __nv_bfloat16 hi, lo;
            split_bf16(e, hi, lo);
            p.Ehi[o] = hi;
            p.Elo[o] = lo;
        }
    }
}

}  // namespace gq
