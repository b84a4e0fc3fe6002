// Codebook step of the layer-wise quantiser (Section 4.2, Eq. 8; the codebook steps of Algorithm 2): for every
// output channel j of group k, with the assignment matrix P in {0,1}^{d_in x m} given by the codes Q,
//
//     c^(j) = (P^T H_k P + lambda I)^-1  P^T H_k w_j .
//
// The two d_in^2-sized contractions run on the tensor cores (pair_gemm_kernel<MODE_FULL>):
//     HW = H_k W_k^T                      [d_in x channels]
//     HP = H_k [P^(j0) ... P^(j0+c-1)]    [d_in x (channels * m)]   for a slab of channels at a time
// with H and W as bf16 hi + lo pairs (16 significant bits, what is dropped is below 2^-16 of each entry: the
// size of the fp32 accumulation error of these 4096-long sums); accumulation is fp32.  HW takes
// hi hi + hi lo + lo hi; HP, where the one-hot columns are exact in bf16, the two terms of H.  (Three-way
// splits that reproduce the fp32 values exactly were measured to change the codebooks by less than the
// difference to the fp64 oracle that remains either way.)
// The kernels here prepare those operands, fold HP and HW over the rows of each level (fp64),
//     G^(j)[q][q'] = sum_{i : Q_ij = q} HP[i][j m + q'],      r^(j)[q] = sum_{i : Q_ij = q} HW[i][j],
// and solve the m x m systems by Cholesky in fp64.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gq {

constexpr int CB_MAX_LEVELS = 16;
constexpr int CB_SLAB_CHANNELS = 1024;      // channels whose one-hot columns are multiplied at a time

// v = t0 + t1 up to 2^-17 |v|: round to bf16, round the remainder to bf16.
__device__ __forceinline__ void split2_bf16(float v, __nv_bfloat16 &t0, __nv_bfloat16 &t1)
{
    t0 = __float2bfloat16_rn(v);
    t1 = __float2bfloat16_rn(v - __bfloat162float(t0));
}

__global__ void __launch_bounds__(256)
cb_split2_kernel(const float *__restrict__ src, long long count, __nv_bfloat16 *__restrict__ d0,
                 __nv_bfloat16 *__restrict__ d1)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < count; idx += stride) {
        __nv_bfloat16 a, b;
        split2_bf16(src[idx], a, b);
        d0[idx] = a;
        d1[idx] = b;
    }
}

// W [d_out][d_in] -> bf16 hi + lo of W^T [d_in][d_out]; Q [d_out][d_in] -> Qt [d_in][d_out].  32 x 32 tiles.
__global__ void __launch_bounds__(256)
cb_transpose_kernel(const float *__restrict__ W, const uint8_t *__restrict__ Q, int d_in, int d_out,
                    __nv_bfloat16 *__restrict__ W0, __nv_bfloat16 *__restrict__ W1, uint8_t *__restrict__ Qt)
{
    __shared__ float tw[32][33];
    __shared__ uint8_t tq[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int i0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, i = i0 + tx;
        const bool ok = j < d_out && i < d_in;
        tw[r][tx] = ok ? W[static_cast<size_t>(j) * d_in + i] : 0.0f;
        tq[r][tx] = ok ? Q[static_cast<size_t>(j) * d_in + i] : 0;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int i = i0 + r, j = j0 + tx;
        if (i < d_in && j < d_out) {
            const size_t o = static_cast<size_t>(i) * d_out + j;
            __nv_bfloat16 a, b;
            split2_bf16(tw[tx][r], a, b);
            W0[o] = a;
            W1[o] = b;
            Qt[o] = tq[tx][r];
        }
    }
}

// One-hot columns of channels [j0, j0 + nch): Pm[i][jj * m + q] = (Qt[i][j0 + jj] == q), bf16, row stride ld.
// One thread writes the m columns of one (row, channel); with m = 16 and ld a multiple of 8 that is two
// 16-byte stores, and consecutive threads write consecutive 32-byte pieces.
__global__ void __launch_bounds__(256)
cb_onehot_kernel(const uint8_t *__restrict__ Qt, int d_in, int d_out, int j0, int nch, int m,
                 __nv_bfloat16 *__restrict__ Pm, long long ld)
{
    const long long total = static_cast<long long>(d_in) * nch;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    const bool wide = m == 16 && (ld & 7) == 0;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const int i = static_cast<int>(idx / nch);
        const int jj = static_cast<int>(idx - static_cast<long long>(i) * nch);
        int code = Qt[static_cast<size_t>(i) * d_out + j0 + jj];
        code = code < m ? code : m - 1;
        __nv_bfloat16 *dst = Pm + static_cast<size_t>(i) * ld + static_cast<size_t>(jj) * m;
        if (wide) {
            uint32_t w[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)            // bf16 1.0 = 0x3F80 in the low or the high half of word t
                w[t] = (code >> 1) == t ? ((code & 1) ? 0x3F800000u : 0x00003F80u) : 0u;
            uint4 *d4 = reinterpret_cast<uint4 *>(dst);
            d4[0] = make_uint4(w[0], w[1], w[2], w[3]);
            d4[1] = make_uint4(w[4], w[5], w[6], w[7]);
        } else {
            for (int q = 0; q < m; ++q) dst[q] = __float2bfloat16_rn(q == code ? 1.0f : 0.0f);
        }
    }
}

// Fold over the rows of each level.  One CTA = CB_FOLD_CH channels of the slab x 16 threads x one of gridDim.y
// row ranges; thread (ch, q') owns column q' of G^(ch) in shared memory, so no two threads of a CTA ever add
// to the same word; thread q' = 0 also owns r.  Within a row range (a few hundred rows, a few dozen per level)
// the sums are fp32 and use shared-memory reductions whose results are not read back, so that nothing in the
// row loop waits for an addition; the row ranges are combined in fp64 with atomic adds (the order of at most
// gridDim.y fp64 partial sums is the only thing that can vary from run to run).
constexpr int CB_FOLD_CH = 16;
__global__ void __launch_bounds__(CB_FOLD_CH * 16)
cb_fold_kernel(const float *__restrict__ HP, long long ld_hp, const float *__restrict__ HW, const uint8_t *__restrict__ Qt,
               int d_in, int d_out, int j0, int nch, int m, double *__restrict__ G, double *__restrict__ R)
{
    __shared__ float Gs[CB_FOLD_CH][CB_MAX_LEVELS][CB_MAX_LEVELS + 1];
    __shared__ float Rs[CB_FOLD_CH][CB_MAX_LEVELS];
    const int ch = threadIdx.x >> 4, qp = threadIdx.x & 15;
    const int jj = blockIdx.x * CB_FOLD_CH + ch;
    for (int q = 0; q < CB_MAX_LEVELS; ++q) Gs[ch][q][qp] = 0.0f;
    Rs[ch][qp] = 0.0f;
    __syncthreads();
    if (jj < nch && qp < m) {
        const int j = j0 + jj;
        const float *hp = HP + static_cast<size_t>(jj) * m + qp;
        constexpr int BATCH = 8;                         // independent loads in flight per thread
        const int rows_per = (d_in + static_cast<int>(gridDim.y) - 1) / static_cast<int>(gridDim.y);
        const int i_begin = static_cast<int>(blockIdx.y) * rows_per;
        const int i_end = i_begin + rows_per < d_in ? i_begin + rows_per : d_in;
        for (int i0 = i_begin; i0 < i_end; i0 += BATCH) {
            int q[BATCH];
            float v[BATCH], w[BATCH];
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                const int i = i0 + t;
                const bool ok = i < i_end;
                q[t] = ok ? Qt[static_cast<size_t>(i) * d_out + j] : 0;
                v[t] = ok ? hp[static_cast<size_t>(i) * ld_hp] : 0.0f;
                w[t] = (ok && qp == 0) ? HW[static_cast<size_t>(i) * d_out + j] : 0.0f;
            }
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                const int qq = q[t] < m ? q[t] : m - 1;  // codes are expected to be < m
                atomicAdd(&Gs[ch][qq][qp], v[t]);
                if (qp == 0) atomicAdd(&Rs[ch][qq], w[t]);
            }
        }
    }
    __syncthreads();
    if (jj < nch && qp < m) {                        // G and R were zeroed by the host; row ranges add up
        const int j = j0 + jj;
        for (int q = 0; q < m; ++q)
            atomicAdd(&G[(static_cast<size_t>(j) * CB_MAX_LEVELS + q) * CB_MAX_LEVELS + qp], static_cast<double>(Gs[ch][q][qp]));
        atomicAdd(&R[static_cast<size_t>(j) * CB_MAX_LEVELS + qp], static_cast<double>(Rs[ch][qp]));
    }
}

// The same fold for m a multiple of 4 (the usual 2-, 3- and 4-bit codebooks have m = 4, 8, 16): a thread takes
// four neighbouring columns q' of one channel with one 16-byte load per row, so the row loop spends its
// instructions on the data rather than on addresses (the one-column form above is issue-bound).  One CTA =
// CB_FOLD4_CH channels x 4 threads.
constexpr int CB_FOLD4_CH = 32;
__global__ void __launch_bounds__(CB_FOLD4_CH * 4)
cb_fold4_kernel(const float *__restrict__ HP, long long ld_hp, const float *__restrict__ HW, const uint8_t *__restrict__ Qt,
                int d_in, int d_out, int j0, int nch, int m, double *__restrict__ G, double *__restrict__ R)
{
    __shared__ float Gs[CB_FOLD4_CH][CB_MAX_LEVELS][CB_MAX_LEVELS + 1];
    __shared__ float Rs[CB_FOLD4_CH][CB_MAX_LEVELS];
    const int ch = threadIdx.x >> 2, q4 = (threadIdx.x & 3) * 4;
    const int jj = blockIdx.x * CB_FOLD4_CH + ch;
    for (int q = 0; q < CB_MAX_LEVELS; ++q)
        for (int e = 0; e < 4; ++e) Gs[ch][q][q4 + e] = 0.0f;
    for (int e = 0; e < 4; ++e) Rs[ch][q4 + e] = 0.0f;
    __syncthreads();
    const bool active = jj < nch && q4 < m;
    if (active) {
        const int j = j0 + jj;
        constexpr int BATCH = 8;                         // independent loads in flight per thread
        const int rows_per = (d_in + static_cast<int>(gridDim.y) - 1) / static_cast<int>(gridDim.y);
        const int i_begin = static_cast<int>(blockIdx.y) * rows_per;
        const int i_end = i_begin + rows_per < d_in ? i_begin + rows_per : d_in;
        const float *hp = HP + static_cast<size_t>(i_begin) * ld_hp + static_cast<size_t>(jj) * m + q4;
        const uint8_t *qt = Qt + static_cast<size_t>(i_begin) * d_out + j;
        const float *hw = HW + static_cast<size_t>(i_begin) * d_out + j;
        float *gbase = &Gs[ch][0][q4];
        int i0 = i_begin;
        for (; i0 + BATCH <= i_end; i0 += BATCH) {       // whole batches: no row predicates
            int q[BATCH];
            float4 v[BATCH];
            float w[BATCH];
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                q[t] = qt[static_cast<size_t>(t) * d_out];
                v[t] = *reinterpret_cast<const float4 *>(hp + static_cast<size_t>(t) * ld_hp);
                w[t] = q4 == 0 ? hw[static_cast<size_t>(t) * d_out] : 0.0f;
            }
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                const int qq = q[t] < m ? q[t] : m - 1;  // codes are expected to be < m
                float *gp = gbase + qq * (CB_MAX_LEVELS + 1);
                atomicAdd(gp + 0, v[t].x);
                atomicAdd(gp + 1, v[t].y);
                atomicAdd(gp + 2, v[t].z);
                atomicAdd(gp + 3, v[t].w);
                if (q4 == 0) atomicAdd(&Rs[ch][qq], w[t]);
            }
            hp += static_cast<size_t>(BATCH) * ld_hp;
            qt += static_cast<size_t>(BATCH) * d_out;
            hw += static_cast<size_t>(BATCH) * d_out;
        }
        for (; i0 < i_end; ++i0) {                       // ragged end of the row range
            const int qr = *qt;
            const int qq = qr < m ? qr : m - 1;
            const float4 v = *reinterpret_cast<const float4 *>(hp);
            float *gp = gbase + qq * (CB_MAX_LEVELS + 1);
            atomicAdd(gp + 0, v.x);
            atomicAdd(gp + 1, v.y);
            atomicAdd(gp + 2, v.z);
            atomicAdd(gp + 3, v.w);
            if (q4 == 0) atomicAdd(&Rs[ch][qq], *hw);
            hp += ld_hp;
            qt += d_out;
            hw += d_out;
        }
    }
    __syncthreads();
    if (active) {                                    // G and R were zeroed by the host; row ranges add up
        const int j = j0 + jj;
        for (int q = 0; q < m; ++q)
            for (int e = 0; e < 4; ++e)
                atomicAdd(&G[(static_cast<size_t>(j) * CB_MAX_LEVELS + q) * CB_MAX_LEVELS + q4 + e],
                          static_cast<double>(Gs[ch][q][q4 + e]));
        for (int e = 0; e < 4; ++e)
            atomicAdd(&R[static_cast<size_t>(j) * CB_MAX_LEVELS + q4 + e], static_cast<double>(Rs[ch][q4 + e]));
    }
}

// (G + lambda I) c = r by Cholesky, one thread per channel, fp64; G is symmetrised first (its two triangles
// come from different sums).  A pivot that is not positive (possible only through rounding) is replaced by
// lambda-sized regularisation so that the solve always completes.
__global__ void __launch_bounds__(128)
cb_solve_kernel(const double *__restrict__ G, const double *__restrict__ R, int d_out, int m, double lambda,
                float *__restrict__ codebook)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_out) return;
    double A[CB_MAX_LEVELS][CB_MAX_LEVELS];
    double b[CB_MAX_LEVELS];
    const double *g = G + static_cast<size_t>(j) * CB_MAX_LEVELS * CB_MAX_LEVELS;
    for (int q = 0; q < m; ++q) {
        for (int p = 0; p <= q; ++p) A[q][p] = 0.5 * (g[q * CB_MAX_LEVELS + p] + g[p * CB_MAX_LEVELS + q]);
        A[q][q] += lambda;
        b[q] = R[static_cast<size_t>(j) * CB_MAX_LEVELS + q];
    }
    for (int q = 0; q < m; ++q) {                 // A = L L^T, L stored in the lower triangle
        for (int p = 0; p < q; ++p) {
            double v = A[q][p];
            for (int t = 0; t < p; ++t) v -= A[q][t] * A[p][t];
            A[q][p] = v / A[p][p];
        }
        double d = A[q][q];
        for (int t = 0; t < q; ++t) d -= A[q][t] * A[q][t];
        if (!(d > 0.0)) d = lambda > 0.0 ? lambda : 1e-300;
        A[q][q] = sqrt(d);
    }
    for (int q = 0; q < m; ++q) {                 // L y = b
        double v = b[q];
        for (int t = 0; t < q; ++t) v -= A[q][t] * b[t];
        b[q] = v / A[q][q];
    }
    for (int q = m - 1; q >= 0; --q) {            // L^T c = y
        double v = b[q];
        for (int t = q + 1; t < m; ++t) v -= A[t][q] * b[t];
        b[q] = v / A[q][q];
    }
    for (int q = 0; q < m; ++q) codebook[static_cast<size_t>(j) * m + q] = static_cast<float>(b[q]);
}

// What[j][i] = codebook[j][Q[j][i]]
__global__ void __launch_bounds__(256)
cb_apply_kernel(const float *__restrict__ codebook, const uint8_t *__restrict__ Q, long long count, int d_in, int m,
                float *__restrict__ What)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < count; idx += stride) {
        const long long j = idx / d_in;
        const int q = Q[idx];
        What[idx] = codebook[j * m + (q < m ? q : m - 1)];
    }
}

}  // namespace gq
