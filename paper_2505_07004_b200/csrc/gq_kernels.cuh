// Bandwidth-bound kernels of libgq: saliency reduction, mirror, weight-error split,
// final fp64 reduction.  All use 128-bit accesses and grid-stride loops over a grid sized from the
// SM count.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gq {

__device__ __forceinline__ void bf16x8_to_float(const uint4 &v, float (&f)[8])
{
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 t = __bfloat1622float2(h[e]);
        f[2 * e] = t.x;
        f[2 * e + 1] = t.y;
    }
}

__device__ __forceinline__ uint4 float_to_bf16x8(const float (&f)[8])
{
    uint4 v;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
    for (int e = 0; e < 4; ++e) h[e] = __floats2bfloat162_rn(f[2 * e], f[2 * e + 1]);
    return v;
}

// A saliency value as the guided-Hessian kernel's scalers consume it: two bf16 terms packed in one word, low
// half hi = bf16(a), high half lo = bf16(a - hi); hi + lo carries a to 16 significant bits.
__device__ __forceinline__ uint32_t split_scale(float a)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(a);
    const __nv_bfloat16 lo = __float2bfloat16_rn(a - __bfloat162float(hi));
    return static_cast<uint32_t>(__bfloat16_as_ushort(hi)) | (static_cast<uint32_t>(__bfloat16_as_ushort(lo)) << 16);
}

// 16 bytes that are read once (evict-first).  Written as volatile asm so that the loads of a group are all
// issued, in order, before the first of them is consumed.
__device__ __forceinline__ uint4 ld_once_16(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float sum_sq_bf16x8(const uint4 &v, float acc)
{
    float f[8];
    bf16x8_to_float(v, f);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc = fmaf(f[e], f[e], acc);
    return acc;
}

// ------------------------------------------------------------------------------------------------
// Algorithm 1, saliency step.  One warp per (token, group) segment of m = d_out / g gradients:
//   s[k][i] = (grad_scale^2 / m) * sum_j grad[i][m k + j]^2.
// A lane reads 16 bytes (8 bf16) per load; the first four loads of a segment (all of it for m <= 1024) are
// issued back to back before anything is used, longer segments continue eight loads at a time.  The grid has one
// warp per segment (no grid-stride loop: thousands of short-lived blocks keep every SM at full occupancy and
// balance the tail at a granularity of 8 segments) and the index arithmetic is 32-bit, so the loads of a warp
// leave a few dozen cycles after it starts; measured on 67 MB launches this streams at 5.4 TB/s where a
// persistent grid with 64-bit segment arithmetic reached 3.6 TB/s.
// The lane-to-element assignment and the butterfly reduction are fixed, so the result does not depend on
// the grid.
// If `words` is not null the value is also stored in the packed form of split_scale, laid out as the
// guided-Hessian kernel reads it: [ceil(g / 2)][n] pairs of words, pair q of token i = groups 2q and 2q + 1
// (the second word of an odd last group is 0).
// A lane's share of sum_j grad[j]^2 over one segment of `vecs` 16-byte vectors (before the butterfly).
__device__ __forceinline__ float saliency_lane_sum(const uint4 *__restrict__ src, int vecs, int lane)
{
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    {
        uint4 x[4];
#pragma unroll
        for (int t = 0; t < 4; ++t)
            x[t] = (lane + 32 * t < vecs) ? ld_once_16(src + lane + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int t = 0; t < 4; ++t) acc[t] = sum_sq_bf16x8(x[t], acc[t]);
    }
    int v = lane + 128;
    for (; v + 224 < vecs; v += 256) {                   // eight full loads in flight
        uint4 x[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) x[t] = ld_once_16(src + v + 32 * t);
#pragma unroll
        for (int t = 0; t < 8; ++t) acc[t & 3] = sum_sq_bf16x8(x[t], acc[t & 3]);
    }
    for (; v < vecs; v += 128) {                         // rest: four loads, predicated off past the end
        uint4 x[4];
#pragma unroll
        for (int t = 0; t < 4; ++t)
            x[t] = (v + 32 * t < vecs) ? ld_once_16(src + v + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int t = 0; t < 4; ++t) acc[t] = sum_sq_bf16x8(x[t], acc[t]);
    }
    return (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

__device__ __forceinline__ float warp_sum_butterfly(float sum)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    return sum;
}

// Stores s[k][i] and, if `words` is not null, its packed two-term form (one lane calls this).
__device__ __forceinline__ void saliency_store(float val, unsigned i, int k, unsigned n, int g, float *__restrict__ s,
                                               long long ld_s, uint32_t *__restrict__ words)
{
    s[static_cast<long long>(k) * ld_s + i] = val;
    if (words) {
        uint32_t *w = words + (static_cast<long long>(k >> 1) * n + i) * 2;
        w[k & 1] = split_scale(val);
        if ((k & 1) == 0 && k + 1 == g) w[1] = 0u;
    }
}

__global__ void __launch_bounds__(256)
saliency_kernel(const __nv_bfloat16 *__restrict__ grad, unsigned n, int m, long long ld_grad, int g, float coef,
                float *__restrict__ s, long long ld_s, uint32_t *__restrict__ words)
{
    const int lane = threadIdx.x & 31;
    const unsigned seg = blockIdx.x * 8u + (threadIdx.x >> 5);
    if (seg >= n * static_cast<unsigned>(g)) return;
    const unsigned i = seg / static_cast<unsigned>(g);
    const int k = static_cast<int>(seg - i * static_cast<unsigned>(g));
    const uint4 *src = reinterpret_cast<const uint4 *>(grad + static_cast<long long>(i) * ld_grad + static_cast<long long>(k) * m);
    const float sum = warp_sum_butterfly(saliency_lane_sum(src, m >> 3, lane));
    if (lane == 0) saliency_store(sum * coef, i, k, n, g, s, ld_s, words);
}

// ------------------------------------------------------------------------------------------------
// The saliency step for a gradient as a backward pass hands it over (Section 3.2: only the averaged squared
// gradients of a layer are kept): dl/dZ as [batch][seq][d_out] with element strides (stride_b, stride_t, 1) in
// bf16, IEEE half or fp32; token i = b * seq + t lands in s[k][i].  Same warp-per-segment scheme and the same
// fp32 arithmetic as saliency_kernel (a 16-byte load holds 8 sixteen-bit or 4 fp32 values).
enum { SAL_BF16 = 0, SAL_FP16 = 1, SAL_FP32 = 2 };

template <int DTYPE>
__device__ __forceinline__ float sum_sq_vec16(const uint4 &v, float acc)
{
    if (DTYPE == SAL_BF16) return sum_sq_bf16x8(v, acc);
    if (DTYPE == SAL_FP16) {
        const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 t = __half22float2(h[e]);
            acc = fmaf(t.x, t.x, acc);
            acc = fmaf(t.y, t.y, acc);
        }
        return acc;
    }
    const float *f = reinterpret_cast<const float *>(&v);
#pragma unroll
    for (int e = 0; e < 4; ++e) acc = fmaf(f[e], f[e], acc);
    return acc;
}

template <int DTYPE>
__global__ void __launch_bounds__(256)
saliency_strided_kernel(const void *__restrict__ grad, unsigned n, unsigned seq, int m, long long stride_b, long long stride_t,
                        int g, float coef, float *__restrict__ s, long long ld_s)
{
    constexpr int PER_VEC = (DTYPE == SAL_FP32) ? 4 : 8;          // values per 16-byte load
    constexpr int ELEM = (DTYPE == SAL_FP32) ? 4 : 2;
    const int lane = threadIdx.x & 31;
    const unsigned seg = blockIdx.x * 8u + (threadIdx.x >> 5);
    if (seg >= n * static_cast<unsigned>(g)) return;
    const unsigned i = seg / static_cast<unsigned>(g);
    const int k = static_cast<int>(seg - i * static_cast<unsigned>(g));
    const unsigned b = i / seq, t = i - b * seq;
    const int vecs = m / PER_VEC;
    const long long first = static_cast<long long>(b) * stride_b + static_cast<long long>(t) * stride_t + static_cast<long long>(k) * m;
    const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const char *>(grad) + first * ELEM);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int v = lane; v < vecs; v += 128) {             // four loads in flight, predicated off past the end
        uint4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            x[u] = (v + 32 * u < vecs) ? ld_once_16(src + v + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[u] = sum_sq_vec16<DTYPE>(x[u], acc[u]);
    }
    float sum = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) s[static_cast<long long>(k) * ld_s + i] = sum * coef;
}

// ------------------------------------------------------------------------------------------------
// H[k][b][a] = H[k][a][b] for a < b (H_k is symmetric by definition, Section 3.2).
// blockIdx.x / .y = 32 x 32 block column / row, blockIdx.z = group; blocks below the diagonal exit.
__global__ void __launch_bounds__(256)
mirror_kernel(float *__restrict__ H, int d)
{
    const int bj = blockIdx.x, bi = blockIdx.y;
    if (bi > bj) return;
    __shared__ float tile[32][33];
    float *Hk = H + static_cast<size_t>(blockIdx.z) * d * d;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;    // 32 x 8 threads
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const int a = bi * 32 + r, b = bj * 32 + tx;
        tile[r][tx] = (a < d && b < d) ? Hk[static_cast<size_t>(a) * d + b] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int r = ty; r < 32; r += 8) {
        const int b = bj * 32 + r, a = bi * 32 + tx;          // write H[b][a] = tile[a - bi*32][b - bj*32]
        if (a < d && b < d && a < b) Hk[static_cast<size_t>(b) * d + a] = tile[tx][r];
    }
}

// ------------------------------------------------------------------------------------------------
// Weight error of Eq. 7, delta = W - W_hat in fp32, split into bf16 hi + bf16 lo
// (hi = bf16(delta), lo = bf16(delta - hi)); |delta - hi - lo| <= 2^-17 |delta|.
__global__ void __launch_bounds__(256)
split_delta_kernel(const float *__restrict__ W, const float *__restrict__ What, long long count8,
                   __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; idx < count8; idx += stride) {
        const float4 *w = reinterpret_cast<const float4 *>(W) + idx * 2;
        const float4 *q = reinterpret_cast<const float4 *>(What) + idx * 2;
        const float4 w0 = __ldcs(w), w1 = __ldcs(w + 1), q0 = __ldcs(q), q1 = __ldcs(q + 1);
        const float dlt[8] = {w0.x - q0.x, w0.y - q0.y, w0.z - q0.z, w0.w - q0.w,
                              w1.x - q1.x, w1.y - q1.y, w1.z - q1.z, w1.w - q1.w};
        float h[8], l[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            h[e] = __bfloat162float(__float2bfloat16_rn(dlt[e]));
            l[e] = dlt[e] - h[e];
        }
        reinterpret_cast<uint4 *>(hi)[idx] = float_to_bf16x8(h);
        reinterpret_cast<uint4 *>(lo)[idx] = float_to_bf16x8(l);
    }
}

// ------------------------------------------------------------------------------------------------
// loss[k] = sum over the group's partial sums (fixed order), loss[g] = sum_k loss[k].  One block.
// partials: [tiles][g][per_unit].
__global__ void __launch_bounds__(1024)
reduce_partials_kernel(const double *__restrict__ partials, int tiles, int g, int per_unit, double *__restrict__ loss)
{
    __shared__ double red[1024];
    double total = 0.0;
    for (int k = 0; k < g; ++k) {
        double acc = 0.0;
        for (int idx = threadIdx.x; idx < tiles * per_unit; idx += blockDim.x) {
            const int t = idx / per_unit, q = idx - t * per_unit;
            acc += partials[(static_cast<size_t>(t) * g + k) * per_unit + q];
        }
        red[threadIdx.x] = acc;
        __syncthreads();
        for (int off = blockDim.x >> 1; off > 0; off >>= 1) {
            if (static_cast<int>(threadIdx.x) < off) red[threadIdx.x] += red[threadIdx.x + off];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            loss[k] = red[0];
            total += red[0];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[g] = total;
}

}  // namespace gq
