// Token-sharded accumulation (each GPU builds H from its own tokens; Section 3.2: H is a sum over data
// points, so partial sums over disjoint token sets add up): the exchange that turns R partial matrices, one
// per GPU, into the same full sum on every GPU, written as two kernels over peer memory with a host-side
// barrier between them - no kernel ever waits for another GPU.
//
// The upper triangle of every H_k is cut into 128 x 128 blocks, numbered block column by block column and
// group after group; rank r owns the contiguous range [r B / R, (r + 1) B / R) of the B blocks.
//   reduce: rank r reads its blocks from all R matrices (plain loads over NVLink from the peers), adds them in
//           rank order 0, 1, ... R - 1 (so every GPU would form bit-identical sums) and writes them to its own H;
//   gather: rank r copies every other rank's blocks from that rank's H.
// Entries below the diagonal inside diagonal blocks travel with their block; gq_hessian_finalize overwrites
// them afterwards.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gq {

constexpr int EX_BLOCK = 128;            // edge of an exchanged block
constexpr int EX_MAX_RANKS = 16;

struct ExchangeParams {
    float *H[EX_MAX_RANKS];              // H of every rank as seen from this GPU: [g][d][d]
    int ranks;
    int rank;                            // this GPU
    int d;
    int g;
    int nb;                              // ceil(d / 128)
    long long blocks;                    // g * nb (nb + 1) / 2
};

__host__ __device__ inline long long exchange_share_begin(long long blocks, int ranks, int r)
{
    return blocks * r / ranks;
}

// block number (within one group, column-major triangle) -> (row block bi <= column block bj)
__device__ __forceinline__ void exchange_block_coords(int t, int &bi, int &bj)
{
    int jj = static_cast<int>((sqrtf(8.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
    while (jj * (jj + 1) / 2 > t) --jj;
    while ((jj + 1) * (jj + 2) / 2 <= t) ++jj;
    bj = jj;
    bi = t - jj * (jj + 1) / 2;
}

// One CTA per block of the range [first, first + gridDim.x); 256 threads, each 16 float4 of the block
// (row r = 8 i + threadIdx.x / 32, 512-byte row segments per warp).  REDUCE: sum over all ranks into
// H[rank]; otherwise copy from H[owner of the block] into H[rank] (blocks owned by `rank` are skipped).
template <bool REDUCE>
__global__ void __launch_bounds__(256)
exchange_kernel(const ExchangeParams p, long long first)
{
    const long long blk = first + blockIdx.x;
    if (blk >= p.blocks) return;
    const int per_group = p.nb * (p.nb + 1) / 2;
    const int k = static_cast<int>(blk / per_group);
    int bi, bj;
    exchange_block_coords(static_cast<int>(blk - static_cast<long long>(k) * per_group), bi, bj);
    int owner = 0;
    if (!REDUCE) {
        // owner = the rank whose range holds blk
        owner = static_cast<int>((blk * p.ranks + p.ranks - 1) / p.blocks);
        if (owner >= p.ranks) owner = p.ranks - 1;
        while (owner > 0 && exchange_share_begin(p.blocks, p.ranks, owner) > blk) --owner;
        while (owner + 1 < p.ranks && exchange_share_begin(p.blocks, p.ranks, owner + 1) <= blk) ++owner;
        if (owner == p.rank) return;
    }
    const int c = bj * EX_BLOCK + (threadIdx.x & 31) * 4;
    if (c >= p.d) return;                                   // d % 8 == 0: a float4 is inside or outside as a whole
    const size_t base = static_cast<size_t>(k) * p.d * p.d;
    for (int rr = threadIdx.x >> 5; rr < EX_BLOCK; rr += 8) {
        const int r = bi * EX_BLOCK + rr;
        if (r >= p.d) break;
        const size_t o = base + static_cast<size_t>(r) * p.d + c;
        float4 acc;
        if (REDUCE) {
            acc = *reinterpret_cast<const float4 *>(p.H[0] + o);
            for (int q = 1; q < p.ranks; ++q) {
                const float4 v = *reinterpret_cast<const float4 *>(p.H[q] + o);
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
        } else {
            acc = *reinterpret_cast<const float4 *>(p.H[owner] + o);
        }
        *reinterpret_cast<float4 *>(p.H[p.rank] + o) = acc;
    }
}

}  // namespace gq
