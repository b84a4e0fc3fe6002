// Shared scaffolding of libgq's two tensor-core kernels (guided Hessian, objective): tile geometry, the
// distribution of work units over CTA pairs, and bounded mbarrier waits.
//
// Both kernels run as clusters of two CTAs (one CTA pair per two SMs).  A pair owns one 256 x 256 tile at a
// time; each CTA loads 128 of the tile's A rows and 128 of its B columns per 64-row k-step, the first CTA
// of the pair issues tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16) for both, and each CTA holds the
// fp32 accumulator rows of its own 128 rows in its tensor memory.
//
// Work distribution: units are dealt round-robin to the pairs for `full_waves` rounds, so that pairs that
// run at the same time work on neighbouring tiles and share operands in L2; what is left (fewer units than
// pairs) can be cut along the contraction index into equal pieces, one per pair.
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
constexpr int BOX_FEATURES = 64;                       // 128 bytes of bf16
constexpr int BOX_BYTES = TILE_K * 128;                // one TMA box: 64 rows x 128 B
constexpr uint32_t TMEM_COLS = 512;
constexpr int MIN_PIECE_KSTEPS = 8;                    // smallest k-range worth an epilogue of its own

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

// The same set of tiles in an order that keeps tiles which are worked on at the same time close together in
// BOTH directions: the upper triangle is cut into super-blocks of R x R tiles (column super-blocks outermost,
// row super-blocks inside, tiles of a super-block row by row), so that a round of P consecutive tiles touches
// about 2 sqrt(P) row/column blocks of X instead of P + 1.  Every (i <= j) appears exactly once for
// t in [0, NJ (NJ + 1) / 2).
__host__ __device__ inline void tile_of_slot_blocked(int t, int nj, int R, int &i, int &j)
{
    if (R <= 1) {
        // plain column-major triangle
        int jj = static_cast<int>((sqrtf(8.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
        while (jj * (jj + 1) / 2 > t) --jj;
        while ((jj + 1) * (jj + 2) / 2 <= t) ++jj;
        j = jj;
        i = t - jj * (jj + 1) / 2;
        return;
    }
    const int tri = R * (R + 1) / 2;
    // tiles before super-column J (all of them complete): R^2 J (J - 1) / 2 + J tri
    int J = static_cast<int>(sqrtf(2.0f * static_cast<float>(t) / static_cast<float>(R * R)));
    auto before = [&](int JJ) { return R * R * (JJ * (JJ - 1) / 2) + JJ * tri; };
    while (J > 0 && before(J) > t) --J;
    while ((J + 1) * R < nj && before(J + 1) <= t) ++J;
    int rem = t - before(J);
    const int rj = (nj - J * R < R) ? (nj - J * R) : R;       // columns in this super-column
    const int off_diag = J * R * rj;                          // tiles of the super-blocks above the diagonal one
    if (rem < off_diag) {
        const int I = rem / (R * rj);
        rem -= I * R * rj;
        i = I * R + rem / rj;
        j = J * R + rem % rj;
    } else {
        rem -= off_diag;                                      // triangle of rj x rj tiles, column-major
        int lj = static_cast<int>((sqrtf(8.0f * static_cast<float>(rem) + 1.0f) - 1.0f) * 0.5f);
        while (lj * (lj + 1) / 2 > rem) --lj;
        while ((lj + 1) * (lj + 2) / 2 <= rem) ++lj;
        i = J * R + rem - lj * (lj + 1) / 2;
        j = J * R + lj;
    }
}

// Slot t of the enumeration of (row block i, column-block pair q) with i <= 2q + 1, pairs outermost.
__device__ __forceinline__ void colpair_of_slot(int t, int &i, int &q)
{
    int qq = static_cast<int>((sqrtf(4.0f * static_cast<float>(t) + 1.0f) - 1.0f) * 0.5f);
    while (qq * qq + qq > t) --qq;
    while ((qq + 1) * (qq + 1) + (qq + 1) <= t) ++qq;
    q = qq;
    i = t - qq * qq - qq;
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
__device__ __forceinline__ bool wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site, uint32_t unit)
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
__device__ __forceinline__ bool bounded_wait_hot(uint32_t bar, uint32_t parity, const WaitCtx &w, uint32_t site,
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

// Self-test of the bounded waits: one thread waits, with the kernels' own wait routine, on a barrier that
// nothing will ever signal.  The wait gives up after `budget_ns`, records STATUS_TIMEOUT (site 99) in the
// status word and the kernel returns normally - the context stays usable.
__global__ void wait_selftest_kernel(uint32_t *status, unsigned long long budget_ns)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ volatile uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0u;
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const WaitCtx wc{&abort_flag, status, budget_ns};
        (void)bounded_wait(smem_u32(&bar), 0u, wc, 99u, 0u);
    }
}

__device__ __forceinline__ void spin_ns(unsigned long long ns)
{
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < ns) {}
}

// Walks the k-steps of a pair's work items in order, across item boundaries.
struct KstepCursor {
    const Schedule &sched;
    int pair;
    int it;
    int ks;
    bool valid;
    WorkItem w;
    __device__ KstepCursor(const Schedule &sc, int pr) : sched(sc), pair(pr), it(0), ks(0), valid(false)
    {
        valid = work_item(sched, pair, 0, w);
        ks = w.ks0;
    }
    __device__ void advance(int n)
    {
        while (n > 0 && valid) {
            const int left = w.ks1 - ks;
            if (n < left) {
                ks += n;
                n = 0;
            } else {
                n -= left;
                ++it;
                valid = work_item(sched, pair, it, w);
                ks = w.ks0;
            }
        }
    }
};

}  // namespace gq
