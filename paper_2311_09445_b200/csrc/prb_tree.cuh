// Sum-tree maintenance shared by the update and insert kernels: the priority transform, the
// batched leaf update with last-writer-wins deduplication, and the re-sum of a contiguous range
// of inserted leaves.  All of it is written for a "team": a whole number of warps of one CTA
// that synchronise on their own barrier, so that the same code runs as a full CTA (the update
// kernel) or as a few warps beside the copy warps of an insert kernel.
#pragma once
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

#ifdef __CUDACC__

// Inputs of entry `rank` that a kernel may have fetched before the team's work starts (so that the
// fetch overlaps an earlier wait); valid only where the matching flag is set.
struct PrbPreloaded {
    bool has_update, has_prio;
    int32_t idx;
    float val, prio;
};

struct PrbTeam {
    uint32_t rank, size;     // this thread's rank in the team, number of threads (multiple of 32)
    bool whole_cta;          // the team is the whole CTA: plain __syncthreads; otherwise named barrier 1
    // Several CTAs of one thread-block cluster may share the tree work: each holds the full sorted
    // key list, CTA `part` of `parts` takes the slots whose warp-sized group number is congruent to
    // it, and the phases are separated by the cluster's hardware barrier.  parts == 1: one CTA.
    uint32_t part = 0, parts = 1;

    __device__ __forceinline__ void sync() const
    {
        if (whole_cta) __syncthreads();
        else asm volatile("bar.sync 1, %0;" ::"r"(size) : "memory");
    }
    __device__ __forceinline__ bool takes(uint32_t slot) const { return parts == 1 || ((slot >> 5) % parts) == part; }
    // Between the phases of the tree work (leaves, then level by level): what the team -- or every
    // CTA of the cluster -- wrote to global memory before is visible to all of it after.
    __device__ __forceinline__ void phase_sync() const
    {
        if (parts == 1) { sync(); return; }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    // barrier + OR-reduction of a predicate over the team
    __device__ __forceinline__ bool sync_or(bool pred) const
    {
        if (whole_cta) return __syncthreads_or(pred) != 0;
        uint32_t out;
        asm volatile("{ .reg .pred p, q; setp.ne.u32 q, %1, 0; bar.red.or.pred p, 1, %2, q; selp.u32 %0, 1, 0, p; }"
                     : "=r"(out) : "r"((uint32_t)pred), "r"(size) : "memory");
        return out != 0;
    }
};

// p = (|delta| + eps)^alpha from IEEE basic operations only (binary64, every operation rounded
// once, no fused multiply-add), so that a CPU restatement reproduces it bit for bit:
//   y = |delta| + eps (binary32);  y = m 2^E, m in (sqrt(1/2), sqrt(2)];  t = (m-1)/(m+1);
//   ln m = 2t (1 + t^2/3 + ... + t^24/25);  z = alpha (E ln2 + ln m);  k = rint(z / ln2);
//   r = (z - k ln2_hi) - k ln2_lo;  exp r = sum_{n<=14} r^n/n!;  p = (binary32)(exp r * 2^k).
// Returns false for an invalid entry (non-finite delta, or a result outside binary32).
__device__ __forceinline__ bool prb_priority_pow(float delta, float eps, float alpha, float& p)
{
    if (!(fabsf(delta) <= 3.402823466e+38f)) return false;
    const float y32 = __fadd_rn(fabsf(delta), eps);
    if (!(y32 <= 3.402823466e+38f)) return false;
    if (alpha == 0.0f) { p = 1.0f; return true; }
    if (y32 == 0.0f) { p = 0.0f; return true; }

    const long long bits = __double_as_longlong((double)y32);
    int E = (int)((bits >> 52) & 0x7FF) - 1023;
    double m = __longlong_as_double((bits & 0x000FFFFFFFFFFFFFll) | 0x3FF0000000000000ll);
    if (m > 1.4142135623730951) { m = __dmul_rn(m, 0.5); E += 1; }

    // series coefficients 1/(2n+1) and 1/n!: IEEE quotients of exact integers, folded at compile time
    constexpr double kOdd[13] = { 1.0 / 1.0, 1.0 / 3.0, 1.0 / 5.0, 1.0 / 7.0, 1.0 / 9.0, 1.0 / 11.0, 1.0 / 13.0,
                                  1.0 / 15.0, 1.0 / 17.0, 1.0 / 19.0, 1.0 / 21.0, 1.0 / 23.0, 1.0 / 25.0 };
    constexpr double kRfact[15] = { 1.0 / 1.0, 1.0 / 1.0, 1.0 / 2.0, 1.0 / 6.0, 1.0 / 24.0, 1.0 / 120.0, 1.0 / 720.0,
                                    1.0 / 5040.0, 1.0 / 40320.0, 1.0 / 362880.0, 1.0 / 3628800.0, 1.0 / 39916800.0,
                                    1.0 / 479001600.0, 1.0 / 6227020800.0, 1.0 / 87178291200.0 };
    const double t = __ddiv_rn(__dadd_rn(m, -1.0), __dadd_rn(m, 1.0));
    const double t2 = __dmul_rn(t, t);
    double S = kOdd[12];
#pragma unroll
    for (int n = 11; n >= 0; --n) S = __dadd_rn(__dmul_rn(S, t2), kOdd[n]);
    const double lnm = __dmul_rn(__dmul_rn(2.0, t), S);

    const double L = __dadd_rn(__dmul_rn((double)E, 0.6931471805599453), lnm);
    const double z = __dmul_rn((double)alpha, L);
    const double q = __dmul_rn(z, 1.4426950408889634);
    if (q >= 1000.0) return false;
    if (q <= -1000.0) { p = 0.0f; return true; }
    const double k = rint(q);
    double r = __dsub_rn(z, __dmul_rn(k, 0.693147180369123816490));
    r = __dsub_rn(r, __dmul_rn(k, 1.90821492927058770002e-10));

    double P = kRfact[14];
#pragma unroll
    for (int n = 13; n >= 0; --n) P = __dadd_rn(__dmul_rn(P, r), kRfact[n]);
    const double scale = __longlong_as_double(((long long)k + 1023ll) << 52);
    const float out = __double2float_rn(__dmul_rn(P, scale));
    if (!(out <= 3.402823466e+38f)) return false;
    p = out;
    return true;
}

// A skipped entry keeps its batch position under an index of all ones: such keys sort last and, like
// the valid ones, are all different.
constexpr unsigned long long kPrbInvalidKey = ~0ull;
__device__ __forceinline__ bool prb_key_invalid(unsigned long long key) { return (uint32_t)(key >> 32) == 0xFFFFFFFFu; }

// Shared memory an update of a batch padded to n2 entries needs: keys, then values.
__host__ __device__ inline size_t prb_update_smem_bytes(uint32_t n2)
{
    return (size_t)n2 * (sizeof(unsigned long long) + sizeof(float));
}

// Batched priority update by one team (PEARL Section V-A, "priority update", read as set +
// re-sum).  Entries are keyed (index << 32) | batch position and sorted; the last entry of every
// run of equal indices wins and writes its leaf; then, level by level from the deepest, the
// first entry of every run of equal ancestors re-sums that ancestor from its children in
// left-to-right order.  Sorted order survives dropping low digits of the index, so no list is
// compacted and no lock is taken.  n2 = B rounded up to a power of two (>= 2); smem holds
// prb_update_smem_bytes(n2) bytes; fill = the fill count before this launch (indices must be below it).
// With stale > 0 (and n == 0) entries that name one of the `stale` ring slots before `cursor` are
// skipped: they were overwritten after they had been sampled.
// With n > 0 the tree part of an insertion of n transitions at `cursor` follows in the same
// passes: the inserted leaves are written after the update's (an updated leaf that is also
// inserted keeps the inserted priority), and every level is re-summed once for both, the
// insertion's parents being the contiguous range(s) above its slots.  A parent reached both ways
// is computed twice with the same result.
__device__ __forceinline__ void prb_update_team(const PrbView& v, const PrbTeam& team, uint32_t B, uint32_t n2,
                                                const int32_t* __restrict__ idx, const float* __restrict__ val, int raw,
                                                float alpha, float eps, unsigned long long fill, unsigned char* smem,
                                                uint32_t n = 0, const float* __restrict__ prio = nullptr,
                                                uint64_t cursor = 0, PrbPreloaded pre = PrbPreloaded{false, false, 0, 0.0f, 0.0f},
                                                uint32_t stale = 0)
{
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);
    float* vals = reinterpret_cast<float*>(smem + (size_t)n2 * sizeof(unsigned long long));
    const uint32_t rank = team.rank, nt = team.size;

    unsigned flags = 0;
    float wmax = 0.0f;                 // largest priority this thread accepted
    bool unsorted = false;
    unsigned long long my_key = kPrbInvalidKey;      // the key of entry `rank` (one-key-per-thread case)
    for (uint32_t b = rank; b < n2; b += nt) {
        unsigned long long key = 0xFFFFFFFF00000000ull | b;
        if (b < B) {
            const bool mine = pre.has_update && b == rank;
            const int32_t i = mine ? pre.idx : idx[b];
            const float x = mine ? pre.val : val[b];
            float p = 0.0f;
            bool ok_p;
            if (raw) { p = x; ok_p = prb_valid_priority(p); }
            else ok_p = prb_priority_pow(x, eps, alpha, p);
            // stale: one of the `stale` slots written most recently, i.e. overwritten since it was sampled
            const uint64_t back = (i >= 0 && stale) ? (cursor + v.capacity - 1 - (uint64_t)i) % v.capacity : ~0ull;
            if (i < 0 || (unsigned long long)i >= fill) flags |= PEARL_ST_BAD_INDEX;
            else if (back < stale) flags |= PEARL_ST_STALE;
            else if (!ok_p) flags |= PEARL_ST_BAD_PRIORITY;
            else { key = ((unsigned long long)(uint32_t)i << 32) | b; wmax = fmaxf(wmax, p); }
            vals[b] = p;
        }
        keys[b] = key;
        my_key = key;
    }
    if (flags && team.part == 0) atomicOr(&v.state->status, flags);
    prb_note_priorities(v.state, wmax, team.part == 0);
    team.sync();

    // Indices that come straight from a stratified sample are already in order; sort only if needed.
    for (uint32_t b = rank; b + 1 < n2; b += nt) unsorted |= (keys[b] > keys[b + 1]);
    unsorted = team.sync_or(unsorted);

    if (unsorted && n2 <= nt && n2 <= 512) {
        // a small batch is sorted by counting: the keys are all different, so the number of keys
        // below a key is its place (every thread reads the same key at a time: one broadcast per step,
        // no barrier between steps, against the dozens of dependent stages of a sorting network)
        const unsigned long long key = my_key;
        uint32_t place = 0;
        if (rank < n2) {
#pragma unroll 8
            for (uint32_t j = 0; j < n2; ++j) place += (keys[j] < key) ? 1u : 0u;
        }
        team.sync();
        if (rank < n2) keys[place] = key;
        team.sync();
    } else if (unsorted && n2 <= nt) {
        // bitonic sort, one key per thread: exchanges across fewer than 32 positions are warp shuffles
        unsigned long long key = (rank < n2) ? my_key : kPrbInvalidKey;
        for (uint32_t k = 2; k <= n2; k <<= 1) {
            for (uint32_t j = k >> 1; j > 0; j >>= 1) {
                unsigned long long other;
                if (j >= 32) {
                    if (rank < n2) keys[rank] = key;
                    team.sync();
                    other = (rank < n2) ? keys[rank ^ j] : kPrbInvalidKey;
                    team.sync();
                } else {
                    other = __shfl_xor_sync(0xFFFFFFFFu, key, j);
                }
                const bool keep_min = ((rank & k) == 0) == ((rank & j) == 0);
                key = keep_min ? (key < other ? key : other) : (key > other ? key : other);
            }
        }
        if (rank < n2) keys[rank] = key;
        team.sync();
    } else if (unsorted) {
        // bitonic sort in shared memory, several keys per thread
        for (uint32_t k = 2; k <= n2; k <<= 1) {
            for (uint32_t j = k >> 1; j > 0; j >>= 1) {
                for (uint32_t t = rank; t < (n2 >> 1); t += nt) {
                    const uint32_t lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));   // element with bit j clear
                    const uint32_t hi = lo | j;
                    const unsigned long long a = keys[lo], c = keys[hi];
                    const bool up = (lo & k) == 0;
                    if ((a > c) == up) { keys[lo] = c; keys[hi] = a; }
                }
                team.sync();
            }
        }
    }

    // winners write the leaves (unless the insertion overwrites the slot anyway), then the inserted leaves
    const uint64_t N = v.capacity;
    float* leaves = v.level[v.depth];
    for (uint32_t s = rank; s < n2; s += nt) {
        const unsigned long long key = keys[s];
        if (prb_key_invalid(key) || !team.takes(s)) continue;
        const uint32_t i = (uint32_t)(key >> 32);
        const bool last = (s + 1 == n2) || ((uint32_t)(keys[s + 1] >> 32) != i);
        const uint64_t ahead = i >= cursor ? i - cursor : i + N - cursor;     // distance from the cursor along the ring
        if (last && !(ahead < n)) leaves[i] = vals[(uint32_t)key];
    }
    bool bad = false;
    float imax = 0.0f;
    // without priorities the new transitions take the running maximum, this update's writes included
    const float dflt = (n && prio == nullptr) ? prb_default_priority(__ldcg(&v.state->max_prio_bits)) : 0.0f;
    for (uint32_t t = rank; t < n; t += nt) {
        if (!team.takes(t)) continue;
        uint64_t slot = cursor + t;
        if (slot >= N) slot -= N;
        float p = prio == nullptr ? dflt : ((pre.has_prio && t == rank) ? pre.prio : prio[t]);
        if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
        else imax = fmaxf(imax, p);
        leaves[slot] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    if (n) prb_note_priorities(v.state, imax, team.part == 0);      // (a first default insertion writes 1)
    team.phase_sync();

    // re-sum the ancestors, deepest level first; the insertion dirties parent range A = [a0, a1] >> sh
    // and, if the ring wrapped, B = [0, b1] >> sh
    const uint32_t K = v.fanout, lg = v.log2_fanout;
    const uint64_t a0 = cursor, a1 = (n ? min(cursor + n, N) : cursor + 1) - 1;
    const bool wrapped = cursor + n > N;
    const uint64_t b1 = wrapped ? cursor + n - N - 1 : 0;
    for (int l = (int)v.depth - 1; l >= 0; --l) {
        const uint32_t sh = lg * (v.depth - (uint32_t)l);
        const float* child = v.level[l + 1];
        float* par = v.level[l];
        for (uint32_t s = rank; s < n2; s += nt) {
            const unsigned long long key = keys[s];
            if (prb_key_invalid(key) || !team.takes(s)) continue;
            const uint32_t a = (uint32_t)(key >> 32) >> sh;
            const bool first = (s == 0) || (((uint32_t)(keys[s - 1] >> 32) >> sh) != a);
            if (first) par[a] = prb_sum_children_dyn(child + (uint64_t)a * K, K);
        }
        if (n) {
            const uint64_t pa0 = a0 >> sh, cntA = (a1 >> sh) - pa0 + 1;
            uint64_t cntB = 0;
            if (wrapped) cntB = (pa0 == 0) ? 0 : min(b1 >> sh, pa0 - 1) + 1;     // parents of B not already in A
            for (uint64_t i = rank; i < cntA + cntB; i += nt) {
                if (!team.takes((uint32_t)i)) continue;
                const uint64_t j = (i < cntA) ? pa0 + i : i - cntA;
                par[j] = prb_sum_children_dyn(child + j * K, K);
            }
        }
        team.phase_sync();
    }
}

// Tree part of an insertion by one team: write the n leaves of ring slots cursor .. cursor+n-1
// (mod capacity), then re-sum the dirty parents level by level.  A contiguous slot range dirties
// a contiguous parent range on every level (two ranges if the ring wrapped), so nothing is sorted.
__device__ __forceinline__ void prb_insert_tree_team(const PrbView& v, const PrbTeam& team, uint32_t n,
                                                     const float* __restrict__ prio, uint64_t cursor,
                                                     PrbPreloaded pre = PrbPreloaded{false, false, 0, 0.0f, 0.0f},
                                                     unsigned max_bits = 0)
{
    const uint64_t N = v.capacity;
    const uint32_t D = v.depth, K = v.fanout, lg = v.log2_fanout;
    float* leaves = v.level[D];
    bool bad = false;
    float imax = 0.0f;
    const float dflt = prb_default_priority(max_bits);     // used when no priorities are given
    for (uint32_t t = team.rank; t < n; t += team.size) {
        uint64_t slot = cursor + t;
        if (slot >= N) slot -= N;
        float p = prio == nullptr ? dflt : ((pre.has_prio && t == team.rank) ? pre.prio : prio[t]);
        if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
        else imax = fmaxf(imax, p);
        leaves[slot] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    prb_note_priorities(v.state, imax, true);                       // (a first default insertion writes 1)
    team.sync();
    // dirty leaf ranges: A = [a0, a1]; if the ring wrapped also B = [0, b1]
    const uint64_t a0 = cursor;
    const uint64_t a1 = min(cursor + n, N) - 1;
    const bool wrapped = cursor + n > N;
    const uint64_t b1 = wrapped ? cursor + n - N - 1 : 0;
    for (int l = (int)D - 1; l >= 0; --l) {
        const uint32_t sh = lg * (D - (uint32_t)l);
        const uint64_t pa0 = a0 >> sh, pa1 = a1 >> sh;
        const uint64_t cntA = pa1 - pa0 + 1;
        uint64_t cntB = 0;
        if (wrapped) {
            const uint64_t pb1 = b1 >> sh;
            cntB = (pa0 == 0) ? 0 : min(pb1, pa0 - 1) + 1;   // parents of B not already in A
        }
        const float* child = v.level[l + 1];
        float* par = v.level[l];
        for (uint64_t i = team.rank; i < cntA + cntB; i += team.size) {
            const uint64_t j = (i < cntA) ? pa0 + i : i - cntA;
            par[j] = prb_sum_children_dyn(child + j * K, K);
        }
        team.sync();
    }
}

#endif  // __CUDACC__
