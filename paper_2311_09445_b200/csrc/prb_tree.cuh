// Sum-tree maintenance shared by the update and insert kernels: the priority transform, the
// batched leaf update with last-writer-wins deduplication, the leaves of an insertion, and the
// level-by-level re-sum of every dirty ancestor.  All of it is written for a "team": a whole number of warps of one CTA
// that synchronise on their own barrier, so that the same code runs as a full CTA (the update
// kernel) or as a few warps beside the copy warps of an insert kernel.
#pragma once
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

#ifdef __CUDACC__

struct PrbTeam {
    uint32_t rank, size;     // this thread's rank in the team, number of threads (multiple of 32)
    bool whole_cta;          // the team is the whole CTA: plain __syncthreads; otherwise named barrier 1

    __device__ __forceinline__ void sync() const
    {
        if (whole_cta) __syncthreads();
        else asm volatile("bar.sync 1, %0;" ::"r"(size) : "memory");
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

constexpr unsigned long long kPrbInvalidKey = ~0ull;
constexpr uint32_t kPrbNoParent = 0xFFFFFFFFu;

constexpr int kPrbFwdMaxPasses = 8;                 // entries per thread the compaction handles

struct PrbFwdLayout {
    uint32_t gs;                                    // floats between the groups of two parents (16-byte multiple)
    uint32_t off_scan, off_wnode, off_wval;         // byte offsets in shared memory (after keys and vals)
    uint32_t cmax[PRB_MAX_LEVELS];                  // most entries the list of a level can have
    uint32_t off_node[PRB_MAX_LEVELS], off_val[PRB_MAX_LEVELS], off_first[PRB_MAX_LEVELS], off_group[PRB_MAX_LEVELS];
    uint32_t total;
};

// What the tree team does in one launch: an optional priority update (B > 0), then the tree part of
// an optional insertion (n > 0).
struct PrbTreeWork {
    uint32_t B, n2;                 // update batch, and B rounded up to a power of two (>= 2)
    const int32_t* idx;
    const float* val;               // TD errors, or priorities if raw
    int raw;
    float alpha, eps;
    uint32_t n;                     // inserted transitions
    const float* prio;
    uint32_t forward;               // 1: the whole job fits the shared-memory forwarding path ...
    PrbFwdLayout fwd;               // ... laid out like this
};

// Shared memory the team needs: the update's keys and values, then per warp a 32 x (K+1) staging
// area for the cooperative child loads (fanout >= 8 only).
__host__ __device__ inline size_t prb_tree_smem_bytes(uint32_t n2_or_0, uint32_t fanout, uint32_t team_threads)
{
    size_t b = (size_t)n2_or_0 * (sizeof(unsigned long long) + sizeof(float));
    b = (b + 15) / 16 * 16;
    if (fanout >= 8) b += (size_t)(team_threads / 32) * 32 * (fanout + 1) * sizeof(float);
    return b;
}

// Re-sums the parents named by slots [0, n_slots): slot_parent(slot) is a node of the parent level
// or kPrbNoParent.  Each parent becomes the left-to-right binary32 sum of its K children.
// Fanout >= 8: a warp takes 32 slots at a time, loads their child groups with coalesced 16-byte
// loads (a group is K*4 contiguous bytes) into a padded staging area, and then every lane sums
// its own group from shared memory; all the global loads of a pass are in flight together.
template <int K, typename SlotParent>
__device__ __forceinline__ void prb_resum_slots(const PrbTeam& team, const float* child, float* par, uint32_t n_slots,
                                                SlotParent slot_parent, float* scratch)
{
    const uint32_t lane = team.rank & 31u, warp = team.rank >> 5, n_warps = team.size >> 5;
    for (uint32_t base = warp * 32u; base < n_slots; base += n_warps * 32u) {
        const uint32_t slot = base + lane;
        const uint32_t a = slot < n_slots ? slot_parent(slot) : kPrbNoParent;
        if constexpr (K <= 4) {
            if (a != kPrbNoParent) par[a] = prb_sum_children<K>(child + (uint64_t)a * K);
        } else {
            if (!__any_sync(0xFFFFFFFFu, a != kPrbNoParent)) continue;
            constexpr int G = K >= 8 ? K / 4 : 1;         // 16-byte units per child group
            float* mine = scratch + (size_t)warp * 32 * (K + 1);
            float4 c[G];
            uint32_t loaded = 0;                          // bit t: unit t of this lane belongs to a live slot
#pragma unroll
            for (int t = 0; t < G; ++t) {
                const uint32_t u = (uint32_t)t * 32u + lane, job = u / G, part = u % G;
                const uint32_t aj = __shfl_sync(0xFFFFFFFFu, a, job);
                if (aj != kPrbNoParent) {
                    c[t] = __ldcg(reinterpret_cast<const float4*>(child + (uint64_t)aj * K) + part);
                    loaded |= 1u << t;
                }
            }
#pragma unroll
            for (int t = 0; t < G; ++t) {
                const uint32_t u = (uint32_t)t * 32u + lane, job = u / G, part = u % G;
                if (loaded & (1u << t)) {
                    float* d = mine + job * (K + 1) + part * 4;
                    d[0] = c[t].x; d[1] = c[t].y; d[2] = c[t].z; d[3] = c[t].w;
                }
            }
            __syncwarp();
            if (a != kPrbNoParent) {
                const float* g = mine + lane * (K + 1);
                float sum = g[0];
#pragma unroll
                for (int j = 1; j < K; ++j) sum = __fadd_rn(sum, g[j]);
                par[a] = sum;
            }
            __syncwarp();
        }
    }
}

// First step of an update: every entry becomes the key (index << 32) | batch position (invalid
// entries: all ones, which sort last) with its priority in vals[batch position]; then the keys are
// sorted unless they already are, as indices straight from a stratified sample.
__device__ __forceinline__ void prb_update_keys(const PrbView& v, const PrbTeam& team, const PrbTreeWork& w,
                                                unsigned long long fill, unsigned long long* keys, float* vals)
{
    const uint32_t n2 = w.n2, rank = team.rank, nt = team.size;
    unsigned flags = 0;
    bool unsorted = false;
    unsigned long long my_key = kPrbInvalidKey;      // the key of entry `rank` (one-key-per-thread case)
    for (uint32_t b = rank; b < n2; b += nt) {
        unsigned long long key = kPrbInvalidKey;
        if (b < w.B) {
            const int32_t i = w.idx[b];
            float p = 0.0f;
            bool ok_p;
            if (w.raw) { p = w.val[b]; ok_p = prb_valid_priority(p); }
            else ok_p = prb_priority_pow(w.val[b], w.eps, w.alpha, p);
            if (i < 0 || (unsigned long long)i >= fill) flags |= PEARL_ST_BAD_INDEX;
            else if (!ok_p) flags |= PEARL_ST_BAD_PRIORITY;
            else key = ((unsigned long long)(uint32_t)i << 32) | b;
            vals[b] = p;
        }
        keys[b] = key;
        my_key = key;
    }
    if (flags) atomicOr(&v.state->status, flags);
    team.sync();

    for (uint32_t b = rank; b + 1 < n2; b += nt) unsorted |= (keys[b] > keys[b + 1]);
    unsorted = team.sync_or(unsorted);

    if (unsorted && n2 <= nt) {
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

}

// The tree work of one launch by one team (PEARL Section V-A: priority update; insertion =
// retrieval + update), read as SET + re-sum so that the result does not depend on scheduling.
//   Update: entries are keyed (index << 32) | batch position and sorted (skipped if they already
//   are, as indices straight from a stratified sample); the last entry of every run of equal
//   indices wins and writes its leaf.
//   Insertion: the n leaves of ring slots cursor .. cursor+n-1 (mod capacity) are written; they
//   come after the update, so an updated leaf that is also inserted keeps the inserted priority.
//   Then ONE pass per level, deepest first, re-sums every dirty parent: the first entry of every
//   run of equal ancestors in the sorted update list (sorted order survives dropping low digits
//   of the index, so nothing is compacted), and the contiguous parent range(s) of the inserted
//   slots.  No lock is taken; a parent reached both ways is computed twice with the same result.
// `fill` is the fill count before this launch (update indices must be below it).
__device__ __forceinline__ void prb_tree_readback(const PrbView& v, const PrbTeam& team, const PrbTreeWork& w,
                                                  uint64_t cursor, unsigned long long fill, unsigned char* smem)
{
    const uint32_t n2 = w.B ? w.n2 : 0u;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);
    float* vals = reinterpret_cast<float*>(smem + (size_t)n2 * sizeof(unsigned long long));
    float* scratch = reinterpret_cast<float*>(smem + ((size_t)n2 * 12 + 15) / 16 * 16);
    const uint32_t rank = team.rank, nt = team.size;
    const uint64_t N = v.capacity;
    const uint32_t D = v.depth, K = v.fanout, lg = v.log2_fanout;
    float* leaves = v.level[D];

    if (w.B) {
        prb_update_keys(v, team, w, fill, keys, vals);

        // winners write their leaves, unless the insertion below overwrites the slot anyway
        for (uint32_t s = rank; s < n2; s += nt) {
            const unsigned long long key = keys[s];
            if (key == kPrbInvalidKey) continue;
            const uint32_t i = (uint32_t)(key >> 32);
            const bool last = (s + 1 == n2) || ((uint32_t)(keys[s + 1] >> 32) != i);
            const uint64_t ahead = i >= cursor ? i - cursor : i + N - cursor;     // distance from the cursor along the ring
            if (last && !(ahead < w.n)) leaves[i] = vals[(uint32_t)key];
        }
    }

    if (w.n) {
        bool bad = false;
        for (uint32_t t = rank; t < w.n; t += nt) {
            uint64_t slot = cursor + t;
            if (slot >= N) slot -= N;
            float p = w.prio[t];
            if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
            leaves[slot] = p;
        }
        if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    }
    team.sync();

    // dirty leaf ranges of the insertion: A = [a0, a1]; if the ring wrapped also B = [0, b1]
    const uint64_t a0 = cursor;
    const uint64_t a1 = (w.n ? min(cursor + w.n, N) : cursor + 1) - 1;
    const bool wrapped = cursor + w.n > N;
    const uint64_t b1 = wrapped ? cursor + w.n - N - 1 : 0;

    for (int l = (int)D - 1; l >= 0; --l) {
        const uint32_t sh = lg * (D - (uint32_t)l);
        uint32_t pa0 = 0, cntA = 0, cntB = 0;
        if (w.n) {
            pa0 = (uint32_t)(a0 >> sh);
            cntA = (uint32_t)(a1 >> sh) - pa0 + 1;
            if (wrapped) cntB = (pa0 == 0) ? 0u : min((uint32_t)(b1 >> sh), pa0 - 1) + 1;   // parents of B not already in A
        }
        auto slot_parent = [&](uint32_t slot) -> uint32_t {
            if (slot < n2) {
                const unsigned long long key = keys[slot];
                if (key == kPrbInvalidKey) return kPrbNoParent;
                const uint32_t a = (uint32_t)(key >> 32) >> sh;
                const bool first = (slot == 0) || (((uint32_t)(keys[slot - 1] >> 32) >> sh) != a);
                return first ? a : kPrbNoParent;
            }
            const uint32_t i = slot - n2;
            return i < cntA ? pa0 + i : i - cntA;
        };
        const float* child = v.level[l + 1];
        float* par = v.level[l];
        const uint32_t n_slots = n2 + cntA + cntB;
        switch (K) {
        case 2: prb_resum_slots<2>(team, child, par, n_slots, slot_parent, scratch); break;
        case 4: prb_resum_slots<4>(team, child, par, n_slots, slot_parent, scratch); break;
        case 8: prb_resum_slots<8>(team, child, par, n_slots, slot_parent, scratch); break;
        case 16: prb_resum_slots<16>(team, child, par, n_slots, slot_parent, scratch); break;
        default: prb_resum_slots<32>(team, child, par, n_slots, slot_parent, scratch); break;
        }
        team.sync();
    }
}

// ---- forwarding path ----------------------------------------------------------------------
// The read-back path above pays one L2 round trip per level: a level's parents are written to
// global memory, and the next level reads them back.  When the whole job is small enough, the
// same result is produced without reading anything back:
//   1. the dirty leaves (update winners that the insertion does not overwrite, and the inserted
//      slots) are merged into ONE sorted list without sorting again: the update list is sorted,
//      the inserted slots are one or two runs of consecutive numbers, so every entry's place is
//      a count (closed form on one side, a binary search on the other);
//   2. level by level upwards, the distinct parents of the list are compacted into the next list
//      (node numbers only), and the K old children of every listed parent are fetched from
//      global memory into shared memory with asynchronous copies -- all levels at once, since
//      these addresses do not depend on any value;
//   3. once the copies have landed, values flow upwards in shared memory only: a parent
//      overwrites, in its fetched group, the children that are in the list below (a contiguous
//      run), sums the group left to right, keeps the sum for the level above and writes it to
//      global memory.
// The sums are the same operations in the same order as in the read-back path.

__host__ __device__ inline void prb_fwd_layout(const PrbView& v, uint32_t B, uint32_t n2, uint32_t n, PrbFwdLayout* L)
{
    const uint32_t D = v.depth, K = v.fanout;
    L->gs = K >= 4 ? K + 4 : 4;
    uint32_t at = (uint32_t)(((size_t)(B ? n2 : 0) * 12 + 15) / 16 * 16);
    L->off_scan = at; at += (kPrbFwdMaxPasses * 32 + 8) * 4;
    L->off_wnode = at; at += (B + 3) / 4 * 16;
    L->off_wval = at; at += (B + 3) / 4 * 16;
    for (int l = (int)D; l >= 0; --l) {
        // distinct dirty nodes of level l: at most one per update entry, plus the ancestors of n
        // consecutive slots (one more for a range that straddles a boundary, one more if the ring wrapped)
        const uint32_t sh = v.log2_fanout * (D - (uint32_t)l);
        uint64_t c64 = (uint64_t)B + (n ? (l == (int)D ? n : (sh >= 32 ? 0u : ((n - 1) >> sh)) + 3) : 0u);
        const uint32_t c = c64 > v.level_alloc[l] ? v.level_alloc[l] : (uint32_t)c64;
        L->cmax[l] = c;
        const uint32_t lst = (c + 3) / 4 * 16;
        L->off_node[l] = at; at += lst;
        L->off_val[l] = at; at += lst;
        L->off_first[l] = at; at += lst;
        L->off_group[l] = at;
        if (l < (int)D) at += c * L->gs * 4;
    }
    L->total = at;
}

// Decides whether the forwarding path applies to this job (few enough entries for the team, at
// most `limit` bytes of shared memory); if so fills in its layout and returns the bytes, else 0.
__host__ inline uint32_t prb_fwd_plan(const PrbView& v, PrbTreeWork* w, uint32_t team_threads, uint32_t limit)
{
    w->forward = 0;
    if ((uint64_t)w->B + w->n > (uint64_t)team_threads * kPrbFwdMaxPasses || w->n > v.capacity) return 0;
    if (w->B && w->n2 > team_threads * (uint32_t)kPrbFwdMaxPasses) return 0;
    prb_fwd_layout(v, w->B, w->n2, w->n, &w->fwd);
    if (w->fwd.total > limit) return 0;
    w->forward = 1;
    return w->fwd.total;
}

// Stable compaction by the team: entries e in [0, cnt) with flag(e) get consecutive positions in
// entry order; emit(e, pos) is called for each.  Returns the number of flagged entries.  Ends
// with a barrier, so what emit wrote is visible to the team.  s_scan: kPrbFwdMaxPasses*32+1 words.
template <typename Flag, typename Emit>
__device__ __forceinline__ uint32_t prb_team_compact(const PrbTeam& team, uint32_t cnt, Flag flag, Emit emit,
                                                     uint32_t* s_scan)
{
    const uint32_t lane = team.rank & 31u, warp = team.rank >> 5, nw = team.size >> 5;
    const uint32_t passes = (cnt + team.size - 1) / team.size;
    uint32_t ballots[kPrbFwdMaxPasses];
#pragma unroll
    for (int k = 0; k < kPrbFwdMaxPasses; ++k) {
        ballots[k] = 0;
        if ((uint32_t)k < passes) {
            const uint32_t e = (uint32_t)k * team.size + team.rank;
            ballots[k] = __ballot_sync(0xFFFFFFFFu, e < cnt && flag(e));
            if (lane == 0) s_scan[(uint32_t)k * nw + warp] = __popc(ballots[k]);
        }
    }
    team.sync();
    if (warp == 0) {
        const uint32_t S = passes * nw;                 // <= 256 counters: eight per lane
        uint32_t loc[8], sum = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t i = lane * 8u + q;
            loc[q] = i < S ? s_scan[i] : 0u;
            sum += loc[q];
        }
        uint32_t inc = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if ((int)lane >= d) inc += t;
        }
        uint32_t run = inc - sum;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t i = lane * 8u + q;
            if (i < S) s_scan[i] = run;
            run += loc[q];
        }
        if (lane == 31) s_scan[kPrbFwdMaxPasses * 32] = inc;
    }
    team.sync();
#pragma unroll
    for (int k = 0; k < kPrbFwdMaxPasses; ++k) {
        if ((uint32_t)k < passes && (ballots[k] >> lane) & 1u) {
            const uint32_t e = (uint32_t)k * team.size + team.rank;
            emit(e, s_scan[(uint32_t)k * nw + warp] + __popc(ballots[k] & ((1u << lane) - 1u)));
        }
    }
    const uint32_t total = s_scan[kPrbFwdMaxPasses * 32];
    team.sync();
    return total;
}

__device__ __forceinline__ void prb_cp_async16(void* smem_dst, const void* gsrc)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(prb_smem_addr(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void prb_cp_async8(void* smem_dst, const void* gsrc)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(prb_smem_addr(smem_dst)), "l"(gsrc) : "memory");
}

__device__ __forceinline__ void prb_tree_forward(const PrbView& v, const PrbTeam& team, const PrbTreeWork& w,
                                                 uint64_t cursor, unsigned long long fill, unsigned char* smem)
{
    const uint32_t n2 = w.B ? w.n2 : 0u;
    const uint32_t rank = team.rank, nt = team.size;
    const uint64_t N = v.capacity;
    const uint32_t D = v.depth, K = v.fanout, lg = v.log2_fanout;
    const PrbFwdLayout& L = w.fwd;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);
    float* vals = reinterpret_cast<float*>(smem + (size_t)n2 * sizeof(unsigned long long));
    uint32_t* s_scan = reinterpret_cast<uint32_t*>(smem + L.off_scan);
    uint32_t* wnode = reinterpret_cast<uint32_t*>(smem + L.off_wnode);
    float* wval = reinterpret_cast<float*>(smem + L.off_wval);
    auto node_of = [&](uint32_t l) { return reinterpret_cast<uint32_t*>(smem + L.off_node[l]); };
    auto val_of = [&](uint32_t l) { return reinterpret_cast<float*>(smem + L.off_val[l]); };
    auto first_of = [&](uint32_t l) { return reinterpret_cast<uint32_t*>(smem + L.off_first[l]); };
    auto group_of = [&](uint32_t l) { return reinterpret_cast<float*>(smem + L.off_group[l]); };

    // the inserted slots in increasing order: run B0 = [0, b_len) if the ring wrapped, then run A = [a0, a0 + a_len)
    const uint32_t n = w.n;
    const uint32_t a0 = (uint32_t)cursor;
    const uint32_t a_len = n ? (uint32_t)(min((uint64_t)cursor + n, N) - cursor) : 0u;
    const uint32_t b_len = n - a_len;
    auto inserted = [&](uint32_t i) { return i < b_len || (i >= a0 && i - a0 < a_len); };
    auto inserted_below = [&](uint32_t i) {           // inserted slots with a number < i
        return min(i, b_len) + (i > a0 ? min(i - a0, a_len) : 0u);
    };

    // ---- 1. update winners that survive the insertion, compacted in index order ----
    uint32_t cw = 0;
    if (w.B) {
        prb_update_keys(v, team, w, fill, keys, vals);
        cw = prb_team_compact(team, n2,
            [&](uint32_t s) {
                const unsigned long long key = keys[s];
                if (key == kPrbInvalidKey) return false;
                const uint32_t i = (uint32_t)(key >> 32);
                const bool last = (s + 1 == n2) || ((uint32_t)(keys[s + 1] >> 32) != i);
                return last && !inserted(i);
            },
            [&](uint32_t s, uint32_t pos) { wnode[pos] = (uint32_t)(keys[s] >> 32); wval[pos] = vals[(uint32_t)keys[s]]; },
            s_scan);
    }

    // ---- the merged list of dirty leaves; the leaves themselves go to global memory ----
    uint32_t* nodeD = node_of(D);
    float* valD = val_of(D);
    float* leaves = v.level[D];
    for (uint32_t j = rank; j < cw; j += nt) {
        const uint32_t i = wnode[j], pos = j + inserted_below(i);
        nodeD[pos] = i; valD[pos] = wval[j];
        leaves[i] = wval[j];
    }
    bool bad = false;
    for (uint32_t t = rank; t < n; t += nt) {
        uint64_t slot64 = cursor + t;
        if (slot64 >= N) slot64 -= N;
        const uint32_t slot = (uint32_t)slot64;
        float p = w.prio[t];
        if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
        uint32_t lo = 0, hi = cw;                      // winners with an index below this slot
        while (lo < hi) { const uint32_t mid = (lo + hi) >> 1; if (wnode[mid] < slot) lo = mid + 1; else hi = mid; }
        const uint32_t pos = lo + (slot < b_len ? slot : b_len + (slot - a0));
        nodeD[pos] = slot; valD[pos] = p;
        leaves[slot] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    team.sync();

    // ---- 2. lists of distinct parents, level by level, and the fetch of their old children ----
    uint32_t count[PRB_MAX_LEVELS];
    count[D] = cw + n;
    const uint32_t G = K >= 4 ? K / 4 : 1;               // copies per group (16 bytes each; 8 for fanout 2)
    for (int l = (int)D - 1; l >= 0; --l) {
        const uint32_t* below = node_of(l + 1);
        uint32_t* mine = node_of(l);
        uint32_t* first = first_of(l);
        count[l] = prb_team_compact(team, count[l + 1],
            [&](uint32_t j) { return j == 0 || (below[j - 1] >> lg) != (below[j] >> lg); },
            [&](uint32_t j, uint32_t pos) { mine[pos] = below[j] >> lg; first[pos] = j; },
            s_scan);
        float* grp = group_of(l);
        const float* child = v.level[l + 1];
        for (uint32_t u = rank; u < count[l] * G; u += nt) {
            const uint32_t job = u / G, part = u - job * G;
            const float* src = child + (uint64_t)mine[job] * K + part * 4;
            if (K >= 4) prb_cp_async16(grp + (size_t)job * L.gs + part * 4, src);
            else prb_cp_async8(grp + (size_t)job * L.gs, src);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    team.sync();

    // ---- 3. values flow upwards in shared memory ----
    for (int l = (int)D - 1; l >= 0; --l) {
        const uint32_t* below = node_of(l + 1);
        const float* below_val = val_of(l + 1);
        const uint32_t* mine = node_of(l);
        const uint32_t* first = first_of(l);
        float* my_val = val_of(l);
        float* grp = group_of(l);
        float* par = v.level[l];
        for (uint32_t j = rank; j < count[l]; j += nt) {
            const uint32_t P = mine[j];
            float* g = grp + (size_t)j * L.gs;
            for (uint32_t c = first[j]; c < count[l + 1] && (below[c] >> lg) == P; ++c)
                g[below[c] & (K - 1)] = below_val[c];
            float sum = g[0];
            for (uint32_t q = 1; q < K; ++q) sum = __fadd_rn(sum, g[q]);
            my_val[j] = sum;
            par[P] = sum;
        }
        team.sync();
    }
}

// The tree work of one launch: the forwarding path when the host found that the job fits it,
// the read-back path otherwise.  Same results either way.
__device__ __forceinline__ void prb_tree_team(const PrbView& v, const PrbTeam& team, const PrbTreeWork& w,
                                              uint64_t cursor, unsigned long long fill, unsigned char* smem)
{
    if (w.forward) prb_tree_forward(v, team, w, cursor, fill, smem);
    else prb_tree_readback(v, team, w, cursor, fill, smem);
}

#endif  // __CUDACC__
