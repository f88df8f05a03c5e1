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
    // key list and CTA `part` of `parts` takes its share -- by subtree where the tree has staged levels
    // (see prb_update_team), else the slots whose warp-sized group number is congruent to it, the
    // phases then separated by the cluster's hardware barrier.  parts == 1: one CTA.
    uint32_t part = 0, parts = 1;
    // PrbView::min_off in the kernels instantiated for a buffer with a min-tree, the constant 0 in the others
    // (which then carry none of its code)
    uint64_t min_off = 0;

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

// Taken by one thread per CTA of an insertion once the whole CTA holds the cursor: the last of the
// `participants` CTAs to get here publishes the new cursor.  Nothing later in those kernels reads
// it, so this happens while the copies are still running; no CTA waits for another.
//   kPrbPublishAll   a one-kernel insertion: cursor, fill and row_cursor (ticket: insert_ticket)
//   kPrbPublishTree  the tree kernel of a two-kernel insertion: cursor and fill (insert_ticket)
//   kPrbPublishRows  its row kernel: row_cursor (row_ticket)
constexpr int kPrbPublishTree = 1, kPrbPublishRows = 2, kPrbPublishAll = 3;
// (what the drawer of the last ticket does; a kernel whose drawing thread has other work to do first may
// draw early with prb_ticket and come back here with the answer when that work is done)
__device__ __forceinline__ void prb_publish(const PrbView& v, uint32_t n, uint64_t cursor, unsigned long long fill, int what)
{
    unsigned int* ticket = (what == kPrbPublishRows) ? &v.state->row_ticket : &v.state->insert_ticket;
    const uint64_t N = v.capacity;
    uint64_t c = cursor + n;
    if (c >= N) c -= N;
    if (what & kPrbPublishRows) v.state->row_cursor = c;
    if (what & kPrbPublishTree) {
        v.state->cursor = c;
        fill += n;
        v.state->fill = fill > N ? N : fill;
    }
    *ticket = 0;
}
__device__ __forceinline__ void prb_publish_if_last(const PrbView& v, uint32_t n, uint64_t cursor, unsigned long long fill,
                                                    uint32_t participants, int what = kPrbPublishAll)
{
    // (the cursor and fill reads of this CTA were stored to shared memory before the barrier this thread has
    // passed; the ticket's release/acquire pair orders them before the last drawer's stores)
    unsigned int* ticket = (what == kPrbPublishRows) ? &v.state->row_ticket : &v.state->insert_ticket;
    const unsigned int done = prb_ticket(ticket);
    if (done == participants - 1) prb_publish(v, n, cursor, fill, what);
}

// Frame-deduplicated layout: an insertion of n transitions at `cursor` writes n + prb_cleared_after(v, n)
// leaves -- the last ones zero: they belong to the slots that follow the new cursor, whose history the
// insertion overwrites once the ring has wrapped (before that they are empty and zero already) -- and the
// leaf of an episode-start marker (bit 1 of its done byte) is zero whatever priority is given.
// (`stack` is PrbView::stack in the kernels instantiated for the frame layout and the constant 0 in the
// others, which then carry none of this code: measured, its mere presence cost the short-row step 1.2 us)
__device__ __forceinline__ uint32_t prb_cleared_after(const PrbView& v, uint32_t n, uint32_t stack)
{
    if (stack == 0 || n == 0) return 0u;
    const uint64_t room = v.capacity - n;
    return room < stack ? (uint32_t)room : stack;
}
// ... and an update that names one of the `stack` slots that follow the cursor is stale.
__device__ __forceinline__ bool prb_history_less(const PrbView& v, uint64_t cursor, uint64_t i, uint32_t stack)
{
    return stack != 0 && (i + v.capacity - cursor) % v.capacity < stack;
}

// The top of the tree staged in shared memory for the re-sum passes: levels 1 .. v.top_levels as
// they lie in global memory from the start of level 1 (v.top_floats entries).  Below the staged
// levels a pass re-sums only the parents that the batch reaches; a re-summed parent of the deepest
// staged level is written to the staged copy as well, and the levels above it are then re-summed
// whole from shared memory (every parent always equals the sum of its children, so a parent none of
// whose children changed comes out as it was): no sorted keys, no round trip through L2.
// mem == nullptr: nothing is staged and every pass goes through global memory.
// mem_min: the same levels of the min-tree, staged the same way (nullptr: the buffer keeps none, or nothing is staged).
struct PrbTop {
    float* mem = nullptr;
    float* mem_min = nullptr;
};
__device__ __forceinline__ uint32_t prb_top_levels(const PrbView& v, const PrbTop& top) { return top.mem ? v.top_levels : 0u; }

// Starts the copy of the staged levels (asynchronous 16-byte copies, `nthreads` threads share them);
// prb_top_wait() by the same threads, then a barrier, before the first use.
__device__ __forceinline__ void prb_top_begin(const PrbView& v, const PrbTop& top, uint32_t rank, uint32_t nthreads)
{
    if (top.mem == nullptr) return;
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(top.mem);
    const float* src = v.level[1];
    for (uint32_t q = rank; q < v.top_floats / 4u; q += nthreads)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + q * 16u), "l"(src + q * 4u) : "memory");
    if (top.mem_min == nullptr) return;
    const uint32_t dst_min = (uint32_t)__cvta_generic_to_shared(top.mem_min);
    for (uint32_t q = rank; q < v.top_floats / 4u; q += nthreads)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_min + q * 16u), "l"(src + v.min_off + q * 4u) : "memory");
}

// A value for the staged copy of CTA 0 (see prb_resum): a plain store by a single CTA, a store through
// distributed shared memory by a CTA of a cluster.
__device__ __forceinline__ void prb_store_staged(float* t, float x, const PrbTeam& team)
{
    if (team.parts == 1) {
        *t = x;
    } else {
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(t)), "r"(0u));
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(x) : "memory");
    }
}
__device__ __forceinline__ void prb_top_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Re-sums parent `a` of level l >= T (T = staged levels) from its K children in global memory, left
// to right in binary32.  A parent of level T >= 1 also goes to the staged copy: in a cluster
// (team.parts > 1) the one of CTA 0, through distributed shared memory; the cluster barrier that
// ends the pass makes it visible there.
__device__ __forceinline__ void prb_resum(const PrbView& v, const PrbTop& top, const PrbTeam& team, uint32_t T, uint32_t l, uint64_t a)
{
    const uint32_t K = v.fanout;
    if (!PRB_IN_BOUNDS(v, a * K + K <= v.level_alloc[l + 1] && a < v.level_alloc[l])) return;
    float x, m = 0.0f;
    if (team.min_off) {     // the min-tree's node as well: from the leaves themselves one level up, else from its own children
        const float* c = v.level[l + 1] + a * K;
        prb_sum_and_min_dyn(c, c + (l + 1 == v.depth ? 0 : team.min_off), K, x, m);
        (v.level[l] + team.min_off)[a] = m;
    } else {
        x = prb_sum_children_dyn(v.level[l + 1] + a * K, K);
    }
    v.level[l][a] = x;
    if (l == T && l >= 1) {
        prb_store_staged(top.mem + v.top_off[l] + a, x, team);
        if (team.min_off) prb_store_staged(top.mem_min + v.top_off[l] + a, m, team);
    }
}

// Left-to-right binary32 sum of K staged children (all loads first, then the chain of additions).
template <int K>
__device__ __forceinline__ float prb_sum_staged(const float* c)
{
    if (K == 2) {
        const float2 f = *reinterpret_cast<const float2*>(c);
        return __fadd_rn(f.x, f.y);
    } else {
        float4 u[K / 4 > 0 ? K / 4 : 1];
#pragma unroll
        for (int q = 0; q < K / 4; ++q) u[q] = reinterpret_cast<const float4*>(c)[q];
        float x = __fadd_rn(__fadd_rn(__fadd_rn(u[0].x, u[0].y), u[0].z), u[0].w);
#pragma unroll
        for (int q = 1; q < K / 4; ++q) x = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(x, u[q].x), u[q].y), u[q].z), u[q].w);
        return x;
    }
}

// The smallest positive of K staged children (0 if none); 16-byte loads, as for the sums.
template <int K>
__device__ __forceinline__ float prb_min_staged(const float* c)
{
    unsigned best = 0xFFFFFFFFu;
    auto take = [&best](float u) { if (u > 0.0f) best = min(best, __float_as_uint(u)); };
    if (K == 2) {
        const float2 f = *reinterpret_cast<const float2*>(c);
        take(f.x); take(f.y);
    } else {
        float4 u[K / 4 > 0 ? K / 4 : 1];
#pragma unroll
        for (int q = 0; q < K / 4; ++q) u[q] = reinterpret_cast<const float4*>(c)[q];
#pragma unroll
        for (int q = 0; q < K / 4; ++q) { take(u[q].x); take(u[q].y); take(u[q].z); take(u[q].w); }
    }
    return best == 0xFFFFFFFFu ? 0.0f : __uint_as_float(best);
}

// The passes over the staged levels, by one CTA: parents of level T-1, then T-2, ... then the root,
// each level whole; a parent that comes out different is stored, staged copy and global memory.
// The min-tree's staged levels go through the same passes.
template <int K>
__device__ __forceinline__ void prb_top_passes_k(const PrbView& v, const PrbTop& top, const PrbTeam& team, uint32_t T)
{
    constexpr uint32_t lg = K == 2 ? 1 : K == 4 ? 2 : K == 8 ? 3 : K == 16 ? 4 : 5;
    // nodes of level T (then of the levels above, one division by K each, rounded up)
    uint32_t n_l = (uint32_t)((v.capacity - 1) >> (lg * (v.depth - T))) + 1u;
    for (int l = (int)T - 1; l >= 0; --l) {
        n_l = (n_l + K - 1) >> lg;
        const float* child = top.mem + v.top_off[l + 1];
        float* own = top.mem + v.top_off[l];       // (not used for the root)
        for (uint32_t i = team.rank; i < n_l; i += team.size) {
            if (!PRB_IN_BOUNDS(v, v.top_off[l + 1] + (i + 1) * K <= v.top_floats && i < v.level_alloc[l])) continue;
            const float x = prb_sum_staged<K>(child + (size_t)i * K);
            if (l == 0) {
                v.level[0][0] = x;
            } else if (__float_as_uint(x) != __float_as_uint(own[i])) {
                own[i] = x;
                v.level[l][i] = x;
            }
            if (team.min_off) {
                const float m = prb_min_staged<K>(top.mem_min + v.top_off[l + 1] + (size_t)i * K);
                float* own_min = top.mem_min + v.top_off[l];
                if (l == 0) {
                    (v.level[0] + team.min_off)[0] = m;
                } else if (__float_as_uint(m) != __float_as_uint(own_min[i])) {
                    own_min[i] = m;
                    (v.level[l] + team.min_off)[i] = m;
                }
            }
        }
        if (l) team.sync();
    }
}
__device__ __forceinline__ void prb_top_passes(const PrbView& v, const PrbTop& top, const PrbTeam& team, uint32_t T)
{
    switch (v.fanout) {
    case 2: prb_top_passes_k<2>(v, top, team, T); break;
    case 4: prb_top_passes_k<4>(v, top, team, T); break;
    case 8: prb_top_passes_k<8>(v, top, team, T); break;
    case 16: prb_top_passes_k<16>(v, top, team, T); break;
    default: prb_top_passes_k<32>(v, top, team, T); break;
    }
}

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

// Sort keys are (index, batch position) packed into one word, the index in the high bits: all
// different.  A skipped entry keeps its position under an index field of all ones and sorts last.
constexpr unsigned long long kPrbInvalidKey = ~0ull;
__device__ __forceinline__ bool prb_key_invalid(unsigned long long key) { return (uint32_t)(key >> 32) == 0xFFFFFFFFu; }

// One key per thread (threads rank < n2, whole warps): sorts them and returns the key of place
// `rank`; keys[] holds the sorted order afterwards.  Every warp sorts its 32 keys with a bitonic
// network of shuffles; a key's place in the whole is its place in its own run plus, for every other
// run, the number of keys below it there -- a six-step binary search each, independent of one another.
template <typename KeyT>
__device__ __forceinline__ KeyT prb_sort_one_per_thread(const PrbTeam& team, KeyT key, KeyT* keys, uint32_t n2)
{
    const uint32_t rank = team.rank, lane = rank & 31u, run = rank >> 5;
    const bool active = rank < n2;
    if (active) {
        for (uint32_t k = 2; k <= 32; k <<= 1) {
            for (uint32_t j = k >> 1; j > 0; j >>= 1) {
                const KeyT other = __shfl_xor_sync(0xFFFFFFFFu, key, j);
                const bool keep_min = ((lane & k) == 0) == ((lane & j) == 0);
                key = keep_min ? (key < other ? key : other) : (key > other ? key : other);
            }
        }
        keys[rank] = key;
    }
    team.sync();
    uint32_t place = lane;
    if (active) {
        const uint32_t runs = n2 >> 5;
#pragma unroll 4
        for (uint32_t r = 0; r < runs; ++r) {
            const KeyT* other = keys + (r << 5);
            uint32_t below = 0;
#pragma unroll
            for (uint32_t step = 16; step > 0; step >>= 1)
                if (other[below + step - 1] < key) below += step;
            below += (other[below] < key) ? 1u : 0u;
            place += (r == run) ? 0u : below;
        }
    }
    team.sync();
    if (active) keys[place] = key;
    team.sync();
    return active ? keys[rank] : key;
}

// What one thread knows of the sorted batch when every thread holds one entry: the index and batch
// position at its place, and the indices at the places before and after (0xFFFFFFFF: skipped entry,
// or no such place -- no valid index equals it, nor any of its ancestors' numbers).
struct PrbSlot {
    uint32_t idx, pos, prev, next;
};
template <typename KeyT>
__device__ __forceinline__ PrbSlot prb_sorted_slot(const PrbTeam& team, bool valid, uint32_t i, uint32_t n2, uint32_t shift, KeyT* keys)
{
    const uint32_t rank = team.rank;
    const KeyT none = (KeyT)(~(KeyT)0) >> shift;          // index field of all ones
    KeyT key = ((valid ? (KeyT)i : none) << shift) | (KeyT)rank;
    if (rank < n2) keys[rank] = key;
    team.sync();
    // indices that come straight from a stratified sample are already in order; sort only if needed
    bool unsorted = (rank + 1 < n2) && keys[rank] > keys[rank + 1];
    unsorted = team.sync_or(unsorted);
    if (unsorted) key = prb_sort_one_per_thread<KeyT>(team, key, keys, n2);
    PrbSlot out = PrbSlot{0xFFFFFFFFu, 0u, 0xFFFFFFFFu, 0xFFFFFFFFu};
    if (rank < n2) {
        const KeyT f = key >> shift;
        if (f != none) out.idx = (uint32_t)f;
        out.pos = (uint32_t)(key & (((KeyT)1 << shift) - 1));
        if (rank > 0) { const KeyT g = keys[rank - 1] >> shift; if (g != none) out.prev = (uint32_t)g; }
        if (rank + 1 < n2) { const KeyT g = keys[rank + 1] >> shift; if (g != none) out.next = (uint32_t)g; }
    }
    return out;
}

// A batch of B entries is padded to n2 = the smallest power of two >= max(B, 32): whole warps.
__host__ __device__ inline uint32_t prb_update_n2(uint32_t B)
{
    uint32_t n2 = 32;
    while (n2 < B) n2 <<= 1;
    return n2;
}

// Shared memory an update of a batch padded to n2 entries needs: keys, then values.
__host__ __device__ inline size_t prb_update_smem_bytes(uint32_t n2)
{
    return (size_t)n2 * (sizeof(unsigned long long) + sizeof(float));
}

// Batched priority update by one team (PEARL Section V-A, "priority update", read as set +
// re-sum).  Entries are keyed (index, batch position) and sorted -- with one entry per thread by
// warp-wide sorting networks and a merge by rank, each thread then holding its place's index and
// its neighbours' in registers; with more, by a bitonic network in shared memory.  The last entry
// of every run of equal indices wins and writes its leaf (raw == 2: adds the run's changes to the
// leaf in batch order); then, level by level from the deepest down to the staged top, the first
// entry of every run of equal ancestors re-sums that ancestor from its children in left-to-right
// order, and the staged levels are re-summed whole (prb_top_passes).  Sorted order survives
// dropping low digits of the index, so no list is compacted and no lock is taken.
// raw: 0 = val holds TD errors (transformed), 1 = priorities, 2 = changes of priorities.
// n2 = prb_update_n2(B); smem holds
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
                                                uint32_t stale = 0, PrbTop top = PrbTop{}, const unsigned char* __restrict__ ins_done = nullptr,
                                                uint32_t stack = 0)
{
    // (frames: the insertion's dirty leaves reach past its n transitions; cursor, fill and priorities do not)
    const uint32_t n_leaves = n + prb_cleared_after(v, n, stack);
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);
    float* vals = reinterpret_cast<float*>(smem + (size_t)n2 * sizeof(unsigned long long));
    const uint32_t rank = team.rank, nt = team.size;
    const bool one_each = n2 <= nt;        // every thread holds one entry, in registers from the sort on
    const uint64_t N = v.capacity;

    // transform and validate; vals[b] = the priority entry b would write
    unsigned flags = 0;
    float wmax = 0.0f;                 // largest priority this thread accepted
    bool my_valid = false;
    uint32_t my_idx = 0;
    for (uint32_t b = rank; b < n2; b += nt) {
        unsigned long long key = 0xFFFFFFFF00000000ull | b;
        if (b < B) {
            const bool mine = pre.has_update && b == rank;
            const int32_t i = mine ? pre.idx : idx[b];
            const float x = mine ? pre.val : val[b];
            float p = 0.0f;
            bool ok_p;
            if (raw == 2) { p = x; ok_p = fabsf(x) <= 3.402823466e+38f; }      // a change: any finite value
            else if (raw) { p = x; ok_p = prb_valid_priority(p); }
            else ok_p = prb_priority_pow(x, eps, alpha, p);
            // stale: one of the `stale` slots written most recently, i.e. overwritten since it was sampled
            const uint64_t back = (i >= 0 && stale) ? (cursor + N - 1 - (uint64_t)i) % N : ~0ull;
            if (i < 0 || (unsigned long long)i >= fill) flags |= PEARL_ST_BAD_INDEX;
            else if (back < stale || prb_history_less(v, cursor, (uint64_t)i, stack)) flags |= PEARL_ST_STALE;
            else if (!ok_p) flags |= PEARL_ST_BAD_PRIORITY;
            else { key = ((unsigned long long)(uint32_t)i << 32) | b; if (raw != 2) wmax = fmaxf(wmax, p); my_valid = true; my_idx = (uint32_t)i; }
            vals[b] = p;
        }
        if (!one_each) keys[b] = key;
    }
    if (flags && team.part == 0) atomicOr(&v.state->status, flags);
    prb_note_priorities(v.state, wmax, team.part == 0);
    prb_top_wait();                // (the staged top of the tree, if the kernel started a copy)

    PrbSlot slot = PrbSlot{0xFFFFFFFFu, 0u, 0xFFFFFFFFu, 0xFFFFFFFFu};
    if (one_each) {
        // index and position share a 32-bit key when they fit: half the shuffles and comparisons
        const uint32_t pb = 31u - (uint32_t)__clz(n2);
        if (N < (1ull << (32u - pb)))
            slot = prb_sorted_slot<uint32_t>(team, my_valid, my_idx, n2, pb, reinterpret_cast<uint32_t*>(smem));
        else
            slot = prb_sorted_slot<unsigned long long>(team, my_valid, my_idx, n2, 32u, keys);
    } else {
        team.sync();
        bool unsorted = false;
        for (uint32_t b = rank; b + 1 < n2; b += nt) unsorted |= (keys[b] > keys[b + 1]);
        if (team.sync_or(unsorted)) {
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

    // How the CTAs of a cluster share the work below the staged levels: by subtree.  A leaf, and every node
    // above it down to the deepest staged level T, belongs to the CTA that its ancestor on level T falls to; what
    // a pass reads was then written by the same CTA, and a barrier of that CTA separates the passes -- not the
    // cluster's, whose release has every CTA wait until its stores have reached L2.  (Without staged levels the
    // slots are dealt out by position and the cluster's barrier separates the passes.)
    const uint32_t lg = v.log2_fanout, T = prb_top_levels(v, top);
    const bool by_subtree = team.parts > 1 && T >= 1;
    const uint32_t sh_top = min(lg * (v.depth - T), 63u);
    auto mine = [&](uint64_t leaf, uint32_t slot_no) {
        return by_subtree ? ((leaf >> sh_top) % team.parts) == team.part : team.takes(slot_no);
    };
    auto mine_node = [&](uint64_t a, uint32_t l, uint32_t slot_no) {      // node a of level l >= T
        return by_subtree ? ((a >> (lg * (l - T))) % team.parts) == team.part : team.takes(slot_no);
    };
    auto pass_sync = [&](bool next_is_top) {
        if (by_subtree && !next_is_top) team.sync();
        else team.phase_sync();
    };
    float* leaves = v.level[v.depth];
    if (raw == 2) {
        // Changes instead of values (n == 0): the last entry of a run of equal indices adds the run's
        // changes to the leaf one by one in batch order -- the order of the sorted run -- skipping a
        // sum that is not a valid priority.
        float dmax = 0.0f;
        bool refused = false;
        auto add_change = [&](float& p, float change) {
            const float q = __fadd_rn(p, change);
            if (prb_valid_priority(q)) { p = q; dmax = fmaxf(dmax, q); }
            else refused = true;
        };
        if (one_each) {
            // the sorted indices and positions of all slots, in place of the keys
            uint32_t* sidx = reinterpret_cast<uint32_t*>(smem);
            uint32_t* spos = sidx + n2;
            team.sync();
            if (rank < n2) { sidx[rank] = slot.idx; spos[rank] = slot.pos; }
            team.sync();
            if (slot.idx != 0xFFFFFFFFu && slot.next != slot.idx && mine(slot.idx, rank)) {
                uint32_t s0 = rank;
                while (s0 > 0 && sidx[s0 - 1] == slot.idx) --s0;
                if (PRB_IN_BOUNDS(v, slot.idx < v.level_alloc[v.depth])) {
                    float p = __ldcg(leaves + slot.idx);
                    for (uint32_t s2 = s0; s2 <= rank; ++s2) add_change(p, vals[spos[s2]]);
                    leaves[slot.idx] = p;
                }
            }
        } else {
            for (uint32_t s1 = rank; s1 < n2; s1 += nt) {
                const unsigned long long key = keys[s1];
                if (prb_key_invalid(key) || !mine(key >> 32, s1)) continue;
                const uint32_t i = (uint32_t)(key >> 32);
                if (s1 + 1 < n2 && (uint32_t)(keys[s1 + 1] >> 32) == i) continue;      // not the last of its run
                uint32_t s0 = s1;
                while (s0 > 0 && (uint32_t)(keys[s0 - 1] >> 32) == i) --s0;
                float p = __ldcg(leaves + i);
                for (uint32_t s2 = s0; s2 <= s1; ++s2) add_change(p, vals[(uint32_t)keys[s2]]);
                leaves[i] = p;
            }
        }
        if (refused) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
        prb_note_priorities(v.state, dmax, true);
    } else if (one_each) {
        if (slot.idx != 0xFFFFFFFFu && slot.next != slot.idx && mine(slot.idx, rank)) {
            const uint64_t ahead = slot.idx >= cursor ? slot.idx - cursor : slot.idx + N - cursor;   // distance from the cursor along the ring
            if (!(ahead < n_leaves) && PRB_IN_BOUNDS(v, slot.idx < v.level_alloc[v.depth] && slot.pos < n2)) leaves[slot.idx] = vals[slot.pos];
        }
    } else {
        for (uint32_t s = rank; s < n2; s += nt) {
            const unsigned long long key = keys[s];
            if (prb_key_invalid(key) || !mine(key >> 32, s)) continue;
            const uint32_t i = (uint32_t)(key >> 32);
            const bool last = (s + 1 == n2) || ((uint32_t)(keys[s + 1] >> 32) != i);
            const uint64_t ahead = i >= cursor ? i - cursor : i + N - cursor;
            if (last && !(ahead < n_leaves) && PRB_IN_BOUNDS(v, i < v.level_alloc[v.depth] && (uint32_t)key < n2)) leaves[i] = vals[(uint32_t)key];
        }
    }
    bool bad = false;
    float imax = 0.0f;
    // without priorities the new transitions take the running maximum, this update's writes included
    // (reported by CTA 0: in a cluster the others read it after a barrier)
    if (n && prio == nullptr && team.parts > 1) { __threadfence(); team.phase_sync(); }
    const float dflt = (n && prio == nullptr) ? prb_default_priority(__ldcg(&v.state->max_prio_bits)) : 0.0f;
    for (uint32_t t = rank; t < n_leaves; t += nt) {
        uint64_t at = cursor + t;
        if (at >= N) at -= N;
        if (!mine(at, t)) continue;
        float p = 0.0f;
        if (t < n && !(stack && (ins_done[t] & kPrbEpisodeStart))) {
            p = prio == nullptr ? dflt : ((pre.has_prio && t == rank) ? pre.prio : prio[t]);
            if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
            else imax = fmaxf(imax, p);
        }
        if (PRB_IN_BOUNDS(v, at < N)) leaves[at] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    if (n) prb_note_priorities(v.state, imax, true);      // (every CTA of a cluster wrote leaves of its own; a first default insertion writes 1)
    pass_sync(false);

    // re-sum the ancestors below the staged levels, deepest level first: the first entry of every run
    // of equal ancestors does it; the insertion dirties parent range A = [a0, a1] >> sh and, if the
    // ring wrapped, B = [0, b1] >> sh
    const uint64_t a0 = cursor, a1 = (n ? min(cursor + n_leaves, N) : cursor + 1) - 1;
    const bool wrapped = cursor + n_leaves > N;
    const uint64_t b1 = wrapped ? cursor + n_leaves - N - 1 : 0;
    for (int l = (int)v.depth - 1; l >= (int)T; --l) {
        const uint32_t sh = min(lg * (v.depth - (uint32_t)l), 31u);      // (indices are below 2^31)
        if (one_each) {
            const uint32_t a = slot.idx >> sh;
            if (slot.idx != 0xFFFFFFFFu && (slot.prev >> sh) != a && mine_node(a, (uint32_t)l, rank)) prb_resum(v, top, team, T, (uint32_t)l, a);
        } else {
            for (uint32_t s = rank; s < n2; s += nt) {
                const unsigned long long key = keys[s];
                if (prb_key_invalid(key)) continue;
                const uint32_t a = (uint32_t)(key >> 32) >> sh;
                if (!mine_node(a, (uint32_t)l, s)) continue;
                const bool first = (s == 0) || (((uint32_t)(keys[s - 1] >> 32) >> sh) != a);
                if (first) prb_resum(v, top, team, T, (uint32_t)l, a);
            }
        }
        if (n) {
            const uint64_t pa0 = a0 >> sh, cntA = (a1 >> sh) - pa0 + 1;
            uint64_t cntB = 0;
            if (wrapped) cntB = (pa0 == 0) ? 0 : min(b1 >> sh, pa0 - 1) + 1;     // parents of B not already in A
            for (uint64_t i = rank; i < cntA + cntB; i += nt) {
                const uint64_t a = (i < cntA) ? pa0 + i : i - cntA;
                if (mine_node(a, (uint32_t)l, (uint32_t)i)) prb_resum(v, top, team, T, (uint32_t)l, a);
            }
        }
        pass_sync((uint32_t)l == T);
    }
    // the staged levels: CTA 0 alone
    if (team.part == 0) prb_top_passes(v, top, team, T);
}

// Tree part of an insertion by one team: write the n leaves of ring slots cursor .. cursor+n-1
// (mod capacity), then re-sum the dirty parents level by level.  A contiguous slot range dirties
// a contiguous parent range on every level (two ranges if the ring wrapped), so nothing is sorted.
__device__ __forceinline__ void prb_insert_tree_team(const PrbView& v, const PrbTeam& team, uint32_t n,
                                                     const float* __restrict__ prio, uint64_t cursor,
                                                     PrbPreloaded pre = PrbPreloaded{false, false, 0, 0.0f, 0.0f},
                                                     unsigned max_bits = 0, PrbTop top = PrbTop{},
                                                     const unsigned char* __restrict__ ins_done = nullptr, uint32_t stack = 0)
{
    const uint64_t N = v.capacity;
    const uint32_t n_leaves = n + prb_cleared_after(v, n, stack);
    const uint32_t D = v.depth, lg = v.log2_fanout, T = prb_top_levels(v, top);
    float* leaves = v.level[D];
    bool bad = false;
    float imax = 0.0f;
    const float dflt = prb_default_priority(max_bits);     // used when no priorities are given
    for (uint32_t t = team.rank; t < n_leaves; t += team.size) {
        uint64_t slot = cursor + t;
        if (slot >= N) slot -= N;
        float p = 0.0f;
        if (t < n && !(stack && (ins_done[t] & kPrbEpisodeStart))) {
            p = prio == nullptr ? dflt : ((pre.has_prio && t == team.rank) ? pre.prio : prio[t]);
            if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
            else imax = fmaxf(imax, p);
        }
        if (PRB_IN_BOUNDS(v, slot < N)) leaves[slot] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    prb_note_priorities(v.state, imax, true);                       // (a first default insertion writes 1)
    prb_top_wait();
    team.sync();
    // dirty leaf ranges: A = [a0, a1]; if the ring wrapped also B = [0, b1]
    const uint64_t a0 = cursor;
    const uint64_t a1 = min(cursor + n_leaves, N) - 1;
    const bool wrapped = cursor + n_leaves > N;
    const uint64_t b1 = wrapped ? cursor + n_leaves - N - 1 : 0;
    for (int l = (int)D - 1; l >= (int)T; --l) {
        const uint32_t sh = lg * (D - (uint32_t)l);
        const uint64_t pa0 = a0 >> sh, pa1 = a1 >> sh;
        const uint64_t cntA = pa1 - pa0 + 1;
        uint64_t cntB = 0;
        if (wrapped) {
            const uint64_t pb1 = b1 >> sh;
            cntB = (pa0 == 0) ? 0 : min(pb1, pa0 - 1) + 1;   // parents of B not already in A
        }
        for (uint64_t i = team.rank; i < cntA + cntB; i += team.size)
            prb_resum(v, top, team, T, (uint32_t)l, (i < cntA) ? pa0 + i : i - cntA);
        team.sync();
    }
    prb_top_passes(v, top, team, T);
}

#endif  // __CUDACC__
