// Internal declarations shared by the CUDA translation units of libpearl_prb.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pearl_prb.h"

// The checked build (-DPEARL_CHECKED; build.py --checked): every index into a tree level, the Data Storage,
// a batch or a staging area is compared with its extent before it is used; an index out of range raises
// PEARL_ST_INTERNAL and the access is skipped, nothing traps.  The test suite runs against that library
// too: a bit that no test expects is a finding.  In the ordinary build the checks compile to nothing.
#ifdef PEARL_CHECKED
#define PRB_IN_BOUNDS(v, cond) ((cond) ? true : (atomicOr(&(v).state->status, PEARL_ST_INTERNAL), false))
#else
#define PRB_IN_BOUNDS(v, cond) (true)
#endif

#define PRB_MAX_LEVELS 32       // level 0 (root) .. level D (leaves), D <= 30 for fanout 2
#define PRB_NUM_FIELDS 5        // obs, next_obs, act, rew, done
constexpr uint32_t kPrbHandoffs = 4;    // hand-off areas of a two-kernel sample (descents of later calls run ahead of earlier calls' row copies)

enum PrbField { F_OBS = 0, F_NEXT_OBS = 1, F_ACT = 2, F_REW = 3, F_DONE = 4 };
constexpr unsigned char kPrbEpisodeStart = 2;      // done byte, bit 1 (frame-deduplicated layout)

// Mutable state of a buffer; lives in device memory so that enqueued work never depends on
// host-side copies of it.
struct PrbState {
    unsigned long long cursor;        // next ring slot to be written
    unsigned long long fill;          // transitions stored, <= capacity
    unsigned long long sample_calls;  // successful sample calls so far (Philox counter words 2,3)
    unsigned long long pmin_bits;     // smallest positive leaf (bits of a binary32), filled in before a sample that normalises over the buffer
    unsigned int status;              // PEARL_ST_* bits
    unsigned int insert_ticket;       // CTAs of the running insert kernel that have finished
    unsigned int sample_ticket;       // CTAs of the running sample kernel that have finished
    unsigned int max_prio_bits;       // bits of the largest priority written so far (0: none yet)
    unsigned int wide_arrived;        // grid barrier of the running many-CTA update: arrivals so far (0 between launches that ended well)
    unsigned int wide_done;           // its CTAs that have passed their last barrier
    unsigned long long wide_wmax_bits; // largest raw weight of the running large-batch sample (bits of a binary64; 0 between calls)
    // The ring cursor as the kernels that copy rows see it.  An insertion whose tree work and row copy are
    // two kernels on two streams advances `cursor` (and `fill`) from the tree kernel and `row_cursor` from
    // the row kernel, each with a ticket of its own, so that neither kernel's bookkeeping waits for, or
    // races with, the other's; a one-kernel insertion advances both.  Equal whenever no insertion is running.
    unsigned long long row_cursor;
    unsigned int row_ticket;          // CTAs of the running row kernel that have read row_cursor
    unsigned int wide_poisoned;       // a many-CTA update gave up at its barrier once: the barrier's state is not to be trusted, and
                                      // neither is the tree; every later many-CTA update raises INTERNAL and does nothing
};

// Geometry and device addresses, passed to kernels by value.
struct PrbView {
    // (the scalars and the short arrays first, the per-level arrays last: a kernel reads its parameters
    // through the constant cache, and the few lines at the front serve the start of every kernel)
    PrbState* state;
    uint64_t capacity;
    uint32_t fanout;                  // K
    uint32_t log2_fanout;
    uint32_t depth;                   // D
    uint32_t max_batch;
    // levels 1 .. top_levels (< depth; 0: none) lie in the first top_floats entries from the start of
    // level 1: the part of the tree a CTA may stage in shared memory (at most kPrbTopFloats entries)
    uint32_t top_levels;
    uint32_t top_floats;
    // Frame-deduplicated layout (stack > 0): the obs store keeps ONE frame of field_bytes[F_OBS] bytes per slot
    // (the newest frame of the transition's next observation), there is no next_obs store
    // (field_bytes[F_NEXT_OBS] == 0), and a sample rebuilds both observations, `stack` frames each, from
    // consecutive slots (each output row is stack * field_bytes[F_OBS] bytes).  Bit 1 of a slot's done byte
    // marks an episode start.
    uint32_t stack;
    uint32_t field_bytes[PRB_NUM_FIELDS];
    uint32_t field_vec[PRB_NUM_FIELDS];   // copy granule in bytes: largest power of two <= 16 dividing field_bytes
    // Bytes from slot i to slot i + 1 of field f in the store.  Long rows are stored field by field
    // (pitch = field_bytes).  When every field is short the store is ONE padded record per transition
    // (pitch = the record's size, a multiple of 64 bytes; store[f] points at field f of record 0), so that a
    // sampled transition is a few consecutive sectors instead of a sector or three per field.
    uint32_t field_pitch[PRB_NUM_FIELDS];
    unsigned char* store[PRB_NUM_FIELDS];
    double* wraw;                     // scratch: raw IS weights of the running sample call, max_batch entries
    // A sample of long rows that is issued as two kernels (descents, then the row copy) hands indices
    // and leaf priorities from the first to the second through one of a few areas of the slab, used in turn:
    // a 256-byte header (PrbHandoffHeader), max_batch indices, max_batch priorities.
    unsigned char* handoff[kPrbHandoffs];
    // Min-tree (optional, PEARL_LAYOUT_MIN_TREE): node (l, a), l < depth, of a second tree holds the smallest
    // positive leaf below it (0: none); it lies min_off entries behind the sum tree's node, level[l] + min_off
    // (the leaves serve both trees).  0: no min-tree.  Its root is what weights normalised over the whole
    // buffer divide by, without a scan of the leaves.
    uint64_t min_off;
    float* level[PRB_MAX_LEVELS];     // level[l] holds K * n_{l-1} entries (level[0]: 1)
    uint32_t level_alloc[PRB_MAX_LEVELS];   // entries of level l, zero padding included
    uint32_t top_off[PRB_MAX_LEVELS];     // entries from the start of level 1 to the start of staged level l (l >= 1)
};

// Dense caller-side batch, one pointer per field (NULL = field skipped).
struct PrbBatch {
    unsigned char* ptr[PRB_NUM_FIELDS];
};

// A second stream of the handle and the two events that fork it off the caller's stream and join it
// again: with long rows the tree work of an update + insertion runs there, beside the row copy.
struct PrbFork {
    cudaStream_t side;
    cudaEvent_t fork, join;
};

// Kernel launchers; each returns the number of kernels launched, or -1 on a launch error.
// (upd_B > 0 runs a priority update of that batch before the insertion's tree work: in the same
// kernel for short rows; for long rows in a tree kernel of its own on fork->side, or, without a
// fork, in launches of its own before the insertion's)
int prb_launch_insert(const PrbView& v, uint32_t n, const PrbBatch& src, const float* d_prio, cudaStream_t s,
                      uint32_t upd_B = 0, const int32_t* upd_idx = nullptr, const float* upd_val = nullptr,
                      int upd_raw = 0, float alpha = 0.0f, float eps = 0.0f, const PrbFork* fork = nullptr,
                      bool* forked_out = nullptr, bool rows_only = false);
// (rows_only: long rows, and the insertion's tree work is some other launch's -- a prb_launch_update with
// ins_n = n: this one copies the rows and advances the row cursor, nothing else)
// Streams and events of a sample call that is issued as sub-batches (the paper's sub-batch
// streaming, Section IV-C): sub-batch i runs on stream[i]; done[i] fires when its rows are in place.
constexpr uint32_t kPrbMaxSubBatches = 4;
struct PrbSubStreams {
    cudaStream_t stream[kPrbMaxSubBatches];
    cudaEvent_t done[kPrbMaxSubBatches];
    cudaEvent_t fork;
};

// (buffer_norm != 0: weights divided by the largest weight of the whole buffer, found by a scan of
// the leaves in a launch of its own, instead of the batch's;
// uniform != 0: uniform replay, no tree walk, all weights 1; n_sub > 1: as that many launches, one
// per sub-batch of consecutive strata, each on a stream of `subs`, joined back into s)
int prb_launch_sample(const PrbView& v, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w,
                      const PrbBatch& dst, cudaStream_t s, int uniform = 0, uint32_t n_sub = 1,
                      const PrbSubStreams* subs = nullptr, int buffer_norm = 0);
// A sample of long rows as two kernels.  The first walks the tree and leaves, in a hand-off area of the
// slab (one of PrbView::handoff), what the second needs: a header, the leaf index of every stratum and
// that leaf's priority.  The second copies the rows (and turns the priorities into weights meanwhile).
struct PrbHandoffHeader {
    unsigned int found;               // 1: the sample found its batch; 0: the buffer was empty, nothing is to be written
    unsigned int buffer_norm;         // 1: weights are divided by the weight of pmin, else by the largest of the batch
    unsigned long long fill;          // transitions stored when the sample was taken
    float total;                      // the root then
    float pmin;                       // smallest positive priority stored (buffer_norm only)
};
__host__ __device__ inline const PrbHandoffHeader* prb_handoff_header(const unsigned char* h) { return reinterpret_cast<const PrbHandoffHeader*>(h); }
__host__ __device__ inline const int32_t* prb_handoff_idx(const unsigned char* h) { return reinterpret_cast<const int32_t*>(h + 256); }
__host__ __device__ inline const float* prb_handoff_prio(const unsigned char* h, uint32_t max_batch)
{
    return reinterpret_cast<const float*>(h + 256 + ((uint64_t)max_batch * 4 + 255) / 256 * 256);
}
inline uint64_t prb_handoff_bytes(uint32_t max_batch) { return 256 + 2 * (((uint64_t)max_batch * 4 + 255) / 256 * 256); }
// (the descents of B strata into `handoff`; uniform / buffer_norm as for prb_launch_sample)
int prb_launch_descend(const PrbView& v, uint32_t B, uint64_t seed, unsigned char* handoff, cudaStream_t s, int uniform = 0,
                       int buffer_norm = 0);
// (the rows named by `handoff` -- written by a prb_launch_descend that has completed -- to dst, the
// indices to d_idx, the weights with exponent beta to d_w)
// (early_reads: the kernel before this one on s writes no rows of the store -- it is a row copy of a sample
// too -- so this one may read rows while that one is still running)
int prb_launch_gather(const PrbView& v, uint32_t B, float beta, const unsigned char* handoff, int32_t* d_idx, float* d_w,
                      const PrbBatch& dst, cudaStream_t s, bool early_reads = false, int part = 0, uint32_t new_n = 0);
// (part 1 / part 2: the copy as two launches around the row copy of an insertion of new_n transitions whose tree
// work is done -- see the kernel; neither is a programmatic dependent)
// An empty kernel: a node that depends in full on what precedes it on s, for a programmatic dependent to hang on.
int prb_launch_relay(cudaStream_t s);
// true if a sample that writes these fields moves rows long enough for the bulk-copy ring
bool prb_sample_has_long_rows(const PrbView& v, const PrbBatch& dst);
// (stale > 0: skip entries that name one of the `stale` most recently written ring slots)
// (ins_n > 0, B within one sub-batch: the tree part of an insertion of ins_n transitions follows
// the update in the same kernel, which advances the tree's cursor and the fill count)
int prb_launch_update(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                      float alpha, float eps, cudaStream_t s, uint32_t stale = 0,
                      uint32_t ins_n = 0, const float* ins_prio = nullptr, const unsigned char* ins_done = nullptr);
// (ins_done: the done bytes of the inserted batch; read with the frame-deduplicated layout only)
// Update batches above this many entries (one per thread of a CTA) go to one launch of many
// co-resident CTAs instead (measured: 11-20 us for 16384 entries against 15-29 us for 4096 in one CTA);
// an update + insertion of short rows is then two launches, the update's and the insertion's.
constexpr uint32_t kPrbWideFrom = 1024;
// CTAs (one cluster) of the kernel that updates a batch (or sub-batch) of b entries
uint32_t prb_update_ctas(const PrbView& v, uint32_t b);
int prb_launch_get_priorities(const PrbView& v, uint32_t B, const int32_t* d_idx, float* d_out, cudaStream_t s);

// Per-device facts the launchers cache: SM count, and which kernels already have their large
// dynamic shared memory enabled (the attribute is per device).  One slot per device ordinal.
constexpr int kPrbMaxDevices = 64;
constexpr uint32_t kPrbTopFloats = 5120;     // 20 KB of shared memory
inline int prb_current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kPrbMaxDevices) return 0;
    return dev;
}
inline int prb_sm_count()
{
    static int cached[kPrbMaxDevices];
    const int dev = prb_current_device();
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// ---- device helpers -------------------------------------------------------------------
#ifdef __CUDACC__

// Left-to-right binary32 sum of the K children of one parent (children start at c, K-aligned).
// Loads bypass L1: other threads of this kernel may have written the children.
template <int K>
__device__ __forceinline__ float prb_sum_children(const float* c)
{
    if (K == 2) {
        float2 v = __ldcg(reinterpret_cast<const float2*>(c));
        return __fadd_rn(v.x, v.y);
    } else {
        float4 v = __ldcg(reinterpret_cast<const float4*>(c));
        float s = __fadd_rn(__fadd_rn(__fadd_rn(v.x, v.y), v.z), v.w);
#pragma unroll
        for (int q = 1; q < K / 4; ++q) {
            float4 u = __ldcg(reinterpret_cast<const float4*>(c) + q);
            s = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(s, u.x), u.y), u.z), u.w);
        }
        return s;
    }
}

__device__ __forceinline__ float prb_sum_children_dyn(const float* c, uint32_t K)
{
    switch (K) {
    case 2: return prb_sum_children<2>(c);
    case 4: return prb_sum_children<4>(c);
    case 8: return prb_sum_children<8>(c);
    case 16: return prb_sum_children<16>(c);
    default: return prb_sum_children<32>(c);
    }
}

// Both at once: x = the left-to-right binary32 sum of the K children at c, m = the smallest positive of the K
// values at cm (0 if none; cm == c where the children are the leaves, which serve both trees).  All loads are
// issued before anything is computed: one round trip through L2 for the two nodes, not two.
template <int K>
__device__ __forceinline__ void prb_sum_and_min(const float* c, const float* cm, float& x, float& m)
{
    unsigned best = 0xFFFFFFFFu;
    auto take = [&best](float u) { if (u > 0.0f) best = min(best, __float_as_uint(u)); };
    const bool own = cm != c;
    if (K == 2) {
        const float2 a = __ldcg(reinterpret_cast<const float2*>(c));
        float2 b = a;
        if (own) b = __ldcg(reinterpret_cast<const float2*>(cm));
        x = __fadd_rn(a.x, a.y);
        take(b.x); take(b.y);
    } else {
        constexpr int Q = K / 4 > 0 ? K / 4 : 1;
        x = 0.0f;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const float4 a = __ldcg(reinterpret_cast<const float4*>(c) + q);
            float4 b = a;
            if (own) b = __ldcg(reinterpret_cast<const float4*>(cm) + q);
            x = q ? __fadd_rn(x, a.x) : a.x;
            x = __fadd_rn(__fadd_rn(__fadd_rn(x, a.y), a.z), a.w);
            take(b.x); take(b.y); take(b.z); take(b.w);
        }
    }
    m = best == 0xFFFFFFFFu ? 0.0f : __uint_as_float(best);
}
__device__ __forceinline__ void prb_sum_and_min_dyn(const float* c, const float* cm, uint32_t K, float& x, float& m)
{
    switch (K) {
    case 2: prb_sum_and_min<2>(c, cm, x, m); break;
    case 4: prb_sum_and_min<4>(c, cm, x, m); break;
    case 8: prb_sum_and_min<8>(c, cm, x, m); break;
    case 16: prb_sum_and_min<16>(c, cm, x, m); break;
    default: prb_sum_and_min<32>(c, cm, x, m); break;
    }
}

// The smallest positive priority stored, for weights normalised over the whole buffer: the min-tree's root
// if the buffer keeps one, else what the scan launched before this kernel left in the state.
__device__ __forceinline__ float prb_buffer_pmin(const PrbView& v)
{
    if (v.min_off) return __ldcg(v.level[0] + v.min_off);
    return __uint_as_float((unsigned)v.state->pmin_bits);
}

// Runs CALL(frames, min_tree) with the two compile-time options of the tree-writing kernels that view v needs.
#define PRB_WITH_TREE_OPTIONS(v, CALL)                                              \
    do {                                                                            \
        if ((v).stack) { if ((v).min_off) { CALL(true, true); } else { CALL(true, false); } }   \
        else { if ((v).min_off) { CALL(false, true); } else { CALL(false, false); } }           \
    } while (0)

// The running maximum of written priorities: positive binary32 values order like their bit patterns.
__device__ __forceinline__ void prb_note_priorities(PrbState* st, float local_max, bool report)
{
    const unsigned m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(local_max));
    if (report && (threadIdx.x & 31u) == 0 && m) atomicMax(&st->max_prio_bits, m);
}
__device__ __forceinline__ float prb_default_priority(unsigned max_bits)
{
    return max_bits ? __uint_as_float(max_bits) : 1.0f;
}

__device__ __forceinline__ bool prb_valid_priority(float p)
{
    return (p >= 0.0f) && (p <= 3.402823466e+38f);   // false for NaN, negative, +Inf
}

// Contiguous copy of n 16-byte granules by all threads of the CTA (the bandwidth-critical path:
// one chunk of a long row).  Each thread issues up to U independent loads before its stores;
// consecutive threads touch consecutive granules.
template <int U>
__device__ __forceinline__ void prb_copy_span16(uint4* __restrict__ dst, const uint4* __restrict__ src, uint32_t n)
{
    const uint32_t stride = blockDim.x;
    for (uint32_t base = threadIdx.x; base < n; base += stride * U) {
        uint4 tmp[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (base + u * stride < n) tmp[u] = __ldcs(src + base + u * stride);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (base + u * stride < n) __stcs(dst + base + u * stride, tmp[u]);
    }
}

// Copy of short rows: granule e of [e_begin, e_end) is read from src[src_at(e)] and written to
// dst[dst_at(e)], by `nthreads` threads of which this one has rank `rank`.
template <typename T, typename SrcAt, typename DstAt>
__device__ __forceinline__ void prb_copy_mapped(T* __restrict__ dst, const T* __restrict__ src, uint32_t e_begin,
                                                uint32_t e_end, SrcAt src_at, DstAt dst_at, uint32_t rank,
                                                uint32_t nthreads)
{
    uint32_t e = e_begin + rank;
    for (; e + nthreads < e_end; e += 2 * nthreads) {
        const T a = src[src_at(e)], b = src[src_at(e + nthreads)];
        dst[dst_at(e)] = a;
        dst[dst_at(e + nthreads)] = b;
    }
    if (e < e_end) dst[dst_at(e)] = src[src_at(e)];
}

// A ticket: the calling thread adds 1 to *counter and gets the count before it; the CTA that draws the
// last one does a step's bookkeeping (normalises the weights, advances the cursor, bumps the call counter)
// from what the other CTAs wrote or read before they drew theirs.
// In the checked build the atomic carries release and acquire semantics at device scope, which is what the
// PTX memory model asks for.  In the ordinary build it is a relaxed atomic: measured, the acq_rel form costs
// 0.3-0.7 us per kernel (it drains the drawing thread's SM of outstanding memory operations, the bulk
// copies of the ring included; Atari-shaped sample 11.7 -> 12.4 us, MuJoCo-shaped step 14.6 -> 15.4 us).
// The relaxed form relies on this: every value another CTA reads was written by an atomic whose answer the
// writer waited for, or by a store followed by a CTA barrier and this atomic from the same SM, all of which
// are performed at L2 in the order issued; and every later reader uses ld.cg / atomics, which read L2.  The
// memory model does not promise that order for relaxed operations; the hardware keeps it.
__device__ __forceinline__ unsigned int prb_ticket(unsigned int* counter)
{
#ifdef PEARL_CHECKED
    unsigned int before;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(before) : "l"(counter) : "memory");
    return before;
#else
    return atomicAdd(counter, 1u);
#endif
}

// A kernel launched as a programmatic dependent waits here until the kernel before it on its stream has
// completed and its writes are visible; a no-op for a kernel launched the ordinary way.
__device__ __forceinline__ void prb_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- bulk asynchronous copies (TMA, non-tensor form, one destination each) ----------------------
// Long rows move global -> shared -> global as cp.async.bulk transfers.  Warp 0 of a CTA drives
// a ring of up to 32 stages in shared memory, ONE LANE PER STAGE: a lane issues the load of its
// chunk (completion on the stage's mbarrier), waits for it, issues the store (tracked by the
// lane's own bulk group) and, if it has another chunk, waits until the store has read the stage
// before loading again.  All stages of all SMs are in flight together, about 200 KB per SM,
// which registers cannot hold.  Addresses and sizes are multiples of 16 bytes (rows of 16-byte
// granules, 256-byte aligned bases).  Every row is read or written once and not touched again
// soon (a sampled batch is read once by the Learner, right after the call), so all these copies
// carry the L2 hint "evict first": a step's ~100 MB of rows then do not push the few megabytes of
// the tree out of L2, nor one another.

constexpr uint32_t kBulkSpinLimit = 1u << 20;   // mbarrier polls before a wait gives up

__device__ __forceinline__ uint32_t prb_smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

struct PrbBulkLane {
    uint32_t bar;        // shared address of this lane's mbarrier
    uint32_t buf;        // shared address of this lane's stage
    uint32_t parity;     // phase parity of the next load's completion
    bool busy;           // a store issued from the stage may still be reading it
    bool failed;         // a bounded wait ran out
    uint64_t stream_policy;   // L2 policy "evict first"

    __device__ __forceinline__ void init(void* bar_mem, void* buf_mem)
    {
        bar = prb_smem_addr(bar_mem); buf = prb_smem_addr(buf_mem);
        parity = 0; busy = false; failed = false;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(stream_policy));
    }
    // (a lane whose wait ran out moves nothing more: its remaining chunks are skipped, see store())
    __device__ __forceinline__ void load(const void* gsrc, uint32_t bytes)
    {
        if (failed) return;
        if (busy) { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); busy = false; }
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                     ::"r"(buf), "l"(gsrc), "r"(bytes), "r"(bar), "l"(stream_policy) : "memory");
    }
    __device__ __forceinline__ bool landed()
    {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        return ok != 0;
    }
    // Waits (bounded) for the load, then stores the stage to gdst.  The store is issued inside the
    // polling loop so that a lane whose data has landed does not wait for the other lanes.  If the
    // wait runs out the lane is marked failed: the phase parity stays as it is (the load is still
    // outstanding), nothing is stored from the stage, and every later load and store of the lane is
    // skipped; finish() then only waits, again with a limit, for what is in flight.
    // (gdst2 != nullptr: the stage is stored a second time, there, in the same bulk group)
    __device__ __forceinline__ void store(void* gdst, uint32_t bytes, void* gdst2 = nullptr)
    {
        if (failed) return;
        bool done = false;
        for (uint32_t spin = 0; spin < kBulkSpinLimit && !done; ++spin) {
            if (landed()) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                             ::"l"(gdst), "r"(buf), "r"(bytes), "l"(stream_policy) : "memory");
                if (gdst2 != nullptr)
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                                 ::"l"(gdst2), "r"(buf), "r"(bytes), "l"(stream_policy) : "memory");
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                done = true;
            }
        }
        if (done) { parity ^= 1u; busy = true; }
        else failed = true;
    }
    // Before the CTA exits: this lane's stores have read their stages (the writes themselves are
    // complete when the kernel is, like any other store); a failed lane gives its outstanding load
    // one more bounded wait, so that shared memory is not handed back under a copy still landing.
    __device__ __forceinline__ void finish()
    {
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        if (failed)
            for (uint32_t spin = 0; spin < kBulkSpinLimit && !landed(); ++spin) { }
    }
};

#endif  // __CUDACC__
