// Batched priority update (PEARL Section V-A, "priority update"; on the critical path after
// the Learner, Eq. 7).  The paper applies a change Delta along the root-leaf path under a
// mutex; here the leaf is SET and the ancestors are re-summed, so the result does not depend
// on scheduling (see prb_update_team in prb_tree.cuh for the steps).
//
// Up to 1024 entries (and every batch of changes): one CTA, or eight CTAs of one thread-block cluster
// that share the deep levels -- the work is a chain of dependent L2 round trips, one per level below
// the top of the tree, which is staged in shared memory.  More entries: one cooperative launch of
// many CTAs (prb_update_wide_kernel, below).
#include "prb_tree.cuh"

namespace {

// kFrames: the instance for the frame-deduplicated layout (markers, cleared leaves, stale history-less updates)
// kMin: the instance that maintains the min-tree beside the sum tree
template <bool kFrames, bool kMin>
__global__ void __launch_bounds__(1024)
prb_update_kernel(const __grid_constant__ PrbView v, uint32_t B, uint32_t n2, const int32_t* __restrict__ idx,
                  const float* __restrict__ val, int raw, float alpha, float eps, uint32_t stale,
                  uint32_t ins_n, const float* __restrict__ ins_prio, uint32_t ticket_total,
                  const unsigned char* __restrict__ ins_done)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned long long s_cursor, s_fill;
    // (a programmatic dependent behind this kernel may be made resident now; it waits for this kernel's
    // completion before it reads anything)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    PrbTeam team;
    team.rank = threadIdx.x;
    team.size = blockDim.x;
    team.whole_cta = true;
    team.part = blockIdx.x;          // CTAs of one cluster share the work (one CTA: the whole of it)
    team.parts = gridDim.x;
    if (kMin) team.min_off = v.min_off;
    PrbTop top;
    if (v.top_levels) top.mem = reinterpret_cast<float*>(smem + prb_update_smem_bytes(n2));
    if (kMin && v.top_levels) top.mem_min = top.mem + v.top_floats;
    if (team.part == 0) prb_top_begin(v, top, team.rank, team.size);
    unsigned long long fill, cursor = 0;
    unsigned int ticket_drawn = 0;
    PrbPreloaded pre = PrbPreloaded{false, false, 0, 0.0f, 0.0f};
    if (ins_n) {
        // with an insertion: cursor and fill are read once per CTA, before anything is published;
        // every thread fetches its first inputs meanwhile (beside the row copy each round trip is long)
        if (threadIdx.x < B) { pre.has_update = true; pre.idx = idx[threadIdx.x]; pre.val = val[threadIdx.x]; }
        if (threadIdx.x < ins_n && ins_prio != nullptr) { pre.has_prio = true; pre.prio = ins_prio[threadIdx.x]; }
        if (threadIdx.x == 0) { s_cursor = v.state->cursor; s_fill = v.state->fill; }
        __syncthreads();
        cursor = s_cursor;
        fill = s_fill;
        // (thread 0 draws the CTA's ticket now and looks at the answer after the tree work: it has an entry of
        // the batch like every other thread, and the team would wait for it at the first barrier of the sort)
        if (threadIdx.x == 0) ticket_drawn = prb_ticket(&v.state->insert_ticket);
    } else {
        fill = v.state->fill;
        if (stale || kFrames) cursor = v.state->cursor;
    }
    prb_update_team(v, team, B, n2, idx, val, raw, alpha, eps, fill, smem, ins_n, ins_prio, cursor, pre, stale, top, ins_done,
                    kFrames ? v.stack : 0u);
    if (ins_n && threadIdx.x == 0 && ticket_drawn == ticket_total - 1) prb_publish(v, ins_n, cursor, fill, kPrbPublishTree);
}

// ---- large batches: one launch of many CTAs ------------------------------------------------------
// A batch of more than one entry per thread of a CTA is updated by a grid of co-resident CTAs (a cooperative launch)
// whose phases are separated by a grid-wide barrier.  Nothing is sorted and no scratch is used:
//   1. every valid entry b raises the bits of its leaf to 0x80000000 | b with an atomic maximum --
//      a pattern above every valid priority (those are non-negative), so after the barrier the
//      leaf names the LAST valid entry of the batch that writes it;
//   2. the entry that finds its own number there stores its priority (last writer wins);
//   3. level by level, deepest first (fanouts 2 and 4: up to five and two levels per pass, a thread
//      re-summing a whole small subtree), the parents above the named leaves are re-summed from their
//      children, left to right in binary32: per entry (the first of consecutive entries with the same
//      parent) while a level has many more nodes than the batch has entries, the whole level once it
//      has not.  Re-summing a parent none of whose children changed gives back what it held, so
//      an entry that was refused for its priority may take part and duplicates only cost time;
//   4. CTA 0 stages the top of the tree in shared memory and re-sums it whole (prb_top_passes).
// The barrier's wait is bounded: a CTA that gives up raises PEARL_ST_INTERNAL and returns; the update
// is then incomplete (see PEARL_ST_INTERNAL in the header for what that leaves in the tree).
constexpr uint32_t kWideThreads = 256;
constexpr uint32_t kWideSpinLimit = 1u << 22;

struct PrbWideEntry {
    bool valid;
    uint32_t i;
    float p;
    unsigned flags;
};

__device__ __forceinline__ PrbWideEntry prb_wide_classify(const PrbView& v, int32_t i, float x, int raw, float alpha, float eps,
                                                          unsigned long long fill, uint64_t cursor, uint32_t stale)
{
    PrbWideEntry e = PrbWideEntry{false, 0u, 0.0f, 0u};
    const uint64_t N = v.capacity;
    if (i < 0 || (unsigned long long)i >= fill) { e.flags = PEARL_ST_BAD_INDEX; return e; }
    // one of the `stale` slots written most recently: overwritten since it was sampled
    if (stale && (cursor + N - 1 - (uint64_t)i) % N < stale) { e.flags = PEARL_ST_STALE; return e; }
    if (prb_history_less(v, cursor, (uint64_t)i, v.stack)) { e.flags = PEARL_ST_STALE; return e; }
    float p = x;
    const bool ok = raw ? prb_valid_priority(p) : prb_priority_pow(x, eps, alpha, p);
    if (!ok) { e.flags = PEARL_ST_BAD_PRIORITY; return e; }
    e.valid = true;
    e.i = (uint32_t)i;
    e.p = p;
    return e;
}

// Several levels in one pass, for small fanouts (a pass costs a grid barrier): node a of level lt and
// everything below it down to level lt + H - 1 are re-summed from the K^H entries of level lt + H
// under it (one contiguous run of at most 128 bytes), level by level in registers, every sum left to
// right as in a single-level pass.  Nodes past the end of a level are not written; entries past the end
// of the children's array count as zero.
template <int K, int H>
__device__ __forceinline__ void prb_resum_subtree(const PrbView& v, uint32_t lt, uint64_t a)
{
    constexpr int M = (K == 2) ? (1 << H) : (1 << (2 * H));      // K^H for K = 2, 4
    const uint32_t lb = lt + H - 1, D = v.depth, lg = v.log2_fanout;
    const float* ch = v.level[lb + 1];
    const uint64_t base = a * M, alloc = v.level_alloc[lb + 1];
    float c[M];
    if (K == 2 && base + M > alloc) {
        // (the run ends inside the children's array, whose length is a multiple of the fanout only)
#pragma unroll
        for (int q = 0; q < M / 2; ++q) {
            const float2 t = (base + 2 * q < alloc) ? __ldcg(reinterpret_cast<const float2*>(ch + base) + q) : make_float2(0.0f, 0.0f);
            c[2 * q] = t.x; c[2 * q + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int q = 0; q < M / 4; ++q) {
            const float4 t = (base + 4 * q < alloc) ? __ldcg(reinterpret_cast<const float4*>(ch + base) + q) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            c[4 * q] = t.x; c[4 * q + 1] = t.y; c[4 * q + 2] = t.z; c[4 * q + 3] = t.w;
        }
    }
#pragma unroll
    for (int s = 0; s < H; ++s) {
        const uint32_t m = lb - s;                                   // the level written in this step
        const int cnt = M >> ((s + 1) * (K == 2 ? 1 : 2));           // its nodes under a: K^(H-1-s)
        const uint64_t n_m = ((v.capacity - 1) >> (lg * (D - m))) + 1;
        const uint64_t first = a * cnt;
#pragma unroll
        for (int j = 0; j < M / K; ++j) {
            if (j < cnt) {
                float x = c[j * K];
#pragma unroll
                for (int t = 1; t < K; ++t) x = __fadd_rn(x, c[j * K + t]);
                if (first + j < n_m) v.level[m][first + j] = x;
                c[j] = x;
            }
        }
    }
}

// levels one pass takes when `left` levels are still to do: up to 32 entries under a node; with
// tens of thousands of batch entries only two levels (the wider subtrees' extra reads and scattered
// stores then cost more than the barriers they save: measured at 65536 entries)
__device__ __forceinline__ uint32_t prb_levels_per_pass(uint32_t K, uint32_t left, uint32_t B)
{
    const uint32_t most = (K == 2) ? (B > 16384u ? 2u : 5u) : (K == 4) ? 2u : 1u;
    return left < most ? left : most;      // (with a min-tree the caller takes one level per pass)
}

__device__ __forceinline__ void prb_resum_levels(const PrbView& v, uint32_t h, uint32_t lt, uint64_t a)
{
    if (v.fanout == 4) { prb_resum_subtree<4, 2>(v, lt, a); return; }
    switch (h) {
    case 2: prb_resum_subtree<2, 2>(v, lt, a); break;
    case 3: prb_resum_subtree<2, 3>(v, lt, a); break;
    case 4: prb_resum_subtree<2, 4>(v, lt, a); break;
    default: prb_resum_subtree<2, 5>(v, lt, a); break;
    }
}

// One parent of level lt from its K children (and the min-tree's node beside it, if there is one).
// (min_off: PrbView::min_off in the kernel instantiated for a buffer with a min-tree, the constant 0 in the other)
__device__ __forceinline__ void prb_wide_resum_one(const PrbView& v, uint32_t lt, uint64_t a, uint64_t min_off)
{
    const uint32_t K = v.fanout;
    const float* c = v.level[lt + 1] + a * K;
    if (min_off) {
        float x, m;
        prb_sum_and_min_dyn(c, c + (lt + 1 == v.depth ? 0 : min_off), K, x, m);
        v.level[lt][a] = x;
        (v.level[lt] + min_off)[a] = m;
    } else {
        v.level[lt][a] = prb_sum_children_dyn(c, K);
    }
}

// All CTAs of the (co-resident) grid meet; what any of them wrote to global memory before is
// visible, through L2, to all of them after.  `passed` counts the barriers this CTA has been through.
// Returns false if the wait ran out.
__device__ __forceinline__ bool prb_grid_barrier(PrbState* st, uint32_t& passed, uint32_t nctas, int* s_ok)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        // arrival with release semantics (the CTA's writes, ordered before it by the barrier above, are
        // visible to whoever then reads the counter with acquire semantics); no fence, no returned value
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(&st->wide_arrived) : "memory");
        const uint32_t target = (passed + 1u) * nctas;
        int ok = 1;
        for (uint32_t spins = 0;; ++spins) {
            uint32_t seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&st->wide_arrived) : "memory");
            if (seen >= target) break;
            if (spins >= kWideSpinLimit) { ok = 0; break; }
        }
        *s_ok = ok;
    }
    __syncthreads();
    ++passed;
    return *s_ok != 0;
}

template <bool kMin>
__global__ void __launch_bounds__(kWideThreads)
prb_update_wide_kernel(const __grid_constant__ PrbView v, uint32_t B, const int32_t* __restrict__ idx,
                       const float* __restrict__ val, int raw, float alpha, float eps, uint32_t stale)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned s_flags, s_maxbits;
    __shared__ int s_ok;
    const uint32_t tid = threadIdx.x, nctas = gridDim.x;
    const uint32_t gthreads = nctas * kWideThreads, gtid = blockIdx.x * kWideThreads + tid;
    const unsigned long long fill = v.state->fill;
    const uint64_t cursor = (stale || v.stack) ? v.state->cursor : 0ull;
    const uint32_t K = v.fanout, lg = v.log2_fanout, D = v.depth, T = v.top_levels;
    unsigned* leaf_bits = reinterpret_cast<unsigned*>(v.level[D]);
    if (tid == 0) { s_flags = 0u; s_maxbits = 0u; s_ok = (__ldcg(&v.state->wide_poisoned) == 0u) ? 1 : 0; }
    __syncthreads();
    if (!s_ok) {
        // an earlier launch of this kernel gave up at its barrier and left the counter (and the tree) in
        // no known state: no launch after it pretends otherwise
        if (tid == 0 && blockIdx.x == 0) atomicOr(&v.state->status, PEARL_ST_INTERNAL);
        return;
    }

    // 1. validate, transform, name the last writer of every leaf (a thread's first entry stays in registers)
    PrbWideEntry first = PrbWideEntry{false, 0u, 0.0f, 0u};
    unsigned flags = 0u;
    float wmax = 0.0f;
    for (uint32_t b = gtid; b < B; b += gthreads) {
        const PrbWideEntry e = prb_wide_classify(v, idx[b], val[b], raw, alpha, eps, fill, cursor, stale);
        if (b == gtid) first = e;
        flags |= e.flags;
        if (e.valid && PRB_IN_BOUNDS(v, e.i < v.level_alloc[D])) { wmax = fmaxf(wmax, e.p); atomicMax(leaf_bits + e.i, 0x80000000u | b); }
    }
    flags = __reduce_or_sync(0xFFFFFFFFu, flags);
    const unsigned mbits = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(wmax));
    if ((tid & 31u) == 0) {
        if (flags) atomicOr(&s_flags, flags);
        if (mbits) atomicMax(&s_maxbits, mbits);
    }
    __syncthreads();
    if (tid == 0) {
        if (s_flags) atomicOr(&v.state->status, s_flags);
        if (s_maxbits) atomicMax(&v.state->max_prio_bits, s_maxbits);
    }
    uint32_t passed = 0;
    bool alive = prb_grid_barrier(v.state, passed, nctas, &s_ok);

    // 2. the named entry writes the leaf
    if (alive) {
        for (uint32_t b = gtid; b < B; b += gthreads) {
            const PrbWideEntry e = (b == gtid) ? first : prb_wide_classify(v, idx[b], val[b], raw, alpha, eps, fill, cursor, stale);
            if (e.valid && PRB_IN_BOUNDS(v, e.i < v.level_alloc[D]) && __ldcg(leaf_bits + e.i) == (0x80000000u | b)) v.level[D][e.i] = e.p;
        }
        alive = prb_grid_barrier(v.state, passed, nctas, &s_ok);
    }

    // 3. the levels below the staged top, deepest first; small fanouts take several levels per pass
    for (int l = (int)D - 1; alive && l >= (int)T;) {
        const uint32_t h = kMin ? 1u : prb_levels_per_pass(K, (uint32_t)l - T + 1u, B);
        const uint32_t lt = (uint32_t)l - h + 1u;                 // the highest level this pass writes
        const uint32_t sh = lg * (D - lt);
        const uint64_t n_lt = ((v.capacity - 1) >> sh) + 1;       // nodes of level lt
        if (n_lt <= 2ull * B) {
            for (uint64_t a = gtid; a < n_lt; a += gthreads) {
                if (!PRB_IN_BOUNDS(v, a < v.level_alloc[lt] && (h > 1 || a * K + K <= v.level_alloc[lt + 1]))) continue;
                if (h == 1) prb_wide_resum_one(v, lt, a, kMin ? v.min_off : 0ull);
                else prb_resum_levels(v, h, lt, a);
            }
        } else {
            for (uint32_t b = gtid; b < B; b += gthreads) {
                const int32_t i = idx[b];
                if (i < 0 || (unsigned long long)i >= fill) continue;
                const uint64_t a = (uint64_t)i >> sh;
                if (b > 0) {
                    const int32_t before = idx[b - 1];
                    if (before >= 0 && (unsigned long long)before < fill && ((uint64_t)before >> sh) == a) continue;
                }
                if (!PRB_IN_BOUNDS(v, a < v.level_alloc[lt] && (h > 1 || a * K + K <= v.level_alloc[lt + 1]))) continue;
                if (h == 1) prb_wide_resum_one(v, lt, a, kMin ? v.min_off : 0ull);
                else prb_resum_levels(v, h, lt, a);
            }
        }
        alive = prb_grid_barrier(v.state, passed, nctas, &s_ok);
        l -= (int)h;
    }
    if (!alive) {
        // (the barrier's counter is left as it is, and marked: see wide_poisoned)
        if (tid == 0) { atomicOr(&v.state->status, PEARL_ST_INTERNAL); atomicExch(&v.state->wide_poisoned, 1u); }
        return;
    }
    // every CTA is past its last barrier: the last one to say so clears the barrier for the next launch
    if (tid == 0 && atomicAdd(&v.state->wide_done, 1u) == nctas - 1) {
        v.state->wide_arrived = 0u;
        v.state->wide_done = 0u;
    }
    // 4. the staged levels
    if (blockIdx.x == 0 && T > 0) {
        PrbTop top;
        top.mem = reinterpret_cast<float*>(smem);
        if (kMin) top.mem_min = top.mem + v.top_floats;
        prb_top_begin(v, top, tid, kWideThreads);
        prb_top_wait();
        __syncthreads();
        PrbTeam team;
        team.rank = tid;
        team.size = kWideThreads;
        team.whole_cta = true;
        if (kMin) team.min_off = v.min_off;
        prb_top_passes(v, top, team, T);
    }
}

// Priority retrieval: one thread per entry.
__global__ void prb_get_priorities_kernel(const __grid_constant__ PrbView v, uint32_t B, const int32_t* __restrict__ idx,
                                          float* __restrict__ out)
{
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int32_t i = idx[b];
    if (i < 0 || (unsigned long long)i >= v.state->fill) { out[b] = 0.0f; atomicOr(&v.state->status, PEARL_ST_BAD_INDEX); return; }
    out[b] = PRB_IN_BOUNDS(v, (uint32_t)i < v.level_alloc[v.depth]) ? __ldcg(v.level[v.depth] + i) : 0.0f;
}

}  // namespace

int prb_launch_get_priorities(const PrbView& v, uint32_t B, const int32_t* d_idx, float* d_out, cudaStream_t s)
{
    prb_get_priorities_kernel<<<(B + 255) / 256, 256, 0, s>>>(v, B, d_idx, d_out);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

uint32_t prb_update_ctas(const PrbView& v, uint32_t b)
{
    // Many wide child groups per level (fanout 32, hundreds of entries) are more L2 misses than
    // one SM keeps in flight: then eight CTAs of one cluster share each level.
    return (v.fanout * b >= 8192u) ? 8u : 1u;
}

// The many-CTA update of a large batch: 1 launch, or 0 if this device cannot run it (no cooperative
// launch), or -1 on a launch error.
static int prb_launch_update_wide(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                                  float alpha, float eps, cudaStream_t s, uint32_t stale)
{
    static int ctas_per_sm[kPrbMaxDevices];      // 0: not asked yet, -1: not available
    const int dev = prb_current_device();
    const size_t smem = (size_t)kPrbTopFloats * sizeof(float) * 2;     // (room for a min-tree's staged levels too)
    if (ctas_per_sm[dev] == 0) {
        int coop = 0, nb = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, prb_update_wide_kernel<true>, (int)kWideThreads, smem) != cudaSuccess || nb < 1) {
            cudaGetLastError();
            ctas_per_sm[dev] = -1;
        } else {
            ctas_per_sm[dev] = nb > 2 ? 2 : nb;
        }
    }
    if (ctas_per_sm[dev] < 0) return 0;
    uint32_t grid = (B + kWideThreads - 1) / kWideThreads;
    const uint32_t room = (uint32_t)(prb_sm_count() * ctas_per_sm[dev]);
    if (grid > room) grid = room;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kWideThreads);
    cfg.dynamicSmemBytes = (size_t)v.top_floats * sizeof(float) * (v.min_off ? 2 : 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = v.min_off ? cudaLaunchKernelEx(&cfg, prb_update_wide_kernel<true>, v, B, d_idx, d_val, raw, alpha, eps, stale)
                                    : cudaLaunchKernelEx(&cfg, prb_update_wide_kernel<false>, v, B, d_idx, d_val, raw, alpha, eps, stale);
    return e == cudaSuccess ? 1 : -1;
}

int prb_launch_update(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                      float alpha, float eps, cudaStream_t s, uint32_t stale,
                      uint32_t ins_n, const float* ins_prio, const unsigned char* ins_done)
{
    if (ins_n && B > PEARL_UPDATE_SUBBATCH) return -1;
    // a batch of more than one entry per thread of a CTA: one launch of many CTAs (values or TD errors;
    // changes keep their batch order and go sub-batch by sub-batch below)
    if (B > kPrbWideFrom && raw != 2 && ins_n == 0 && B < 0x80000000u) {
        const int k = prb_launch_update_wide(v, B, d_idx, d_val, raw, alpha, eps, s, stale);
        if (k != 0) return k;
    }
    static bool big_smem[kPrbMaxDevices];
    const int dev = prb_current_device();
    if (!big_smem[dev]) {
        const int most = (int)(prb_update_smem_bytes(PEARL_UPDATE_SUBBATCH) + 2 * kPrbTopFloats * sizeof(float));
        if (cudaFuncSetAttribute(prb_update_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(prb_update_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(prb_update_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(prb_update_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess)
            return -1;
        big_smem[dev] = true;
    }
    // A batch beyond one CTA's reach goes sub-batch by sub-batch in batch order: every launch leaves
    // a consistent tree and later entries overwrite earlier ones, as in the whole batch.
    int launches = 0;
    for (uint32_t first = 0; first < B; first += PEARL_UPDATE_SUBBATCH) {
        const uint32_t b = B - first < PEARL_UPDATE_SUBBATCH ? B - first : PEARL_UPDATE_SUBBATCH;
        const uint32_t n2 = prb_update_n2(b);
        const uint32_t threads = n2 < 64 ? 64 : (n2 > 1024 ? 1024 : n2);
        const uint32_t ctas = prb_update_ctas(v, b);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(ctas);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = prb_update_smem_bytes(n2) + v.top_floats * sizeof(float) * (v.min_off ? 2 : 1);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = ctas;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaSuccess;
#define PRB_LAUNCH_UPDATE_AS(FF, MM) \
    e = cudaLaunchKernelEx(&cfg, prb_update_kernel<FF, MM>, v, b, n2, d_idx + first, d_val + first, raw, alpha, eps, stale, ins_n, ins_prio, ctas, ins_done)
        PRB_WITH_TREE_OPTIONS(v, PRB_LAUNCH_UPDATE_AS);
#undef PRB_LAUNCH_UPDATE_AS
        if (e != cudaSuccess) return -1;
        ++launches;
    }
    return launches;
}
