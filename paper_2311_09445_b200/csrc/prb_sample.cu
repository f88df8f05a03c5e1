// Stratified priority sampling, importance-sampling weights and the gather of the sampled
// transitions, in one kernel.
//
// Priority sampling is Eq. 1 of PEARL (Section II-A) carried out as Section V-A describes it:
// "traversing the tree performing prefix sum from root to leaf".  A group of K lanes (K = the
// fanout) owns one stratum: lane j loads child j, so a child group is one 8..128-byte request;
// the children are put in shared memory (the staged levels are there already), every lane reads
// all K and forms the left-to-right binary32 prefix sums in registers (the same association as
// the stored parent), lane j keeping prefix j; a ballot counts the prefixes the binary64 target
// has passed, and that count is the child to enter.  The top levels of the tree (up to 20 KB) are
// staged in shared memory at kernel start, the rest is read from L2, the leaves ahead of time
// while the level above them is on its way.  The read of the sampled
// rows is Listing 2's `D_storage[sampled_indices]`.  Stratification, the Philox stream and the
// weights follow the prioritized-replay reference the paper cites (Schaul et al.).
//
// Work split: the batch is cut into tasks (a stratum, or one <= 8 KB chunk of one long row of
// a stratum) and every CTA of a grid that fits the GPU in one wave takes a contiguous range of
// tasks.  A CTA first walks the tree for the strata its tasks touch (a stratum shared by two
// CTAs is walked by both: L2 reads only), then splits by role: threads 0..127 copy, threads
// 128..255 turn leaf priorities into raw weights.  So the chain of dependent tree reads is paid
// once, and from then on all SMs stream rows.  Long rows (Atari-shaped) move as bulk
// asynchronous copies global -> shared -> global driven by warp 0, one lane per stage of a
// ~200 KB ring, one CTA per SM, so that nearly the whole read set of a batch is in flight at
// once; short rows are copied through registers.  Raw weights go to scratch; the CTA that is
// last to finish its descents normalises them by the batch maximum and bumps the call counter
// while the others are already copying.  No CTA ever waits on another.
#include "prb_descend.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 2;
constexpr uint32_t kChunk = 512;             // upper bound on granules per row chunk (8 KB)
constexpr uint32_t kRowMode = 512;           // rows of at least this many 16-byte granules are split into chunks
constexpr uint32_t kFrameRowMode = 64;       // ... frames of the frame-deduplicated layout from this many granules on
constexpr uint32_t kTopFloats = 5120;        // tree entries staged in shared memory (20 KB) ...
constexpr uint32_t kTopFloats32 = 1152;      // ... at fanout 32 only levels 1 and 2 can fit: 4.5 KB
__host__ __device__ constexpr uint32_t top_floats_of(uint32_t K) { return K == 32 ? kTopFloats32 : kTopFloats; }
constexpr uint32_t kRingBytes = 198 * 1024;  // bulk-copy ring of a long-row CTA (dynamic shared memory), <= 32 stages
constexpr uint32_t kRingBarBytes = 1024;     // room for the ring's mbarriers in front of its buffers

struct SamplePlan {
    uint32_t tps;                            // tasks per stratum (1 unless some field is in row mode)
    uint32_t n_tasks;                        // tasks of this launch: a whole number of strata ...
    uint32_t first_task;                     // ... starting with this task of the batch (sub-batch launches; else 0)
    uint32_t ticket_total;                   // CTAs of all launches of the call: the last of them normalises the weights
    uint32_t task_first[PRB_NUM_FIELDS];     // row mode: tasks [task_first, task_first + chunks) of a stratum
    uint32_t chunks[PRB_NUM_FIELDS];         //   copy the chunks of field f; 0 = short rows, copied flat
    uint32_t chunk[PRB_NUM_FIELDS];          // granules per chunk
    uint32_t ring_stages, ring_stage_bytes;  // bulk-copy ring (long rows only; 0 stages otherwise)
    uint32_t uniform;                        // 1: uniform replay (no tree walk): index = floor(u * fill)
    uint32_t buffer_norm;                    // 1: weights divided by the largest weight over the buffer (state->pmin_bits), not the batch
    uint32_t top_levels;                     // levels 1 .. top_levels are staged in shared memory
    uint32_t top_vec4;                       // 16-byte units staged, from the start of level 1
    uint32_t top_off[PRB_MAX_LEVELS];        // offset (floats) of a staged level from the start of level 1
    // leaf prefetch (when the level above the leaves is read from global memory): the first pf_groups
    // lane groups of a CTA own K*K floats each at byte pf_off of the dynamic shared memory
    uint32_t pf_groups, pf_off;
    // frame-deduplicated layout with frames long enough for the ring: the tasks of field F_OBS are
    // (stack + 1) frames (0 .. stack steps back from the sampled slot) of frame_chunks chunks each
    uint32_t frame_chunks;
};

// The K children of one node lie in shared memory at `row`: every lane of the group reads all of them
// (the same addresses: broadcasts) and forms the left-to-right binary32 prefix sums in registers, one
// chain of K-1 additions; lane j keeps child j and the prefix that ends with it.  (Passing the
// children from lane to lane by shuffles instead puts a shuffle's latency into every step of the chain.)
template <int K>
__device__ __forceinline__ void group_prefix(const float* row, uint32_t lane, float& c, float& acc)
{
    if (K == 2) {
        const float2 v = *reinterpret_cast<const float2*>(row);
        c = lane ? v.y : v.x;
        acc = lane ? __fadd_rn(v.x, v.y) : v.x;
    } else {
        float run = 0.0f;
#pragma unroll
        for (int q = 0; q < K / 4; ++q) {
            const float4 v = reinterpret_cast<const float4*>(row)[q];
            const float e[4] = { v.x, v.y, v.z, v.w };
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int i = 4 * q + t;
                run = (i == 0) ? e[t] : __fadd_rn(run, e[t]);
                if ((int)lane == i) { c = e[t]; acc = run; }
            }
        }
    }
}

// Walks one stratum's target x from the root to a leaf; lane j of the group looks after child j.
// s_child: K floats of shared memory of the group's own, for a level that comes from global memory.
// pf != nullptr: while the group's K nodes of the level above the leaves come from global memory,
// the K*K leaves below them are copied to pf (asynchronously, 16 bytes at a time), so that the last
// level costs no second round trip: its K leaves are read from there.
template <int K>
__device__ __forceinline__ void descend(const PrbView& v, const SamplePlan& plan, const float* s_top, float* s_child, double x,
                                        uint32_t lane, uint32_t& leaf, float& p_leaf, unsigned& flags, float* pf)
{
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const unsigned gshift = (K == 32) ? 0u : ((threadIdx.x & 31u) / K) * K;
    const unsigned gmask = (K == 32) ? FULL : ((1u << (K & 31)) - 1u);
    uint64_t g = 0;
    float c = 0.0f, acc = 0.0f;
    int j = 0;
    for (uint32_t l = 1; l <= v.depth; ++l) {
        const float* row;
        if (!PRB_IN_BOUNDS(v, g * K + K <= v.level_alloc[l])) { flags |= PEARL_ST_INTERNAL; g = 0; }
        if (l <= plan.top_levels) {
            row = s_top + plan.top_off[l] + (uint32_t)g * K;
        } else if (pf != nullptr && l == v.depth) {
            asm volatile("cp.async.wait_all;" ::: "memory");
            __syncwarp();
            row = pf + (uint32_t)j * K;
        } else {
            const float mine = __ldg(v.level[l] + g * K + lane);
            if (pf != nullptr && l + 1 == v.depth) {
                // the leaves under this group's K nodes: K*K/4 units of 16 bytes, dealt over the K lanes
                // (fanout 2: one unit); units past the end of the leaf level are left out
                const float* span = v.level[v.depth] + g * (K * K);
                const uint64_t left = v.level_alloc[v.depth] - g * (K * K);        // entries from the span's start to the end
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(pf);
                constexpr uint32_t kUnits = K * K / 4;
#pragma unroll
                for (uint32_t q = lane; q < kUnits; q += K)
                    if ((uint64_t)q * 4u < left)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + q * 16u), "l"(span + q * 4u) : "memory");
            }
            __syncwarp();              // (the group has read what the level before left in s_child)
            s_child[lane] = mine;
            __syncwarp();
            row = s_child;
        }
        group_prefix<K>(row, lane, c, acc);
        const unsigned passed = (__ballot_sync(FULL, x >= (double)acc) >> gshift) & gmask;
        const unsigned positive = (__ballot_sync(FULL, c > 0.0f) >> gshift) & gmask;
        const int cnt = __popc(passed);
        if (cnt < K) {
            j = cnt;
        } else {
            flags |= PEARL_ST_CLAMPED;
            if (positive) j = 31 - __clz(positive);
            else { j = 0; flags |= PEARL_ST_INTERNAL; }
        }
        const float sprev = __shfl_sync(FULL, acc, j > 0 ? j - 1 : 0, K);
        if (j > 0) x = __dsub_rn(x, (double)sprev);
        g = g * K + (uint64_t)j;
    }
    p_leaf = __shfl_sync(FULL, c, j, K);
    leaf = (uint32_t)g;
}

__device__ __forceinline__ uint4 load_granule(const unsigned char* base, uint64_t g, uint32_t vec)
{
    uint4 r = make_uint4(0u, 0u, 0u, 0u);
    switch (vec) {
    case 16: r = reinterpret_cast<const uint4*>(base)[g]; break;
    case 8: { const uint2 t = reinterpret_cast<const uint2*>(base)[g]; r.x = t.x; r.y = t.y; break; }
    case 4: r.x = reinterpret_cast<const uint32_t*>(base)[g]; break;
    case 2: r.x = reinterpret_cast<const uint16_t*>(base)[g]; break;
    default: r.x = base[g]; break;
    }
    return r;
}

__device__ __forceinline__ void store_granule(unsigned char* base, uint64_t g, uint32_t vec, const uint4& r)
{
    switch (vec) {
    case 16: reinterpret_cast<uint4*>(base)[g] = r; break;
    case 8: reinterpret_cast<uint2*>(base)[g] = make_uint2(r.x, r.y); break;
    case 4: reinterpret_cast<uint32_t*>(base)[g] = r.x; break;
    case 2: reinterpret_cast<uint16_t*>(base)[g] = (uint16_t)r.x; break;
    default: base[g] = (unsigned char)r.x; break;
    }
}

// Short rows of strata [k_first, k_first + n_rows): every short field of the batch, granule by
// granule, by `nthreads` threads.  s_idx[r] is the leaf of stratum k_first + r.  The first two
// granules per thread of ALL fields are loaded before anything is stored, so a small batch costs
// one round trip instead of one per field; what is left goes field by field.
// Frame-deduplicated layout: frame `back` steps back from slot `leaf`, no further back than `clamp` (the
// distance to the episode's first frame): the slot that holds it.
__device__ __forceinline__ uint64_t prb_frame_slot(const PrbView& v, uint32_t leaf, uint32_t back, uint32_t clamp)
{
    const uint64_t b = back < clamp ? back : clamp;
    return ((uint64_t)leaf + v.capacity - b) % v.capacity;
}

// ... and the two observations of strata [k_first, k_first + n_rows) rebuilt granule by granule (short frames):
// position pos (0 = oldest) of next_obs is the frame stack-1-pos steps back, of obs the frame stack-pos steps back.
__device__ __forceinline__ void gather_short_frames(const PrbView& v, const PrbBatch& dst, uint32_t k_first, uint32_t n_rows,
                                                    const uint32_t* s_idx, const uint32_t* s_clamp, uint32_t rank, uint32_t nthreads,
                                                    uint32_t S)
{
    const uint32_t vec = v.field_vec[F_OBS], W = v.field_bytes[F_OBS] / vec, total = n_rows * S * W;
    for (int f = F_OBS; f <= F_NEXT_OBS; ++f) {
        if (dst.ptr[f] == nullptr) continue;
        const uint64_t dbase = (uint64_t)k_first * S * W;
        for (uint32_t e = rank; e < total; e += nthreads) {
            const uint32_t r = e / (S * W), rem = e - r * S * W, pos = rem / W, off = rem - pos * W;
            const uint32_t back = (f == F_NEXT_OBS) ? S - 1 - pos : S - pos;
            const uint64_t slot = prb_frame_slot(v, s_idx[r], back, s_clamp[r]);
            store_granule(dst.ptr[f], dbase + e, vec, load_granule(v.store[F_OBS], slot * W + off, vec));
        }
    }
}

__device__ __forceinline__ void gather_short_fields(const PrbView& v, const SamplePlan& plan, const PrbBatch& dst,
                                                    uint32_t k_first, uint32_t n_rows, const uint32_t* s_idx,
                                                    uint32_t rank, uint32_t nthreads, const uint32_t* s_clamp = nullptr,
                                                    uint32_t stack = 0)
{
    // (stack: PrbView::stack in the kernel instantiated for the frame layout, the constant 0 elsewhere)
    if (stack && plan.frame_chunks == 0) gather_short_frames(v, dst, k_first, n_rows, s_idx, s_clamp, rank, nthreads, stack);
    uint4 tmp[PRB_NUM_FIELDS][2];
#pragma unroll
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0 || plan.chunks[f] != 0 || (stack && f == F_OBS)) continue;
        const uint32_t vec = v.field_vec[f], W = v.field_bytes[f] / vec, Wp = v.field_pitch[f] / vec, total = n_rows * W;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint32_t e = rank + u * nthreads;
            if (e < total) {
                const uint32_t r = (W == 1) ? e : e / W;
                if (PRB_IN_BOUNDS(v, s_idx[r] < v.capacity))
                    tmp[f][u] = load_granule(v.store[f], (uint64_t)s_idx[r] * Wp + (e - r * W), vec);
            }
        }
    }
#pragma unroll
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0 || plan.chunks[f] != 0 || (stack && f == F_OBS)) continue;
        const uint32_t vec = v.field_vec[f], W = v.field_bytes[f] / vec, Wp = v.field_pitch[f] / vec, total = n_rows * W;
        const uint64_t dbase = (uint64_t)k_first * W;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint32_t e = rank + u * nthreads;
            if (e < total) store_granule(dst.ptr[f], dbase + e, vec, tmp[f][u]);
        }
        for (uint32_t e = rank + 2 * nthreads; e < total; e += nthreads) {     // the rest of a larger batch
            const uint32_t r = e / W;
            if (PRB_IN_BOUNDS(v, s_idx[r] < v.capacity))
                store_granule(dst.ptr[f], dbase + e, vec, load_granule(v.store[f], (uint64_t)s_idx[r] * Wp + (e - r * W), vec));
        }
    }
}

// kFrames: the instance for the frame-deduplicated layout (it rebuilds both observations from single frames)
template <int K, bool kFrames>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
prb_sample_kernel(const __grid_constant__ PrbView v, uint32_t B, float beta, uint64_t seed,
                  int32_t* __restrict__ out_idx, float* __restrict__ out_w, const __grid_constant__ PrbBatch dst,
                  const __grid_constant__ SamplePlan plan)
{
    constexpr uint32_t R = kThreads / K;          // strata walked concurrently by one CTA
    __shared__ __align__(16) float s_top[top_floats_of(K)];
    __shared__ __align__(16) float s_child[kThreads];     // K floats per lane group: a level that came from global memory
    __shared__ uint32_t s_idx[R];
    __shared__ double s_wmax[kThreads / 2 / 32];          // the last CTA's maximum of the raw weights, per warp
    __shared__ volatile unsigned long long s_seen[R];     // answers of the atomics that publish the weights
    __shared__ float s_p[R];
    __shared__ unsigned s_flags[R];
    __shared__ uint32_t s_clamp[R];                        // frame-deduplicated layout: how far back a stratum's frames reach
    __shared__ unsigned int s_last;
    extern __shared__ __align__(128) unsigned char s_ring[];   // long rows: mbarriers, then the ring buffers

    const uint32_t tid = threadIdx.x;
    const uint32_t stack = kFrames ? v.stack : 0u;
    const bool bulk = plan.ring_stages > 0;
    PrbBulkLane ring;            // lanes 0 .. ring_stages-1 of warp 0 own one stage each
    const bool ring_lane = bulk && tid < plan.ring_stages;
    if (ring_lane) ring.init(s_ring + 8u * tid, s_ring + kRingBarBytes + tid * plan.ring_stage_bytes);
    // (launched as a programmatic dependent of the kernel before it on the stream: up to here it may have run
    // beside that kernel; nothing has been read or written yet)
    prb_dep_wait();
    // every thread reads the state it needs itself (same addresses: one request per warp), so the
    // targets can be formed while the staged levels are still on their way
    const unsigned long long calls = v.state->sample_calls;
    const unsigned long long fill = v.state->fill;
    const float total32 = __ldg(v.level[0]);
    const float pmin = plan.buffer_norm ? prb_buffer_pmin(v) : 0.0f;
    {
        // stage the top levels: one contiguous run of the slab starting at level 1, 16 bytes at a time
        const float4* src = reinterpret_cast<const float4*>(v.level[1]);
        constexpr uint32_t kPerThread = (top_floats_of(K) / 4 + kThreads - 1) / kThreads;
        float4 t[kPerThread];
#pragma unroll
        for (uint32_t u = 0; u < kPerThread; ++u)
            if (tid + u * kThreads < plan.top_vec4) t[u] = __ldg(src + tid + u * kThreads);
#pragma unroll
        for (uint32_t u = 0; u < kPerThread; ++u)
            if (tid + u * kThreads < plan.top_vec4) reinterpret_cast<float4*>(s_top)[tid + u * kThreads] = t[u];
    }
    const bool empty = (fill == 0) || (!plan.uniform && !(total32 > 0.0f));

    // this CTA's tasks and the strata they touch
    const uint32_t tps = plan.tps;
    const uint32_t t_lo = plan.first_task + (uint32_t)(((uint64_t)blockIdx.x * plan.n_tasks) / gridDim.x);
    const uint32_t t_hi = plan.first_task + (uint32_t)(((uint64_t)(blockIdx.x + 1) * plan.n_tasks) / gridDim.x);
    const uint32_t k_lo = t_lo / tps;
    const uint32_t k_hi = (t_hi + tps - 1) / tps;
    const uint32_t k_own = (t_lo + tps - 1) / tps;       // strata whose first task is here: this CTA writes their idx / weight
    const uint32_t n_rounds = (empty || t_hi <= t_lo) ? 0u : (k_hi - k_lo + R - 1) / R;

    for (uint32_t round = 0; round < max(n_rounds, 1u); ++round) {      // one pass even with nothing to do: the ticket
        const uint32_t kb = k_lo + round * R;
        uint32_t n_round = 0;
        // ---- targets: stratum k of the batch draws x_k ----
        const uint32_t gi = tid / K, lane = tid % K;
        bool walks = false;
        uint32_t k = 0, r0 = 0;
        double x = 0.0;
        const double total = (double)total32;
        if (round < n_rounds) {
            n_round = min(R, k_hi - kb);
            walks = (tid / 32u) * (32u / K) < n_round;   // warp-uniform: whole warps take part in the shuffles
            if (walks) {
                k = min(kb + gi, B - 1);                  // surplus groups repeat a valid stratum and write nothing
                const double seg = __ddiv_rn(total, (double)B);
                r0 = philox4x32_10_word0(k, 0u, (uint32_t)calls, (uint32_t)(calls >> 32),
                                                        (uint32_t)seed, (uint32_t)(seed >> 32));
                const double u = __dmul_rn((double)r0, 2.3283064365386963e-10);     // * 2^-32, exact
                x = __dmul_rn(__dadd_rn((double)k, u), seg);
                if (x >= total) x = __longlong_as_double(__double_as_longlong(total) - 1);   // next binary64 below total
            }
        }
        if (round == 0) __syncthreads();                  // the staged levels are in shared memory
        if (round < n_rounds) {
            // ---- descents: one K-lane group per stratum ----
            if (walks) {
                uint32_t leaf; float p; unsigned flags = 0;
                if (plan.uniform) { leaf = (uint32_t)(((unsigned long long)r0 * fill) >> 32); p = 1.0f; }   // floor(u * fill)
                else descend<K>(v, plan, s_top, s_child + (tid - lane), x, lane, leaf, p, flags,
                                gi < plan.pf_groups ? reinterpret_cast<float*>(s_ring + plan.pf_off) + gi * (K * K) : nullptr);
                if (lane == 0 && gi < n_round) {
                    s_idx[gi] = leaf; s_p[gi] = p; s_flags[gi] = flags;
                    if (stack) {
                        // frames: the distance back to the episode's first frame -- the nearest marker among the
                        // `stack` slots before this one (or slot 0 while the ring has not wrapped)
                        unsigned marks = 0;
                        for (uint32_t d = 1; d <= stack; ++d)
                            marks |= (unsigned)((v.store[F_DONE][((uint64_t)leaf + v.capacity - d) % v.capacity] & kPrbEpisodeStart) ? 1u : 0u) << d;
                        uint32_t c = stack;
                        for (uint32_t d = stack; d >= 1; --d) {
                            if (fill < v.capacity && leaf < d) c = d - 1;
                            else if ((marks >> d) & 1u) c = d;
                        }
                        s_clamp[gi] = c;
                    }
                }
            }
            __syncthreads();
        }

        // From here the CTA splits by role: threads 0..127 copy, threads 128..255 look after the weights.
        const bool last_descents = round + 1 >= n_rounds;      // true exactly once per CTA
        if (tid >= kThreads / 2) {
            // raw weights, indices and flags of the strata this CTA owns (off the copy's critical path).
            // What another CTA reads -- the raw weights -- is written by atomics whose results are
            // waited for, so that the values are on their way to L2 at once; the barrier below and the
            // ticket's release/acquire pair (one thread's, not a fence in every thread, which was
            // measured to wait for the bulk copies the ring has in flight) order them before the reads
            // of the CTA that draws the last ticket.
            const uint32_t gi2 = tid - kThreads / 2;
            if (gi2 < n_round) {
                if (kb + gi2 >= k_own) {
                    const uint32_t k2 = kb + gi2;
                    // (one call site for the power: with the buffer-wide divisor the loop runs twice)
                    double base = __ddiv_rn(__dmul_rn((double)fill, (double)s_p[gi2]), total);
                    double wr = 1.0, wmax = 1.0;
#pragma unroll 1
                    for (uint32_t q = 0; q < 1u + plan.buffer_norm; ++q) {
                        const double r = plan.uniform ? 1.0 : pow(base, -(double)beta);
                        if (q == 0) wr = r; else wmax = r;
                        base = __ddiv_rn(__dmul_rn((double)fill, (double)pmin), total);     // the buffer's smallest positive priority
                    }
                    out_idx[k2] = (int32_t)s_idx[gi2];
                    if (plan.buffer_norm) {
                        if (out_w != nullptr) out_w[k2] = (float)__ddiv_rn(wr, wmax);
                    } else {
                        // (the old value goes to shared memory: a store that cannot issue before the atomic has answered)
                        s_seen[gi2] = atomicExch(reinterpret_cast<unsigned long long*>(v.wraw + k2),
                                                 (unsigned long long)__double_as_longlong(wr));
                    }
                    if (s_flags[gi2]) atomicOr(&v.state->status, s_flags[gi2]);
                }
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kThreads / 2) : "memory");
            if (tid == kThreads / 2 && last_descents) {
                // every descent of this CTA is done and its weights are in L2: the last CTA to get
                // here normalises the weights of the whole batch
                s_last = (prb_ticket(&v.state->sample_ticket) == plan.ticket_total - 1) ? 1u : 0u;
            }
            if (last_descents) {
                asm volatile("bar.sync 2, %0;" ::"n"(kThreads / 2) : "memory");
                if (s_last) {
                    if (empty) {
                        if (tid == kThreads / 2) atomicOr(&v.state->status, PEARL_ST_EMPTY);
                    } else if (out_w != nullptr && !plan.buffer_norm) {
                        // the batch maximum, then the division: the first raw weights of every thread stay in registers
                        constexpr uint32_t kHalf = kThreads / 2, kHeld = 4;
                        const uint32_t j = tid - kHalf;
                        double held[kHeld];
                        double m = 0.0;
#pragma unroll
                        for (uint32_t u = 0; u < kHeld; ++u) {
                            const uint32_t k = j + u * kHalf;
                            held[u] = k < B ? __ldcg(v.wraw + k) : 0.0;
                            m = fmax(m, held[u]);
                        }
                        for (uint32_t k = j + kHeld * kHalf; k < B; k += kHalf) m = fmax(m, __ldcg(v.wraw + k));
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
                        if ((tid & 31u) == 0) s_wmax[(tid - kHalf) >> 5] = m;
                        asm volatile("bar.sync 2, %0;" ::"n"(kThreads / 2) : "memory");
                        double wmax = s_wmax[0];
#pragma unroll
                        for (uint32_t q = 1; q < kHalf / 32; ++q) wmax = fmax(wmax, s_wmax[q]);
#pragma unroll
                        for (uint32_t u = 0; u < kHeld; ++u) {
                            const uint32_t k = j + u * kHalf;
                            if (k < B) out_w[k] = (float)__ddiv_rn(held[u], wmax);
                        }
                        for (uint32_t k = j + kHeld * kHalf; k < B; k += kHalf)
                            out_w[k] = (float)__ddiv_rn(__ldcg(v.wraw + k), wmax);
                    }
                    asm volatile("bar.sync 2, %0;" ::"n"(kThreads / 2) : "memory");
                    if (tid == kThreads / 2) {
                        if (!empty) v.state->sample_calls = calls + 1;
                        if (plan.buffer_norm) v.state->pmin_bits = ~0ull;      // (ready for the next scan)
                        v.state->sample_ticket = 0u;
                    }
                }
            }
        } else if (round < n_rounds) {
            // ---- gather: Data Storage rows of this round's strata ----
            if (ring_lane) {
                // long rows: this CTA's tasks of the round, one chunk each; lane s takes tasks a+s, a+s+S, ...
                const uint32_t a = max(t_lo, kb * tps), b = min(t_hi, (kb + n_round) * tps);
                for (uint32_t t = a + tid; t < b; t += plan.ring_stages) {
                    const uint32_t k = t / tps, r = t - k * tps;
                    int f = 0;
                    while (plan.chunks[f] == 0 || r >= plan.task_first[f] + plan.chunks[f]) ++f;
                    const uint32_t W = v.field_bytes[f] / 16u;
                    if constexpr (kFrames) { if (plan.frame_chunks) {
                        // one chunk of the frame `back` steps back: it is a part of next_obs (position stack-1-back)
                        // and of obs (position stack-back): one load, up to two stores
                        const uint32_t S = stack, in = r - plan.task_first[f], back = in / plan.frame_chunks;
                        const uint32_t e0 = (in - back * plan.frame_chunks) * plan.chunk[f];
                        const uint32_t bytes = min(W - e0, plan.chunk[f]) * 16u;
                        if (!PRB_IN_BOUNDS(v, s_idx[k - kb] < v.capacity && k < B && back <= S && e0 < W && bytes <= plan.ring_stage_bytes)) continue;
                        unsigned char* to_next = (back < S && dst.ptr[F_NEXT_OBS]) ? dst.ptr[F_NEXT_OBS] + (((uint64_t)k * S + (S - 1 - back)) * W + e0) * 16u : nullptr;
                        unsigned char* to_obs = (back >= 1 && dst.ptr[F_OBS]) ? dst.ptr[F_OBS] + (((uint64_t)k * S + (S - back)) * W + e0) * 16u : nullptr;
                        if (to_next == nullptr && to_obs == nullptr) continue;
                        ring.load(v.store[F_OBS] + (prb_frame_slot(v, s_idx[k - kb], back, s_clamp[k - kb]) * W + e0) * 16u, bytes);
                        ring.store(to_next ? to_next : to_obs, bytes, to_next ? to_obs : nullptr);
                        continue;
                    } }
                    const uint32_t e0 = (r - plan.task_first[f]) * plan.chunk[f];
                    const uint32_t bytes = min(W - e0, plan.chunk[f]) * 16u;
                    if (!PRB_IN_BOUNDS(v, s_idx[k - kb] < v.capacity && k < B && e0 < W && bytes <= plan.ring_stage_bytes)) continue;
                    ring.load(v.store[f] + ((uint64_t)s_idx[k - kb] * W + e0) * 16u, bytes);
                    ring.store(dst.ptr[f] + ((uint64_t)k * W + e0) * 16u, bytes);
                }
            }
            // short rows: copied by the stratum's owner through registers (warp 0 drives the ring when there is one)
            const uint32_t k_flat = max(kb, k_own);
            if (k_flat < kb + n_round && (!bulk || tid >= 32)) {
                const uint32_t rank = bulk ? tid - 32u : tid, nthreads = bulk ? kThreads / 2 - 32u : kThreads / 2;
                gather_short_fields(v, plan, dst, k_flat, kb + n_round - k_flat, s_idx + (k_flat - kb), rank, nthreads, s_clamp + (k_flat - kb), stack);
            }
        }
        __syncthreads();        // s_idx is rewritten by the next round
    }
    if (ring_lane) {
        ring.finish();
        if (ring.failed) atomicOr(&v.state->status, PEARL_ST_INTERNAL);
    }
}

// ---- large batches of short rows: one stratum per thread -------------------------------------------
// With thousands of strata the K-lane groups above keep too few tree reads in flight (a CTA walks
// 256 / K strata at a time, round after round).  Here every thread walks a stratum of its own: it
// loads the K children of its node itself (one 8..128-byte group: whole sectors), forms the same
// left-to-right binary32 prefix sums one after another and enters the first child whose prefix
// exceeds the binary64 target -- the count of prefixes the target has passed, as the lanes' ballot
// gives it.  A CTA takes a contiguous range of strata, 256 at a time: targets, descents, index and raw
// weight per thread; then all its threads copy the rows, granule by granule (consecutive threads,
// consecutive granules), up to sixteen loads in flight each.  Every CTA raises the batch's largest raw
// weight with one atomic maximum (positive binary64 values order like their bit patterns); a second,
// small launch divides all raw weights by it.
constexpr uint32_t kWideSampleFrom = 2048;      // batches of at least this many strata (short rows)
constexpr uint32_t kWideSampleStrata = 32;      // ... spread over CTAs of at least this many strata

// Short rows of strata [k_first, k_first + n_rows) by all `nthreads` threads, field by field, in
// granules of type T: up to U granules per thread are loaded before the first is stored.
template <typename T, int U>
__device__ __forceinline__ void gather_field_deep(const T* __restrict__ store, T* __restrict__ out, uint32_t W, uint32_t Wp, uint32_t total,
                                                  const uint32_t* s_idx, uint32_t rank, uint32_t nthreads)
{
    for (uint32_t e0 = rank; e0 < total; e0 += nthreads * U) {
        T tmp[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t e = e0 + u * nthreads;
            if (e < total) {
                const uint32_t r = (W == 1) ? e : e / W;
                tmp[u] = store[(uint64_t)s_idx[r] * Wp + (e - r * W)];     // (s_idx comes from a descent, checked there; Wp: granules per slot)
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t e = e0 + u * nthreads;
            if (e < total) out[e] = tmp[u];
        }
    }
}

__device__ __forceinline__ void gather_short_fields_deep(const PrbView& v, const PrbBatch& dst, uint32_t k_first, uint32_t n_rows,
                                                         const uint32_t* s_idx, uint32_t rank, uint32_t nthreads)
{
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0) continue;
        const uint32_t vec = v.field_vec[f], W = v.field_bytes[f] / vec, Wp = v.field_pitch[f] / vec, total = n_rows * W;
        const unsigned char* src = v.store[f];
        unsigned char* out = dst.ptr[f] + (uint64_t)k_first * v.field_bytes[f];
        switch (vec) {
        case 16: gather_field_deep<uint4, 4>(reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(out), W, Wp, total, s_idx, rank, nthreads); break;
        case 8: gather_field_deep<uint2, 8>(reinterpret_cast<const uint2*>(src), reinterpret_cast<uint2*>(out), W, Wp, total, s_idx, rank, nthreads); break;
        case 4: gather_field_deep<uint32_t, 16>(reinterpret_cast<const uint32_t*>(src), reinterpret_cast<uint32_t*>(out), W, Wp, total, s_idx, rank, nthreads); break;
        case 2: gather_field_deep<uint16_t, 8>(reinterpret_cast<const uint16_t*>(src), reinterpret_cast<uint16_t*>(out), W, Wp, total, s_idx, rank, nthreads); break;
        default: gather_field_deep<unsigned char, 8>(src, out, W, Wp, total, s_idx, rank, nthreads); break;
        }
    }
}

template <int K>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
prb_sample_wide_kernel(const __grid_constant__ PrbView v, uint32_t B, float beta, uint64_t seed,
                       int32_t* __restrict__ out_idx, float* __restrict__ out_w, const __grid_constant__ PrbBatch dst,
                       const __grid_constant__ SamplePlan plan)
{
    __shared__ __align__(16) float s_top[top_floats_of(K)];
    __shared__ uint32_t s_idx[kThreads];
    __shared__ unsigned long long s_wmax;
    __shared__ unsigned s_flags;
    __shared__ unsigned int s_last;
    const uint32_t tid = threadIdx.x;
    const unsigned long long calls = v.state->sample_calls;
    const unsigned long long fill = v.state->fill;
    const float total32 = __ldg(v.level[0]);
    {
        const float4* src = reinterpret_cast<const float4*>(v.level[1]);
        for (uint32_t q = tid; q < plan.top_vec4; q += kThreads) reinterpret_cast<float4*>(s_top)[q] = __ldg(src + q);
    }
    if (tid == 0) { s_wmax = 0ull; s_flags = 0u; }
    const bool empty = (fill == 0) || !(total32 > 0.0f);
    const double total = (double)total32;
    const uint32_t k_lo = (uint32_t)(((uint64_t)blockIdx.x * B) / gridDim.x);
    const uint32_t k_hi = (uint32_t)(((uint64_t)(blockIdx.x + 1) * B) / gridDim.x);
    __syncthreads();
    unsigned long long my_wmax = 0ull;
    unsigned my_flags = 0u;
    for (uint32_t kb = k_lo; kb < k_hi && !empty; kb += kThreads) {
        const uint32_t k = kb + tid, n_here = min(kThreads, k_hi - kb);
        if (k < k_hi) {
            // target of stratum k (Eq. 1's x, one per equal segment of the total), then the walk
            const double x = prb_stratum_target(k, B, total, calls, seed);
            uint32_t leaf; float p;
            prb_descend_alone<K>(v, plan.top_levels, plan.top_off, s_top, x, leaf, p, my_flags);
            s_idx[tid] = leaf;
            out_idx[k] = (int32_t)leaf;
            if (out_w != nullptr) {
                const double wr = pow(__ddiv_rn(__dmul_rn((double)fill, (double)p), total), -(double)beta);
                v.wraw[k] = wr;
                my_wmax = max(my_wmax, (unsigned long long)__double_as_longlong(wr));
            }
        }
        __syncthreads();
        gather_short_fields_deep(v, dst, kb, n_here, s_idx, tid, kThreads);
        __syncthreads();            // s_idx is rewritten by the next pass
    }
    if (my_wmax) atomicMax(&s_wmax, my_wmax);
    if (my_flags) atomicOr(&s_flags, my_flags);
    __syncthreads();
    if (tid == 0) {
        if (s_flags) atomicOr(&v.state->status, s_flags);
        if (s_wmax) atomicMax(&v.state->wide_wmax_bits, s_wmax);
        s_last = (prb_ticket(&v.state->sample_ticket) == gridDim.x - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (tid == 0 && s_last) {
        // the last CTA to finish: the call's bookkeeping (the weights are divided by a launch of their own)
        if (empty) atomicOr(&v.state->status, PEARL_ST_EMPTY);
        else v.state->sample_calls = calls + 1;
        v.state->sample_ticket = 0u;
    }
}

// Second launch of a large-batch sample: w_k = raw weight / the batch's largest, by as many CTAs as
// it takes (one CTA would need B / 1024 dependent round trips).  The largest raw weight is zero only
// if the buffer was empty: then nothing is written.  The last CTA to have read it clears it.
__global__ void __launch_bounds__(kThreads)
prb_normalise_weights_kernel(const __grid_constant__ PrbView v, uint32_t B, float* __restrict__ out_w)
{
    const unsigned long long bits = __ldcg(&v.state->wide_wmax_bits);
    if (bits) {
        const double wmax = __longlong_as_double((long long)bits);
        const uint32_t k0 = blockIdx.x * kThreads * 4u + threadIdx.x;
        double held[4];
#pragma unroll
        for (uint32_t u = 0; u < 4; ++u) if (k0 + u * kThreads < B) held[u] = __ldcg(v.wraw + k0 + u * kThreads);
#pragma unroll
        for (uint32_t u = 0; u < 4; ++u) if (k0 + u * kThreads < B) out_w[k0 + u * kThreads] = (float)__ddiv_rn(held[u], wmax);
    }
    __syncthreads();        // every thread of the CTA has read the maximum
    if (threadIdx.x == 0 && prb_ticket(&v.state->sample_ticket) == gridDim.x - 1) {
        v.state->wide_wmax_bits = 0ull;
        v.state->sample_ticket = 0u;
    }
}

// The smallest positive leaf among the `fill` stored ones, into state->pmin_bits (all ones at creation and
// again after every sample that used it): positive binary32 values order like their bit patterns.
__global__ void prb_leaf_min_kernel(const __grid_constant__ PrbView v)
{
    const unsigned long long fill = v.state->fill;
    const float* leaves = v.level[v.depth];
    unsigned best = 0xFFFFFFFFu;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < fill;
         i += (unsigned long long)gridDim.x * blockDim.x) {
        const float p = __ldg(leaves + i);
        if (p > 0.0f) best = min(best, __float_as_uint(p));
    }
    __shared__ unsigned s_best[8];
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    if ((threadIdx.x & 31u) == 0) s_best[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (unsigned w = 1; w < blockDim.x / 32u; ++w) best = min(best, s_best[w]);
        if (best != 0xFFFFFFFFu) atomicMin(&v.state->pmin_bits, (unsigned long long)best);      // one atomic per CTA
    }
}

// ---- a sample of long rows as two kernels ------------------------------------------------------------------
// In a captured sequence of calls (a step that is replayed many times) the descents of a sample of long
// rows run as a kernel of their own on the handle's second stream, where they can overlap whatever the
// caller's stream is still copying, and the indexed row copy follows on the caller's stream.
//
// prb_descend_kernel<K>: targets and descents only, a lane group per stratum as in prb_sample_kernel, a grid
// of at most one CTA per SM (it has to fit beside the CTAs of a row copy).  Lane 0 of a group stores the
// leaf's index and priority in the hand-off area; the last CTA to finish (ticket) writes the header,
// bumps the call counter and raises EMPTY if there was nothing to sample.  No weights here: the power
// and the chain that finds their maximum are the longer half of a small sample, and nothing of the row
// copy waits for them.
template <int K>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
prb_descend_kernel(const __grid_constant__ PrbView v, uint32_t B, uint64_t seed, unsigned char* __restrict__ handoff,
                   const __grid_constant__ SamplePlan plan)
{
    constexpr uint32_t R = kThreads / K;
    __shared__ __align__(16) float s_top[top_floats_of(K)];
    __shared__ __align__(16) float s_child[kThreads];
    __shared__ unsigned long long s_calls;
    extern __shared__ __align__(128) unsigned char s_pf[];      // leaf prefetch: K*K floats per walking group
    const uint32_t tid = threadIdx.x;
    const unsigned long long calls = v.state->sample_calls;
    const unsigned long long fill = v.state->fill;
    const float total32 = __ldg(v.level[0]);
    {
        const float4* src = reinterpret_cast<const float4*>(v.level[1]);
        constexpr uint32_t kPerThread = (top_floats_of(K) / 4 + kThreads - 1) / kThreads;
        float4 t[kPerThread];
#pragma unroll
        for (uint32_t u = 0; u < kPerThread; ++u)
            if (tid + u * kThreads < plan.top_vec4) t[u] = __ldg(src + tid + u * kThreads);
#pragma unroll
        for (uint32_t u = 0; u < kPerThread; ++u)
            if (tid + u * kThreads < plan.top_vec4) reinterpret_cast<float4*>(s_top)[tid + u * kThreads] = t[u];
    }
    if (tid == 0) s_calls = calls;        // (the value is in hand before this CTA's ticket below: the last CTA may then move the counter)
    const bool empty = (fill == 0) || (!plan.uniform && !(total32 > 0.0f));
    const double total = (double)total32;
    int32_t* out_idx = const_cast<int32_t*>(prb_handoff_idx(handoff));
    float* out_p = const_cast<float*>(prb_handoff_prio(handoff, v.max_batch));
    const uint32_t k_lo = (uint32_t)(((uint64_t)blockIdx.x * B) / gridDim.x);
    const uint32_t k_hi = (uint32_t)(((uint64_t)(blockIdx.x + 1) * B) / gridDim.x);
    const uint32_t gi = tid / K, lane = tid % K;
    __syncthreads();
    for (uint32_t kb = k_lo; kb < k_hi && !empty; kb += R) {
        const uint32_t n_round = min(R, k_hi - kb);
        if ((tid / 32u) * (32u / K) < n_round) {              // warp-uniform: whole warps take part in the shuffles
            const uint32_t k = min(kb + gi, B - 1);          // surplus groups repeat a valid stratum and write nothing
            uint32_t leaf; float p; unsigned flags = 0;
            if (plan.uniform) {
                const uint32_t r0 = philox4x32_10_word0(k, 0u, (uint32_t)calls, (uint32_t)(calls >> 32), (uint32_t)seed, (uint32_t)(seed >> 32));
                leaf = (uint32_t)(((unsigned long long)r0 * fill) >> 32);
                p = 1.0f;
            } else {
                descend<K>(v, plan, s_top, s_child + (tid - lane), prb_stratum_target(k, B, total, calls, seed), lane, leaf, p, flags,
                           gi < plan.pf_groups ? reinterpret_cast<float*>(s_pf) + gi * (K * K) : nullptr);
            }
            if (lane == 0 && gi < n_round) {
                out_idx[kb + gi] = (int32_t)leaf;
                out_p[kb + gi] = p;
                if (flags) atomicOr(&v.state->status, flags);
            }
        }
        __syncthreads();        // (a group's scratch and prefetch buffer are reused by the next round)
    }
    if (tid == 0 && prb_ticket(&v.state->sample_ticket) == gridDim.x - 1) {
        PrbHandoffHeader* hd = reinterpret_cast<PrbHandoffHeader*>(handoff);
        hd->found = empty ? 0u : 1u;
        hd->buffer_norm = plan.buffer_norm;
        hd->fill = fill;
        hd->total = total32;
        hd->pmin = plan.buffer_norm ? prb_buffer_pmin(v) : 0.0f;
        if (empty) atomicOr(&v.state->status, PEARL_ST_EMPTY);
        else v.state->sample_calls = s_calls + 1;
        if (plan.buffer_norm) v.state->pmin_bits = ~0ull;      // (ready for the next scan)
        v.state->sample_ticket = 0u;
    }
}

// prb_gather_rows_kernel: the indexed copy, one CTA per SM.  Warp 0 drives the bulk-copy ring (a lane's first
// load goes out one L2 read -- its row's index -- after the kernel starts); four more warps look after the
// strata whose first chunk the CTA holds: the index, the short fields, and the importance-sampling weight
//   w_k = (fill p_k / total)^-beta / max_j (fill p_j / total)^-beta = (p_k / p_min)^-beta
// where p_min is the smallest priority of the batch (every CTA scans the B priorities in the hand-off area
// for it: the power does not increase with p), or the smallest priority stored when the weights are
// normalised over the buffer.  The task numbering is that of prb_sample_kernel.
constexpr uint32_t kGatherRingBytes = 198 * 1024;      // the row copy's ring
constexpr int kGatherWorkers = 128;
constexpr int kGatherThreads = 32 + kGatherWorkers;

//
// kPart: 0, the whole copy.  1 and 2, the copy in two launches around an insertion of new_n transitions whose
// priorities are in the tree (so the descents may have drawn them) and whose rows are not yet in the store:
// launch 1 moves the long rows of every stratum that drew none of the new slots -- the new_n slots before the
// published cursor -- and launch 2, once the new rows are stored, the long rows of the others and everything
// else (indices, weights, short fields).
template <int kPart>
__global__ void __launch_bounds__(kGatherThreads, 1)
prb_gather_rows_kernel(const __grid_constant__ PrbView v, uint32_t B, float beta, const unsigned char* __restrict__ handoff,
                       int32_t* __restrict__ out_idx, float* __restrict__ out_w, const __grid_constant__ PrbBatch dst,
                       const __grid_constant__ SamplePlan plan, uint32_t early_reads, uint32_t new_n)
{
    extern __shared__ __align__(128) unsigned char s_ring[];
    __shared__ uint32_t s_idx[kGatherWorkers];
    __shared__ unsigned s_pmin[kGatherWorkers / 32];
    const uint32_t tid = threadIdx.x;
    // Programmatic dependent launch, both ways.  As a primary: the kernel after this one on the stream may
    // be scheduled as soon as every CTA here has said so, i.e. at once -- its CTAs then take over SMs one by
    // one as CTAs of this kernel leave, instead of after the last of them.  As a secondary: this kernel may
    // itself have started while the kernel before it on the stream was still running.  Nothing is stored
    // before that kernel has completed (prb_dep_wait below: its writes, to the same output arrays perhaps,
    // come first), and no row is read before then either, unless the host knows that kernel to be a row
    // copy like this one, which writes no rows of the store (early_reads): then a CTA's whole read phase
    // runs under the tail of the copy before it.  The hand-off area was written by a kernel this one
    // depends on in full.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int32_t* pre_idx = prb_handoff_idx(handoff);
    const uint32_t tps = plan.tps;
    const uint32_t t_lo = (uint32_t)(((uint64_t)blockIdx.x * plan.n_tasks) / gridDim.x);
    const uint32_t t_hi = (uint32_t)(((uint64_t)(blockIdx.x + 1) * plan.n_tasks) / gridDim.x);
    if (tid < plan.ring_stages) {
        PrbBulkLane ring;
        uint32_t t = t_lo + tid;
        // (the index of the lane's first row is asked for before anything else)
        int32_t leaf = t < t_hi ? __ldcg(pre_idx + t / tps) : 0;
        ring.init(s_ring + 8u * tid, s_ring + kRingBarBytes + tid * plan.ring_stage_bytes);
        if (__ldcg(&prb_handoff_header(handoff)->found) == 0u) return;          // the buffer was empty: nothing is written
        bool waited = false;
        if (!early_reads) { prb_dep_wait(); waited = true; }
        uint64_t new_lo = 0;
        if (kPart) {
            const uint64_t cursor = __ldcg(&v.state->cursor);
            new_lo = cursor >= new_n ? cursor - new_n : cursor + v.capacity - new_n;
        }
        while (t < t_hi) {
            const uint32_t k = t / tps, r = t - k * tps;
            int f = 0;
            while (plan.chunks[f] == 0 || r >= plan.task_first[f] + plan.chunks[f]) ++f;
            const uint32_t W = v.field_bytes[f] / 16u;
            const uint32_t e0 = (r - plan.task_first[f]) * plan.chunk[f];
            const uint32_t bytes = min(W - e0, plan.chunk[f]) * 16u;
            bool inside = PRB_IN_BOUNDS(v, (uint32_t)leaf < v.capacity && k < B && e0 < W && bytes <= plan.ring_stage_bytes);
            if (kPart) {
                const uint64_t i = (uint32_t)leaf;
                const bool is_new = (i >= new_lo ? i - new_lo : i + v.capacity - new_lo) < new_n;
                inside = inside && (is_new == (kPart == 2));
            }
            if (inside) ring.load(v.store[f] + ((uint64_t)(uint32_t)leaf * W + e0) * 16u, bytes);
            const uint32_t t_next = t + plan.ring_stages;
            const int32_t leaf_next = t_next < t_hi ? __ldcg(pre_idx + t_next / tps) : 0;
            if (!waited) { prb_dep_wait(); waited = true; }
            if (inside) ring.store(dst.ptr[f] + ((uint64_t)k * W + e0) * 16u, bytes);
            t = t_next;
            leaf = leaf_next;
        }
        ring.finish();
        if (ring.failed) atomicOr(&v.state->status, PEARL_ST_INTERNAL);
    } else if (tid >= 32 && kPart != 1) {
        const uint32_t rank = tid - 32u;
        const uint32_t k_own = (t_lo + tps - 1) / tps, k_end = (t_hi + tps - 1) / tps;
        const PrbHandoffHeader* hd = prb_handoff_header(handoff);
        if (__ldcg(&hd->found) == 0u) return;
        const float* pre_p = prb_handoff_prio(handoff, v.max_batch);
        const bool weights = out_w != nullptr && k_own < k_end;
        float pmin = 0.0f;
        if (weights) {
            pmin = __ldcg(&hd->pmin);
            if (__ldcg(&hd->buffer_norm) == 0u) {
                unsigned best = 0xFFFFFFFFu;     // (priorities are not negative: they order like their bits)
                for (uint32_t k = rank; k < B; k += kGatherWorkers) best = min(best, __float_as_uint(__ldcg(pre_p + k)));
                best = __reduce_min_sync(0xFFFFFFFFu, best);
                if ((rank & 31u) == 0) s_pmin[rank >> 5] = best;
                asm volatile("bar.sync 1, %0;" ::"n"(kGatherWorkers) : "memory");
#pragma unroll
                for (int q = 0; q < kGatherWorkers / 32; ++q) best = min(best, s_pmin[q]);
                pmin = __uint_as_float(best);
            }
        }
        prb_dep_wait();
        for (uint32_t kb = k_own; kb < k_end; kb += kGatherWorkers) {
            const uint32_t n_here = min((uint32_t)kGatherWorkers, k_end - kb);
            const bool mine = rank < n_here;
            float p = 1.0f;
            if (mine) {
                const int32_t leaf = __ldcg(pre_idx + kb + rank);
                s_idx[rank] = (uint32_t)leaf;
                out_idx[kb + rank] = leaf;
                if (weights) p = __ldcg(pre_p + kb + rank);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kGatherWorkers) : "memory");
            gather_short_fields(v, plan, dst, kb, n_here, s_idx, rank, kGatherWorkers);
            // (fill p / total)^-beta / (fill pmin / total)^-beta as one power, (p / pmin)^-beta: the same number to a
            // few units of the binary64 rounding error, exactly 1 where p is the smallest, and half the arithmetic
            if (weights && mine) out_w[kb + rank] = (float)pow(__ddiv_rn((double)p, (double)pmin), -(double)beta);
            asm volatile("bar.sync 1, %0;" ::"n"(kGatherWorkers) : "memory");
        }
    }
}

__global__ void prb_relay_kernel() {}

}  // namespace

int prb_launch_relay(cudaStream_t s)
{
    prb_relay_kernel<<<1, 32, 0, s>>>();
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// The row-mode part of a plan: which fields move as chunks of long rows, and how they are cut.
static bool plan_row_mode(const PrbView& v, const PrbBatch& dst, SamplePlan& plan)
{
    plan.tps = 0;
    plan.frame_chunks = 0;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        plan.task_first[f] = 0;
        plan.chunks[f] = 0;
        plan.chunk[f] = 0;
        if (v.stack && f == F_OBS) {
            // frames of at least 1 KB go through the ring, a frame at a time (stack + 1 frames per stratum serve
            // both observations); shorter ones are rebuilt granule by granule
            const uint32_t W = v.field_bytes[f] / v.field_vec[f];
            if ((dst.ptr[F_OBS] != nullptr || dst.ptr[F_NEXT_OBS] != nullptr) && v.field_vec[f] == 16 && W >= kFrameRowMode) {
                plan.frame_chunks = (W + kChunk - 1) / kChunk;
                plan.chunk[f] = (W + plan.frame_chunks - 1) / plan.frame_chunks;
                plan.chunks[f] = (v.stack + 1) * plan.frame_chunks;
                plan.task_first[f] = plan.tps;
                plan.tps += plan.chunks[f];
            }
            continue;
        }
        if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0) continue;
        const uint32_t W = v.field_bytes[f] / v.field_vec[f];
        if (v.field_vec[f] == 16 && W >= kRowMode) {
            plan.task_first[f] = plan.tps;
            plan.chunks[f] = (W + kChunk - 1) / kChunk;
            plan.chunk[f] = (W + plan.chunks[f] - 1) / plan.chunks[f];
            plan.tps += plan.chunks[f];
        }
    }
    const bool row_mode = plan.tps > 0;
    if (!row_mode) plan.tps = 1;
    return row_mode;
}

// The top levels a sample kernel stages in shared memory (levels 1 .. top_levels, while they fit; the
// levels lie one after another in the slab, each start 256-byte aligned), into the plan.
static void plan_staged_top(const PrbView& v, bool uniform, SamplePlan& plan)
{
    plan.top_levels = 0;
    plan.top_vec4 = 0;
    for (uint32_t l = 0; l < PRB_MAX_LEVELS; ++l) plan.top_off[l] = 0;
    for (uint32_t l = 1; l <= v.depth && !uniform; ++l) {
        const uint64_t off = (uint64_t)(v.level[l] - v.level[1]);
        if (off + v.level_alloc[l] > top_floats_of(v.fanout)) break;
        plan.top_off[l] = (uint32_t)off;
        plan.top_vec4 = (uint32_t)((off + v.level_alloc[l] + 3) / 4);
        plan.top_levels = l;
    }
}

bool prb_sample_has_long_rows(const PrbView& v, const PrbBatch& dst)
{
    SamplePlan plan;
    return v.stack == 0 && plan_row_mode(v, dst, plan);      // (rebuilt observations: the one-kernel sample only)
}

int prb_launch_sample(const PrbView& v, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w,
                      const PrbBatch& dst, cudaStream_t s, int uniform, uint32_t n_sub, const PrbSubStreams* subs, int buffer_norm)
{
    if (n_sub < 1 || n_sub > kPrbMaxSubBatches || n_sub > B || (n_sub > 1 && subs == nullptr)) return -1;
    const int sm_count = prb_sm_count();
    const int dev = prb_current_device();
    SamplePlan plan;
    const bool row_mode = plan_row_mode(v, dst, plan);
    plan.n_tasks = B * plan.tps;
    plan.first_task = 0;
    plan.ticket_total = 0;
    // levels 1 .. top_levels staged in shared memory while they fit
    // (the levels lie one after another in the slab, each start 256-byte aligned)
    plan.uniform = uniform ? 1u : 0u;
    plan.buffer_norm = (buffer_norm && !uniform) ? 1u : 0u;
    plan_staged_top(v, uniform != 0, plan);
    const uint32_t R = kThreads / v.fanout;
    const int ki = v.log2_fanout;
    if (!row_mode && n_sub == 1 && !uniform && !buffer_norm && B >= kWideSampleFrom && v.stack == 0) {
        // a large batch of short rows: one stratum per thread
        uint32_t grid = (B + kWideSampleStrata - 1) / kWideSampleStrata;
        const uint32_t one_wave = (uint32_t)sm_count * kCtasPerSm;
        if (grid > one_wave) grid = one_wave;
        plan.ring_stages = 0; plan.ring_stage_bytes = 0; plan.pf_groups = 0; plan.pf_off = 0;
        plan.ticket_total = grid;
        switch (v.fanout) {
        case 2: prb_sample_wide_kernel<2><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
        case 4: prb_sample_wide_kernel<4><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
        case 8: prb_sample_wide_kernel<8><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
        case 16: prb_sample_wide_kernel<16><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
        default: prb_sample_wide_kernel<32><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
        }
        if (d_w != nullptr) prb_normalise_weights_kernel<<<(B + kThreads * 4u - 1) / (kThreads * 4u), kThreads, 0, s>>>(v, B, d_w);
        return cudaGetLastError() == cudaSuccess ? (d_w != nullptr ? 2 : 1) : -1;
    }
    // dynamic shared memory a CTA of this kernel may have: what the device allows less its static part
    static uint32_t dyn_max[kPrbMaxDevices][6];
    if (dyn_max[dev][ki] == 0) {
        // (the frame-layout instance has the same static shared memory: one figure serves both)
        cudaFuncAttributes fa;
        int optin = 0;
        cudaError_t e = cudaSuccess;
        switch (v.fanout) {
        case 2: e = cudaFuncGetAttributes(&fa, prb_sample_kernel<2, true>); break;
        case 4: e = cudaFuncGetAttributes(&fa, prb_sample_kernel<4, true>); break;
        case 8: e = cudaFuncGetAttributes(&fa, prb_sample_kernel<8, true>); break;
        case 16: e = cudaFuncGetAttributes(&fa, prb_sample_kernel<16, true>); break;
        default: e = cudaFuncGetAttributes(&fa, prb_sample_kernel<32, true>); break;
        }
        if (e != cudaSuccess || cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return -1;
        const long room = (long)optin - (long)fa.sharedSizeBytes - 256;
        if (room < (long)(kRingBarBytes + 16 * 1024)) return -1;
        dyn_max[dev][ki] = (uint32_t)room;
    }
    // leaf prefetch: when the level above the leaves is not staged, every walking lane group copies
    // the K*K leaves under its K nodes to shared memory while those nodes are on their way
    const bool prefetch = !uniform && v.depth >= 2 && plan.top_levels < v.depth - 1;
    // All lane groups of a warp take the same path through the descent (its warp-wide barriers and
    // ballots are met by every lane): the groups that prefetch are a whole number of warps' worth.
    const uint32_t groups_per_warp = 32u / v.fanout;       // (fanout 32: one)
    const uint32_t pf_group_bytes = v.fanout * v.fanout * (uint32_t)sizeof(float);
    plan.pf_groups = 0;
    plan.pf_off = 0;
    // One launch, or one per sub-batch of strata [k0, k1): sized like a call of its own, on a stream
    // of its own, so that the first sub-batch is complete while the others are still being copied.
    SamplePlan sub_plan[kPrbMaxSubBatches];
    uint32_t sub_grid[kPrbMaxSubBatches], sub_smem[kPrbMaxSubBatches];
    uint32_t ticket_total = 0, max_smem = 0;
    for (uint32_t i = 0; i < n_sub; ++i) {
        SamplePlan& sp = sub_plan[i];
        sp = plan;
        const uint32_t k0 = (uint32_t)((uint64_t)i * B / n_sub), k1 = (uint32_t)((uint64_t)(i + 1) * B / n_sub);
        const uint32_t strata_here = k1 - k0;
        sp.first_task = k0 * plan.tps;
        sp.n_tasks = strata_here * plan.tps;
        uint32_t grid, smem = 0;
        sp.ring_stages = 0;
        sp.ring_stage_bytes = 0;
        if (row_mode) {
            // one CTA per SM, each with a ring of chunk-sized stages
            uint32_t stage = 0;
            for (int f = 0; f < PRB_NUM_FIELDS; ++f) stage = plan.chunk[f] * 16u > stage ? plan.chunk[f] * 16u : stage;
            stage = (stage + 127u) / 128u * 128u;
            // (sub-batch launches take half the SMs' worth each way round: two of them run side by side,
            // so a later one's prologue hides behind an earlier one's copy)
            uint32_t room = (uint32_t)sm_count;
            if (n_sub > 1) room = (room * 2u + n_sub - 1) / n_sub;
            if (room > (uint32_t)sm_count) room = (uint32_t)sm_count;
            grid = sp.n_tasks < room ? sp.n_tasks : room;
            // strata a CTA can touch: its share of the tasks, plus one for a range that straddles
            const uint32_t tasks_per_cta = (sp.n_tasks + grid - 1) / grid;
            uint32_t strata = (tasks_per_cta + plan.tps - 1) / plan.tps + 1;
            strata = (strata + groups_per_warp - 1) / groups_per_warp * groups_per_warp;
            if (strata > R) strata = R;
            uint32_t pf_bytes = prefetch ? strata * pf_group_bytes : 0u;
            uint32_t ring_bytes = dyn_max[dev][ki] - kRingBarBytes;
            if (pf_bytes + 8u * stage > ring_bytes) pf_bytes = 0;      // (not at the price of the ring)
            ring_bytes -= pf_bytes;
            if (ring_bytes > kRingBytes) ring_bytes = kRingBytes;
            sp.ring_stage_bytes = stage;
            sp.ring_stages = ring_bytes / stage;
            if (sp.ring_stages > 32) sp.ring_stages = 32;
            sp.pf_off = kRingBarBytes + sp.ring_stages * stage;
            sp.pf_groups = pf_bytes ? strata : 0u;
            smem = sp.pf_off + pf_bytes;
        } else {
            // a small batch is spread over more CTAs than it needs: its descents are chains of dependent
            // L2 reads, and more SMs keep more of them in flight
            const uint32_t one_wave = (uint32_t)sm_count * kCtasPerSm;
            const uint32_t per_cta = R >= 4 ? R / 4 : 1;
            const uint32_t want = (strata_here + per_cta - 1) / per_cta;
            grid = want < one_wave ? want : one_wave;
            if (prefetch) {
                uint32_t strata = (strata_here + grid - 1) / grid;
                strata = (strata + groups_per_warp - 1) / groups_per_warp * groups_per_warp;
                if (strata > R) strata = R;
                sp.pf_groups = strata;
                smem = strata * pf_group_bytes;
            }
        }
        sub_grid[i] = grid;
        sub_smem[i] = smem;
        ticket_total += grid;
        if (smem > max_smem) max_smem = smem;
    }
    for (uint32_t i = 0; i < n_sub; ++i) sub_plan[i].ticket_total = ticket_total;
    int extra_launches = 0;
    if (plan.buffer_norm && v.min_off == 0) {
        // the scan of the leaves goes first, on the caller's stream (no min-tree to read the minimum from)
        const uint64_t per_cta = 256ull * 16ull;
        uint64_t ctas = (v.capacity + per_cta - 1) / per_cta;
        if (ctas > (uint64_t)sm_count * 4) ctas = (uint64_t)sm_count * 4;
        prb_leaf_min_kernel<<<(unsigned)ctas, 256, 0, s>>>(v);
        extra_launches = 1;
    }
    static bool big_smem[kPrbMaxDevices][2][6];
    const int fr = v.stack ? 1 : 0;
    cudaError_t attr = cudaSuccess;
    if (n_sub > 1 && (cudaEventRecord(subs->fork, s) != cudaSuccess)) return -1;
    for (uint32_t i = 0; i < n_sub; ++i) {
        cudaStream_t at = s;
        if (n_sub > 1) {
            at = subs->stream[i];
            if (cudaStreamWaitEvent(at, subs->fork, 0) != cudaSuccess) return -1;
        }
        const uint32_t grid = sub_grid[i], smem = sub_smem[i];
        const SamplePlan& sp = sub_plan[i];
        // (a whole batch is launched as a programmatic dependent of the kernel before it on the stream -- its
        // launch is then under way while that kernel runs; it waits for that kernel before its first read)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = at;
        cudaLaunchAttribute pss[1];
        pss[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pss[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = pss;
        cfg.numAttrs = n_sub == 1 ? 1 : 0;
#define PRB_LAUNCH_SAMPLE_AS(KK, FF)                                                                              \
    do {                                                                                                          \
        if (max_smem && !big_smem[dev][fr][ki]) {                                                                 \
            attr = cudaFuncSetAttribute(prb_sample_kernel<KK, FF>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                        (int)dyn_max[dev][ki]);                                                   \
            big_smem[dev][fr][ki] = (attr == cudaSuccess);                                                        \
        }                                                                                                         \
        if (attr == cudaSuccess)                                                                                  \
            attr = cudaLaunchKernelEx(&cfg, prb_sample_kernel<KK, FF>, v, B, beta, seed, d_idx, d_w, dst, sp);     \
    } while (0)
#define PRB_LAUNCH_SAMPLE(KK)                                                                                     \
    do { if (fr) PRB_LAUNCH_SAMPLE_AS(KK, true); else PRB_LAUNCH_SAMPLE_AS(KK, false); } while (0)
        switch (v.fanout) {
        case 2: PRB_LAUNCH_SAMPLE(2); break;
        case 4: PRB_LAUNCH_SAMPLE(4); break;
        case 8: PRB_LAUNCH_SAMPLE(8); break;
        case 16: PRB_LAUNCH_SAMPLE(16); break;
        default: PRB_LAUNCH_SAMPLE(32); break;
        }
#undef PRB_LAUNCH_SAMPLE
#undef PRB_LAUNCH_SAMPLE_AS
        if (attr != cudaSuccess) return -1;
        if (n_sub > 1) {
            // the sub-batch's rows and indices are in place when its event fires; the caller's stream
            // goes on when all of them have (the weights are final only then)
            if (cudaEventRecord(subs->done[i], at) != cudaSuccess || cudaStreamWaitEvent(s, subs->done[i], 0) != cudaSuccess)
                return -1;
        }
    }
    return cudaGetLastError() == cudaSuccess ? (int)n_sub + extra_launches : -1;
}

int prb_launch_descend(const PrbView& v, uint32_t B, uint64_t seed, unsigned char* handoff, cudaStream_t s, int uniform, int buffer_norm)
{
    const int sm_count = prb_sm_count();
    SamplePlan plan;
    PrbBatch none;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) none.ptr[f] = nullptr;
    plan_row_mode(v, none, plan);
    plan.n_tasks = B; plan.first_task = 0; plan.ticket_total = 0;
    plan.ring_stages = 0; plan.ring_stage_bytes = 0;
    plan.uniform = uniform ? 1u : 0u;
    plan.buffer_norm = (buffer_norm && !uniform) ? 1u : 0u;
    plan_staged_top(v, uniform != 0, plan);
    int launches = 1;
    if (plan.buffer_norm && v.min_off == 0) {
        // the scan of the leaves goes first, on the same stream (no min-tree to read the minimum from)
        const uint64_t per_cta = 256ull * 16ull;
        uint64_t ctas = (v.capacity + per_cta - 1) / per_cta;
        if (ctas > (uint64_t)sm_count * 4) ctas = (uint64_t)sm_count * 4;
        prb_leaf_min_kernel<<<(unsigned)ctas, 256, 0, s>>>(v);
        launches = 2;
    }
    // one CTA per SM at most (the kernel has to fit beside a row copy's CTAs), each walking its strata
    // kThreads / K at a time; a small batch is spread thin, a group or two per CTA
    const uint32_t R = kThreads / v.fanout;
    const uint32_t per_cta = R >= 4 ? R / 4 : 1;
    uint32_t grid = (B + per_cta - 1) / per_cta;
    if (grid > (uint32_t)sm_count) grid = (uint32_t)sm_count;
    const bool prefetch = !uniform && v.depth >= 2 && plan.top_levels < v.depth - 1;
    const uint32_t groups_per_warp = 32u / v.fanout;
    uint32_t smem = 0;
    plan.pf_groups = 0; plan.pf_off = 0;
    if (prefetch) {
        uint32_t strata = (B + grid - 1) / grid;
        strata = (strata + groups_per_warp - 1) / groups_per_warp * groups_per_warp;      // whole warps' worth of groups
        if (strata > R) strata = R;
        plan.pf_groups = strata;
        smem = strata * v.fanout * v.fanout * (uint32_t)sizeof(float);
    }
    switch (v.fanout) {
    case 2: prb_descend_kernel<2><<<grid, kThreads, smem, s>>>(v, B, seed, handoff, plan); break;
    case 4: prb_descend_kernel<4><<<grid, kThreads, smem, s>>>(v, B, seed, handoff, plan); break;
    case 8: prb_descend_kernel<8><<<grid, kThreads, smem, s>>>(v, B, seed, handoff, plan); break;
    case 16: prb_descend_kernel<16><<<grid, kThreads, smem, s>>>(v, B, seed, handoff, plan); break;
    default: prb_descend_kernel<32><<<grid, kThreads, smem, s>>>(v, B, seed, handoff, plan); break;
    }
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int prb_launch_gather(const PrbView& v, uint32_t B, float beta, const unsigned char* handoff, int32_t* d_idx, float* d_w,
                      const PrbBatch& dst, cudaStream_t s, bool early_reads, int part, uint32_t new_n)
{
    if (part < 0 || part > 2 || (part && (early_reads || new_n == 0 || new_n > v.capacity))) return -1;
    SamplePlan plan;
    if (!plan_row_mode(v, dst, plan)) return -1;
    const int sm_count = prb_sm_count();
    const int dev = prb_current_device();
    plan.n_tasks = B * plan.tps;
    plan.first_task = 0;
    plan.ticket_total = 0;
    plan.uniform = 0; plan.buffer_norm = 0; plan.top_levels = 0; plan.top_vec4 = 0;
    for (uint32_t l = 0; l < PRB_MAX_LEVELS; ++l) plan.top_off[l] = 0;
    plan.pf_groups = 0; plan.pf_off = 0;
    uint32_t stage = 0;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) stage = plan.chunk[f] * 16u > stage ? plan.chunk[f] * 16u : stage;
    stage = (stage + 127u) / 128u * 128u;
    plan.ring_stage_bytes = stage;
    plan.ring_stages = kGatherRingBytes / stage;
    if (plan.ring_stages > 32) plan.ring_stages = 32;
    const uint32_t smem = kRingBarBytes + plan.ring_stages * stage;
    static bool big_smem[kPrbMaxDevices];
    if (!big_smem[dev]) {
        const int most = (int)(kRingBarBytes + kGatherRingBytes);
        if (cudaFuncSetAttribute(prb_gather_rows_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(prb_gather_rows_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(prb_gather_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess)
            return -1;
        big_smem[dev] = true;
    }
    const uint32_t grid = plan.n_tasks < (uint32_t)sm_count ? plan.n_tasks : (uint32_t)sm_count;
    // (launched as a programmatic dependent of the kernel before it on the stream: see the kernel)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGatherThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = part ? 0 : 1;      // (the two launches of a split copy depend in full on what precedes them)
    const uint32_t early = early_reads ? 1u : 0u;
    cudaError_t e;
    if (part == 0) e = cudaLaunchKernelEx(&cfg, prb_gather_rows_kernel<0>, v, B, beta, handoff, d_idx, d_w, dst, plan, early, 0u);
    else if (part == 1) e = cudaLaunchKernelEx(&cfg, prb_gather_rows_kernel<1>, v, B, beta, handoff, d_idx, d_w, dst, plan, early, new_n);
    else e = cudaLaunchKernelEx(&cfg, prb_gather_rows_kernel<2>, v, B, beta, handoff, d_idx, d_w, dst, plan, early, new_n);
    return e == cudaSuccess ? 1 : -1;
}
