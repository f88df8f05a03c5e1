// Batched insertion: ring write of n transitions into the Data Storage and the matching
// leaf writes + ancestor re-sum in the sum tree (PEARL Section V-A: insertion is realised as
// priority retrieval followed by priority update; Listing 2: experiences are added to the
// Data Storage and insertion requests go to the Replay Manager).
//
// One kernel per call, in one of two shapes.
//   Short rows: CTA 0 owns the tree, the other CTAs copy tiles of the dense batch to ring slots
//   through registers.
//   Long rows (at least 8 KB of 16-byte granules, Atari-shaped): one CTA per SM; warp 0 of
//   every CTA drives bulk asynchronous copies global -> shared -> global through a ~200 KB
//   ring (row chunks of <= 8 KB, one lane per stage), issuing its loads before the cursor has
//   even arrived; the other warps copy the short fields.  CTA 0 does the tree and moves no rows;
//   with a priority update in the same call the tree work is a kernel of its own on a second
//   stream (prb_update.cu) and every CTA here copies.
// Tree work: write the n leaves, then re-sum the dirty parents level by level (a contiguous
// slot range dirties a contiguous parent range on every level, so no sorting is needed).
// The CTA that is last to have read the cursor advances it (and the fill count) while the copies
// are still running.  No CTA waits on another.
#include "prb_tree.cuh"

namespace {

constexpr int kWorkers = 256;                // threads that copy short rows / do the tree work
constexpr int kThreadsShort = kWorkers + 32;     // short-row kernel: workers, then the warp whose lane 0 publishes the cursor
constexpr int kThreadsRows = 32 + kWorkers + 32; // long-row kernel: ring warp, workers, publishing warp
constexpr uint32_t kChunk = 512;             // upper bound on granules per chunk of a long row (8 KB)
constexpr uint32_t kTile = kWorkers * 8;     // granules per tile of short rows
constexpr uint32_t kRowMode = 512;           // rows of at least this many 16-byte granules are split into chunks
constexpr uint32_t kRingBytes = 198 * 1024;  // bulk-copy ring (dynamic shared memory), <= 32 stages
constexpr uint32_t kRingBarBytes = 1024;     // room for the ring's mbarriers in front of its buffers

struct InsertPlan {
    // short-row tiles, numbered field by field: tiles of field f are [first_tile[f], first_tile[f+1])
    uint32_t first_tile[PRB_NUM_FIELDS + 1];
    // long-row tasks (one chunk of one row), numbered field by field
    uint32_t first_task[PRB_NUM_FIELDS + 1];
    uint32_t chunks[PRB_NUM_FIELDS];          // chunks per row of a long-row field, else 0
    uint32_t chunk[PRB_NUM_FIELDS];           // granules per chunk
    uint32_t ring_stages, ring_stage_bytes;
    // CTAs of a tree kernel that runs beside this one and does the insertion's tree work (0: this
    // kernel does it); they share the cursor ticket
    uint32_t tree_ctas;
};

// Short rows: tile `tile` of the dense batch of field f, which may span many rows.
template <typename T>
__device__ __forceinline__ void copy_flat_tile(const PrbView& v, int f, const PrbBatch& src, uint32_t n, uint64_t cursor,
                                               uint32_t tile, uint32_t rank, uint32_t nthreads)
{
    const uint32_t W = v.field_bytes[f] / sizeof(T), Wp = v.field_pitch[f] / sizeof(T);     // granules per row, per slot of the store
    const uint64_t N = v.capacity;
    const uint64_t total = (uint64_t)n * W;
    const uint64_t e0 = (uint64_t)tile * kTile;
    const uint32_t e1 = (uint32_t)min(total, e0 + kTile);
    prb_copy_mapped<T>(reinterpret_cast<T*>(v.store[f]), reinterpret_cast<const T*>(src.ptr[f]), (uint32_t)e0, e1,
                       [=](uint32_t e) { return (uint64_t)e; },
                       [=](uint32_t e) {
                           const uint32_t r = e / W;
                           uint64_t slot = cursor + r;
                           if (slot >= N) slot -= N;
                           if (!PRB_IN_BOUNDS(v, slot < N && r < n)) slot = 0;
                           return slot * Wp + (e - r * W);
                       },
                       rank, nthreads);
}

__device__ __forceinline__ void copy_tile(const PrbView& v, const InsertPlan& plan, const PrbBatch& src, uint32_t n,
                                          uint64_t cursor, uint32_t tile, uint32_t rank, uint32_t nthreads)
{
    int f = 0;
    while (tile >= plan.first_tile[f + 1]) ++f;
    const uint32_t local = tile - plan.first_tile[f];
    switch (v.field_vec[f]) {
    case 16: copy_flat_tile<uint4>(v, f, src, n, cursor, local, rank, nthreads); break;
    case 8: copy_flat_tile<uint2>(v, f, src, n, cursor, local, rank, nthreads); break;
    case 4: copy_flat_tile<uint32_t>(v, f, src, n, cursor, local, rank, nthreads); break;
    case 2: copy_flat_tile<uint16_t>(v, f, src, n, cursor, local, rank, nthreads); break;
    default: copy_flat_tile<uint8_t>(v, f, src, n, cursor, local, rank, nthreads); break;
    }
}

// A priority update to run before the insertion's tree work, by the same team (B == 0: none).
struct FusedUpdate {
    uint32_t B, n2;
    const int32_t* idx;
    const float* val;
    int raw;
    float alpha, eps;
};

// Short rows only: CTA 0 = tree (after the optional update), CTAs 1.. = a contiguous range of tiles
// each.  Threads 0..kWorkers-1 work; thread kWorkers reads the cursor for the CTA and takes the ticket.
template <bool kFrames, bool kMin>
__global__ void __launch_bounds__(kThreadsShort, 2)
prb_insert_kernel(const __grid_constant__ PrbView v, uint32_t n, const __grid_constant__ PrbBatch src,
                  const float* __restrict__ prio, const __grid_constant__ InsertPlan plan,
                  const __grid_constant__ FusedUpdate upd)
{
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ unsigned long long s_cursor, s_fill;     // read once per CTA, before anything is published
    __shared__ unsigned int s_maxp;                     // running maximum of priorities at kernel start
    const uint32_t tid = threadIdx.x;
    // (the kernel after this one on the stream, if it was launched as a programmatic dependent, may be made
    // resident now; it waits for this kernel's completion before it reads anything)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == kWorkers) { s_cursor = v.state->cursor; s_fill = v.state->fill; s_maxp = v.state->max_prio_bits; }
    // the tree CTA fetches its first inputs now, while the cursor is on its way
    // (and starts the copy of the tree's top into shared memory, behind the update's keys)
    PrbPreloaded pre = PrbPreloaded{false, false, 0, 0.0f, 0.0f};
    PrbTop top;
    if (blockIdx.x == 0 && tid < kWorkers) {
        if (tid < upd.B) { pre.has_update = true; pre.idx = upd.idx[tid]; pre.val = upd.val[tid]; }
        if (tid < n && prio != nullptr) { pre.has_prio = true; pre.prio = prio[tid]; }
        if (v.top_levels) top.mem = reinterpret_cast<float*>(s_dyn + (upd.B ? prb_update_smem_bytes(upd.n2) : 0));
        if (kMin && v.top_levels) top.mem_min = top.mem + v.top_floats;
        prb_top_begin(v, top, tid, kWorkers);
    }
    __syncthreads();
    const uint64_t cursor = s_cursor;
    if (tid == kWorkers) {
        prb_publish_if_last(v, n, cursor, s_fill, gridDim.x);
    } else if (tid < kWorkers) {
        if (blockIdx.x == 0) {
            PrbTeam team;
            team.rank = tid; team.size = kWorkers; team.whole_cta = false;
            if (kMin) team.min_off = v.min_off;
            if (upd.B)      // update and insertion share one re-sum pass per level
                prb_update_team(v, team, upd.B, upd.n2, upd.idx, upd.val, upd.raw, upd.alpha, upd.eps, s_fill, s_dyn, n, prio, cursor, pre, 0, top,
                                src.ptr[F_DONE], kFrames ? v.stack : 0u);
            else
                prb_insert_tree_team(v, team, n, prio, cursor, pre, s_maxp, top, src.ptr[F_DONE], kFrames ? v.stack : 0u);
        } else {
            const uint32_t n_tiles = plan.first_tile[PRB_NUM_FIELDS];
            const uint32_t copy_ctas = gridDim.x - 1, c = blockIdx.x - 1;
            const uint32_t t_lo = (uint32_t)(((uint64_t)c * n_tiles) / copy_ctas);
            const uint32_t t_hi = (uint32_t)(((uint64_t)(c + 1) * n_tiles) / copy_ctas);
            for (uint32_t t = t_lo; t < t_hi; ++t) copy_tile(v, plan, src, n, cursor, t, tid, kWorkers);
        }
    }
}

// Long rows present.  Warp 0: lane s owns ring stage s and moves row chunks t_lo+s, t_lo+s+S, ...
// of this CTA's range; the first loads go out before the cursor has arrived (a source address does
// not depend on it).  Threads 32..32+kWorkers-1: the tree work (CTA 0, unless a tree kernel beside
// this one does it) and the short-field tiles (dealt round-robin, CTA 1 first).  Thread
// 32+kWorkers: cursor and ticket.
template <bool kFrames, bool kMin>
__global__ void __launch_bounds__(kThreadsRows, 1)
prb_insert_rows_kernel(const __grid_constant__ PrbView v, uint32_t n, const __grid_constant__ PrbBatch src,
                       const float* __restrict__ prio, const __grid_constant__ InsertPlan plan)
{
    extern __shared__ __align__(128) unsigned char s_ring[];
    __shared__ unsigned long long s_cursor, s_fill;     // read once per CTA, before anything is published
    __shared__ unsigned int s_maxp;                     // running maximum of priorities at kernel start
    const uint32_t tid = threadIdx.x;
    const uint32_t n_tasks = plan.first_task[PRB_NUM_FIELDS];
    // A CTA that does the tree work moves no rows: the answers to its tree reads would queue behind
    // the data of its own bulk loads.
    const uint32_t first_copy_cta = (plan.tree_ctas == 0 && gridDim.x > 1) ? 1u : 0u;
    const uint32_t copy_ctas = gridDim.x - first_copy_cta;
    const bool copies = blockIdx.x >= first_copy_cta;
    const uint32_t cc = blockIdx.x - first_copy_cta;
    const uint32_t t_lo = copies ? (uint32_t)(((uint64_t)cc * n_tasks) / copy_ctas) : 0u;
    const uint32_t t_hi = copies ? (uint32_t)(((uint64_t)(cc + 1) * n_tasks) / copy_ctas) : 0u;
    const bool ring_lane = copies && tid < plan.ring_stages;
    constexpr uint32_t kPublisher = 32 + kWorkers;

    // one row chunk: field, row in the batch, first granule, bytes
    auto locate = [&](uint32_t t, int& f, uint32_t& row, uint32_t& W, uint32_t& e0, uint32_t& bytes) {
        f = 0;
        while (t >= plan.first_task[f + 1]) ++f;
        const uint32_t local = t - plan.first_task[f];
        row = local / plan.chunks[f];
        W = v.field_bytes[f] / 16u;
        e0 = (local - row * plan.chunks[f]) * plan.chunk[f];
        bytes = min(W - e0, plan.chunk[f]) * 16u;
    };

    PrbBulkLane ring;
    int f = 0; uint32_t row = 0, W = 0, e0 = 0, bytes = 0;
    uint32_t t = t_lo + tid;
    // (beside a tree kernel this kernel keeps the row cursor only: see PrbState)
    if (tid == kPublisher) { s_cursor = plan.tree_ctas ? v.state->row_cursor : v.state->cursor; s_fill = v.state->fill; s_maxp = v.state->max_prio_bits; }
    if (ring_lane) {
        ring.init(s_ring + 8u * tid, s_ring + kRingBarBytes + tid * plan.ring_stage_bytes);
        if (t < t_hi) {
            locate(t, f, row, W, e0, bytes);
            ring.load(src.ptr[f] + ((uint64_t)row * W + e0) * 16u, bytes);
        }
    }
    __syncthreads();
    const uint64_t cursor = s_cursor;

    if (tid == kPublisher) {
        prb_publish_if_last(v, n, cursor, s_fill, gridDim.x, plan.tree_ctas ? kPrbPublishRows : kPrbPublishAll);
    } else if (ring_lane) {
        while (t < t_hi) {
            uint64_t slot = cursor + row;
            if (slot >= v.capacity) slot -= v.capacity;
            if (!PRB_IN_BOUNDS(v, slot < v.capacity && row < n && e0 < W && bytes <= plan.ring_stage_bytes)) slot = 0;
            ring.store(v.store[f] + (slot * W + e0) * 16u, bytes);
            t += plan.ring_stages;
            if (t < t_hi) {
                locate(t, f, row, W, e0, bytes);
                ring.load(src.ptr[f] + ((uint64_t)row * W + e0) * 16u, bytes);
            }
        }
        ring.finish();
        if (ring.failed) atomicOr(&v.state->status, PEARL_ST_INTERNAL);
    } else if (tid >= 32 && tid < kPublisher) {
        PrbTeam team;
        team.rank = tid - 32u; team.size = kWorkers; team.whole_cta = false;
        if (kMin) team.min_off = v.min_off;
        if (blockIdx.x == 0 && plan.tree_ctas == 0)
            prb_insert_tree_team(v, team, n, prio, cursor, PrbPreloaded{false, false, 0, 0.0f, 0.0f}, s_maxp, PrbTop{}, src.ptr[F_DONE],
                                 kFrames ? v.stack : 0u);
        const uint32_t n_tiles = plan.first_tile[PRB_NUM_FIELDS];
        for (uint32_t tile = (blockIdx.x + gridDim.x - 1) % gridDim.x; tile < n_tiles; tile += gridDim.x)
            copy_tile(v, plan, src, n, cursor, tile, team.rank, team.size);
    }
}

}  // namespace

int prb_launch_insert(const PrbView& v, uint32_t n, const PrbBatch& src, const float* d_prio, cudaStream_t s,
                      uint32_t upd_B, const int32_t* upd_idx, const float* upd_val, int upd_raw, float alpha, float eps,
                      const PrbFork* fork, bool* forked_out, bool rows_only)
{
    if (forked_out) *forked_out = false;
    if (rows_only && upd_B) return -1;
    const int sm_count = prb_sm_count();
    const int dev = prb_current_device();
    FusedUpdate upd;
    upd.B = upd_B; upd.n2 = prb_update_n2(upd_B); upd.idx = upd_idx; upd.val = upd_val; upd.raw = upd_raw; upd.alpha = alpha; upd.eps = eps;

    InsertPlan plan;
    uint32_t tiles = 0, tasks = 0, stage = 0;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        plan.first_tile[f] = tiles;
        plan.first_task[f] = tasks;
        plan.chunks[f] = 0;
        plan.chunk[f] = 0;
        if (v.field_bytes[f] == 0 || src.ptr[f] == nullptr) continue;
        const uint32_t W = v.field_bytes[f] / v.field_vec[f];
        if (v.field_vec[f] == 16 && W >= kRowMode) {
            plan.chunks[f] = (W + kChunk - 1) / kChunk;
            plan.chunk[f] = (W + plan.chunks[f] - 1) / plan.chunks[f];
            tasks += n * plan.chunks[f];
            if (plan.chunk[f] * 16u > stage) stage = plan.chunk[f] * 16u;
        } else {
            const uint64_t total = (uint64_t)n * W;
            tiles += (uint32_t)((total + kTile - 1) / kTile);
        }
    }
    plan.first_tile[PRB_NUM_FIELDS] = tiles;
    plan.first_task[PRB_NUM_FIELDS] = tasks;
    plan.ring_stages = 0;
    plan.ring_stage_bytes = 0;
    plan.tree_ctas = 0;
    int launches = 1;
    bool forked = false;
    uint32_t rows_grid = 0;
    if (rows_only && tasks == 0) return -1;
    const bool fork_tree = upd.B && tasks > 0 && upd.B <= PEARL_UPDATE_SUBBATCH && fork != nullptr;
    if (tasks > 0) {
        stage = (stage + 127u) / 128u * 128u;
        plan.ring_stage_bytes = stage;
        plan.ring_stages = kRingBytes / stage;
        if (plan.ring_stages > 32) plan.ring_stages = 32;
    }
    if (tasks > 0) {
        // Without a tree kernel CTA 0 does the tree work and no copies; with one, its CTAs get SMs of
        // their own: a copy CTA takes an SM's whole shared memory and would wait for them to leave.
        const uint32_t want = tasks + ((fork_tree || rows_only) ? 0u : 1u);
        uint32_t room = (uint32_t)sm_count;
        if (fork_tree && room > 2u * prb_update_ctas(v, upd.B)) room -= prb_update_ctas(v, upd.B);
        rows_grid = want < room ? want : room;
    }
    if (rows_only) {
        plan.tree_ctas = 1;       // (CTA 0 copies like the others and the row cursor is published by itself)
    } else if (fork_tree) {
        // Long rows: the update and the insertion's tree work are one kernel on the side stream, the
        // row copy another on the caller's stream; neither waits for the other (each advances a
        // cursor of its own), and the caller's stream goes on when both are done.  (In one kernel the tree's chain of dependent reads, slowed by the
        // copy's traffic, was measured to outlast the copy by far.)
        plan.tree_ctas = prb_update_ctas(v, upd.B);
        if (cudaEventRecord(fork->fork, s) != cudaSuccess || cudaStreamWaitEvent(fork->side, fork->fork, 0) != cudaSuccess)
            return -1;
        const int k = prb_launch_update(v, upd_B, upd_idx, upd_val, upd_raw, alpha, eps, fork->side, 0, n, d_prio, src.ptr[F_DONE]);
        if (k != 1 || cudaEventRecord(fork->join, fork->side) != cudaSuccess) return -1;
        upd.B = 0;
        launches = 2;
        forked = true;
        if (forked_out) *forked_out = true;
    } else if (upd.B && (tasks > 0 || upd.B >= kPrbWideFrom)) {
        // (a batch for the many-CTA update, or no side stream: the update goes first, in launches of its
        // own; so does a batch of exactly one entry per thread, measured 14-25 us as two launches against
        // 15-33 us fused at 1024 entries + 1024 insertions)
        const int k = prb_launch_update(v, upd_B, upd_idx, upd_val, upd_raw, alpha, eps, s);
        if (k < 0) return -1;
        upd.B = 0;
        launches = 1 + k;
    }
    const uint32_t upd_smem = upd.B ? (uint32_t)prb_update_smem_bytes(upd.n2) : 0u;
    if (tasks == 0) {
        static bool big_smem[kPrbMaxDevices];
        if (!big_smem[dev]) {
            const int most = (int)(prb_update_smem_bytes(PEARL_UPDATE_SUBBATCH) + 2 * kPrbTopFloats * sizeof(float));
            bool ok = true;
#define PRB_ALLOW_SMEM(FF, MM) ok = ok && cudaFuncSetAttribute(prb_insert_kernel<FF, MM>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) == cudaSuccess
            PRB_ALLOW_SMEM(false, false); PRB_ALLOW_SMEM(true, false); PRB_ALLOW_SMEM(false, true); PRB_ALLOW_SMEM(true, true);
#undef PRB_ALLOW_SMEM
            if (!ok) return -1;
            big_smem[dev] = true;
        }
        const uint32_t one_wave = (uint32_t)sm_count * 2 - 1;     // CTA 0 is the tree CTA
        const uint32_t copy_ctas = tiles < one_wave ? tiles : one_wave;
        const uint32_t smem = upd_smem + v.top_floats * (uint32_t)sizeof(float) * (v.min_off ? 2u : 1u);
#define PRB_LAUNCH_INSERT_AS(FF, MM) prb_insert_kernel<FF, MM><<<copy_ctas + 1, kThreadsShort, smem, s>>>(v, n, src, d_prio, plan, upd)
        PRB_WITH_TREE_OPTIONS(v, PRB_LAUNCH_INSERT_AS);
#undef PRB_LAUNCH_INSERT_AS
    } else {
        const uint32_t smem = kRingBarBytes + plan.ring_stages * plan.ring_stage_bytes;
        static bool big_rows[kPrbMaxDevices];
        if (!big_rows[dev]) {
            bool ok = true;
#define PRB_ALLOW_SMEM(FF, MM) \
    ok = ok && cudaFuncSetAttribute(prb_insert_rows_kernel<FF, MM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kRingBarBytes + kRingBytes)) == cudaSuccess
            PRB_ALLOW_SMEM(false, false); PRB_ALLOW_SMEM(true, false); PRB_ALLOW_SMEM(false, true); PRB_ALLOW_SMEM(true, true);
#undef PRB_ALLOW_SMEM
            if (!ok) return -1;
            big_rows[dev] = true;
        }
#define PRB_LAUNCH_ROWS_AS(FF, MM) prb_insert_rows_kernel<FF, MM><<<rows_grid, kThreadsRows, smem, s>>>(v, n, src, d_prio, plan)
        PRB_WITH_TREE_OPTIONS(v, PRB_LAUNCH_ROWS_AS);
#undef PRB_LAUNCH_ROWS_AS
        if (forked && cudaStreamWaitEvent(s, fork->join, 0) != cudaSuccess) return -1;
    }
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}
