// Batched insertion: ring write of n transitions into the Data Storage and the matching
// leaf writes + ancestor re-sum in the sum tree (PEARL Section V-A: insertion is realised as
// priority retrieval followed by priority update; Listing 2: experiences are added to the
// Data Storage and insertion requests go to the Replay Manager).
//
// One kernel per call, in one of two shapes.
//   Short rows: CTA 0 owns the tree, the other CTAs copy tiles of the dense batch to ring slots
//   through registers.
//   Long rows (at least 8 KB of 16-byte granules, Atari-shaped): one CTA per SM; CTA 0 does the
//   tree work, in every other CTA warp 0 drives bulk asynchronous copies global -> shared ->
//   global through a ~200 KB ring (row chunks of <= 8 KB, one lane per stage), issuing its
//   loads before the cursor has even arrived, and the other warps copy the short fields.
// Tree work (prb_tree.cuh): an optional priority update first (pearl_prb_update_insert), then
// the n leaves, then one re-sum pass per level over every dirty parent.
// The CTA that is last to have read the cursor advances it (and the fill count) while the copies
// are still running.  No CTA waits on another.
#include "prb_tree.cuh"

namespace {

constexpr int kTeamShort = 256;                  // short-row kernel: threads that copy tiles / do the tree work
constexpr int kThreadsShort = kTeamShort + 32;   //   ... then the warp whose lane 0 publishes the cursor
constexpr int kTeamRows = 960;                   // long-row kernel: warps 1..30 do the tree work / short fields
constexpr int kThreadsRows = 32 + kTeamRows + 32;   //   warp 0 drives the ring, lane 0 of warp 31 publishes
constexpr uint32_t kChunk = 512;             // upper bound on granules per chunk of a long row (8 KB)
constexpr uint32_t kTile = 2048;             // granules per tile of short rows
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
};

// Short rows: tile `tile` of the dense batch of field f, which may span many rows.
template <typename T>
__device__ __forceinline__ void copy_flat_tile(const PrbView& v, int f, const PrbBatch& src, uint32_t n, uint64_t cursor,
                                               uint32_t tile, uint32_t rank, uint32_t nthreads)
{
    const uint32_t W = v.field_bytes[f] / sizeof(T);
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
                           return slot * W + (e - r * W);
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

// Taken by one thread per CTA once the whole CTA holds the cursor and the fill count: the last CTA
// to get here publishes the new values.  Nothing later in the kernel reads them from global
// memory, so this happens while the copies are still running.
__device__ __forceinline__ void publish_if_last(const PrbView& v, uint32_t n, uint64_t cursor, unsigned long long fill)
{
    __threadfence();
    const unsigned int done = atomicAdd(&v.state->insert_ticket, 1u);
    if (done == gridDim.x - 1) {
        const uint64_t N = v.capacity;
        uint64_t c = cursor + n;
        if (c >= N) c -= N;
        v.state->cursor = c;
        fill += n;
        v.state->fill = fill > N ? N : fill;
        v.state->insert_ticket = 0;
    }
}

// Short rows only: CTA 0 = the tree work (an optional priority update, then the insertion's leaves
// and re-sum), CTAs 1.. = a contiguous range of tiles each.  Threads 0..kTeamShort-1 work; thread
// kTeamShort reads cursor and fill for the CTA and takes the ticket.
__global__ void __launch_bounds__(kThreadsShort, 2)
prb_insert_kernel(const __grid_constant__ PrbView v, const __grid_constant__ PrbBatch src,
                  const __grid_constant__ InsertPlan plan, const __grid_constant__ PrbTreeWork work)
{
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ unsigned long long s_cursor, s_fill;
    const uint32_t tid = threadIdx.x, n = work.n;
    if (tid == kTeamShort) { s_cursor = v.state->cursor; s_fill = v.state->fill; }
    __syncthreads();
    const uint64_t cursor = s_cursor;
    if (tid == kTeamShort) {
        publish_if_last(v, n, cursor, s_fill);
    } else if (tid < kTeamShort) {
        if (blockIdx.x == 0) {
            PrbTeam team;
            team.rank = tid; team.size = kTeamShort; team.whole_cta = false;
            prb_tree_team(v, team, work, cursor, s_fill, s_dyn);
        } else {
            const uint32_t n_tiles = plan.first_tile[PRB_NUM_FIELDS];
            const uint32_t copy_ctas = gridDim.x - 1, c = blockIdx.x - 1;
            const uint32_t t_lo = (uint32_t)(((uint64_t)c * n_tiles) / copy_ctas);
            const uint32_t t_hi = (uint32_t)(((uint64_t)(c + 1) * n_tiles) / copy_ctas);
            for (uint32_t t = t_lo; t < t_hi; ++t) copy_tile(v, plan, src, n, cursor, t, tid, kTeamShort);
        }
    }
}

// Long rows present.  CTA 0 does the tree work (optional update, then the insertion) with warps
// 1..30 and moves no rows.  In the other CTAs warp 0 drives the ring: lane s owns stage s and moves
// row chunks t_lo+s, t_lo+s+S, ... of the CTA's range, its first load going out before the cursor
// has arrived (a source address does not depend on it); warps 1..30 copy the short-field tiles,
// dealt round-robin.  Lane 0 of warp 31: cursor, fill and ticket.
__global__ void __launch_bounds__(kThreadsRows, 1)
prb_insert_rows_kernel(const __grid_constant__ PrbView v, const __grid_constant__ PrbBatch src,
                       const __grid_constant__ InsertPlan plan, const __grid_constant__ PrbTreeWork work)
{
    extern __shared__ __align__(128) unsigned char s_ring[];
    __shared__ unsigned long long s_cursor, s_fill;
    const uint32_t tid = threadIdx.x, n = work.n;
    const uint32_t n_tasks = plan.first_task[PRB_NUM_FIELDS];
    const uint32_t copy_ctas = gridDim.x - 1;
    const bool copies = blockIdx.x > 0;
    const uint32_t c = blockIdx.x - 1;
    const uint32_t t_lo = copies ? (uint32_t)(((uint64_t)c * n_tasks) / copy_ctas) : 0u;
    const uint32_t t_hi = copies ? (uint32_t)(((uint64_t)(c + 1) * n_tasks) / copy_ctas) : 0u;
    const bool ring_lane = copies && tid < plan.ring_stages;
    constexpr uint32_t kPublisher = 32 + kTeamRows;

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
    if (tid == kPublisher) { s_cursor = v.state->cursor; s_fill = v.state->fill; }
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
        publish_if_last(v, n, cursor, s_fill);
    } else if (ring_lane) {
        while (t < t_hi) {
            uint64_t slot = cursor + row;
            if (slot >= v.capacity) slot -= v.capacity;
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
        team.rank = tid - 32u; team.size = kTeamRows; team.whole_cta = false;
        if (blockIdx.x == 0) {
            prb_tree_team(v, team, work, cursor, s_fill, s_ring);
        } else {
            const uint32_t n_tiles = plan.first_tile[PRB_NUM_FIELDS];
            for (uint32_t tile = c; tile < n_tiles; tile += copy_ctas)
                copy_tile(v, plan, src, n, cursor, tile, team.rank, team.size);
        }
    }
}

}  // namespace

int prb_launch_insert(const PrbView& v, uint32_t n, const PrbBatch& src, const float* d_prio, cudaStream_t s,
                      uint32_t upd_B, const int32_t* upd_idx, const float* upd_val, int upd_raw, float alpha, float eps)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
            sm_count = 148;
    }
    PrbTreeWork w;
    w.B = upd_B; w.n2 = 2; w.idx = upd_idx; w.val = upd_val; w.raw = upd_raw; w.alpha = alpha; w.eps = eps;
    w.n = n; w.prio = d_prio; w.forward = 0;
    while (w.n2 < upd_B) w.n2 <<= 1;

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
    if (tasks == 0) {
        const uint32_t fwd = prb_fwd_plan(v, &w, kTeamShort, 96 * 1024);
        const uint32_t smem = fwd ? fwd : (uint32_t)prb_tree_smem_bytes(upd_B ? w.n2 : 0u, v.fanout, kTeamShort);
        static bool big_smem = false;
        if (smem + 64 > 48 * 1024 && !big_smem) {
            if (cudaFuncSetAttribute(prb_insert_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess)
                return -1;
            big_smem = true;
        }
        const uint32_t one_wave = (uint32_t)sm_count * 2 - 1;     // CTA 0 is the tree CTA
        const uint32_t copy_ctas = tiles < one_wave ? tiles : one_wave;
        prb_insert_kernel<<<copy_ctas + 1, kThreadsShort, smem, s>>>(v, src, plan, w);
    } else {
        stage = (stage + 127u) / 128u * 128u;
        plan.ring_stage_bytes = stage;
        plan.ring_stages = kRingBytes / stage;
        if (plan.ring_stages > 32) plan.ring_stages = 32;
        uint32_t smem = kRingBarBytes + plan.ring_stages * stage;
        const uint32_t fwd = prb_fwd_plan(v, &w, kTeamRows, kRingBarBytes + kRingBytes);
        const uint32_t tree_smem = fwd ? fwd : (uint32_t)prb_tree_smem_bytes(upd_B ? w.n2 : 0u, v.fanout, kTeamRows);
        if (tree_smem > smem) smem = tree_smem;
        static bool big_smem = false;
        if (!big_smem) {
            if (cudaFuncSetAttribute(prb_insert_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)(kRingBarBytes + kRingBytes)) != cudaSuccess)
                return -1;
            big_smem = true;
        }
        const uint32_t want = tasks + 1;                           // CTA 0 is the tree CTA
        const uint32_t grid = want < (uint32_t)sm_count ? want : (uint32_t)sm_count;
        prb_insert_rows_kernel<<<grid, kThreadsRows, smem, s>>>(v, src, plan, w);
    }
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
