// Batched insertion: ring write of n transitions into the Data Storage and the matching
// leaf writes + ancestor re-sum in the sum tree (PEARL Section V-A: insertion is realised as
// priority retrieval followed by priority update; Listing 2: experiences are added to the
// Data Storage and insertion requests go to the Replay Manager).
//
// One kernel.  CTA 0 owns the tree: it writes the n leaves and then re-sums the dirty parents
// level by level (a contiguous slot range dirties a contiguous parent range on every level,
// so no sorting is needed).  The other CTAs copy rows from the dense batch to ring slots,
// HBM-bound, 16-byte granules where the row size allows.  The CTA that finishes last advances
// the cursor and the fill count, after every CTA has read them.
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

namespace {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 4;
constexpr uint32_t kChunk = kThreads * 4;  // upper bound on granules per chunk of a long row
constexpr uint32_t kTile = kThreads * 8;   // granules per tile of short rows
constexpr uint32_t kRowMode = 512;         // rows of at least this many 16-byte granules are split into chunks

// The copy is cut into tasks, numbered field by field; every copy CTA takes a contiguous range.
struct InsertPlan {
    uint32_t first_task[PRB_NUM_FIELDS + 1];  // tasks of field f: [first_task[f], first_task[f+1])
    uint32_t chunks[PRB_NUM_FIELDS];          // > 0: long rows, task = one chunk of one row; 0: short rows, task = one tile
    uint32_t chunk[PRB_NUM_FIELDS];           // granules per chunk
};

// Short rows: tile `tile` of the dense batch of field f, which may span many rows.
template <typename T>
__device__ __forceinline__ void copy_flat_tile(const PrbView& v, int f, const PrbBatch& src, uint32_t n,
                                               uint64_t cursor, uint32_t tile)
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
                       });
}

__device__ __forceinline__ void copy_task(const PrbView& v, const InsertPlan& plan, int f, const PrbBatch& src,
                                          uint32_t n, uint64_t cursor, uint32_t local)
{
    if (plan.chunks[f] > 0) {
        // long rows: one chunk of one row, contiguous on both sides
        const uint32_t W = v.field_bytes[f] / 16u;
        const uint32_t t = local / plan.chunks[f];
        const uint32_t e0 = (local - t * plan.chunks[f]) * plan.chunk[f];
        const uint32_t cnt = min(W - e0, plan.chunk[f]);
        uint64_t slot = cursor + t;
        if (slot >= v.capacity) slot -= v.capacity;
        prb_copy_span16<4>(reinterpret_cast<uint4*>(v.store[f]) + slot * W + e0,
                           reinterpret_cast<const uint4*>(src.ptr[f]) + (uint64_t)t * W + e0, cnt);
        return;
    }
    switch (v.field_vec[f]) {
    case 16: copy_flat_tile<uint4>(v, f, src, n, cursor, local); break;
    case 8: copy_flat_tile<uint2>(v, f, src, n, cursor, local); break;
    case 4: copy_flat_tile<uint32_t>(v, f, src, n, cursor, local); break;
    case 2: copy_flat_tile<uint16_t>(v, f, src, n, cursor, local); break;
    default: copy_flat_tile<uint8_t>(v, f, src, n, cursor, local); break;
    }
}

__device__ void insert_tree(const PrbView& v, uint32_t n, const float* __restrict__ prio, uint64_t cursor)
{
    const uint64_t N = v.capacity;
    const uint32_t D = v.depth, K = v.fanout, lg = v.log2_fanout;
    float* leaves = v.level[D];
    bool bad = false;
    for (uint32_t t = threadIdx.x; t < n; t += blockDim.x) {
        uint64_t slot = cursor + t;
        if (slot >= N) slot -= N;
        float p = prio[t];
        if (!prb_valid_priority(p)) { p = 0.0f; bad = true; }
        leaves[slot] = p;
    }
    if (bad) atomicOr(&v.state->status, PEARL_ST_BAD_PRIORITY);
    __syncthreads();
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
        for (uint64_t i = threadIdx.x; i < cntA + cntB; i += blockDim.x) {
            const uint64_t j = (i < cntA) ? pa0 + i : i - cntA;
            par[j] = prb_sum_children_dyn(child + j * K, K);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm)
prb_insert_kernel(PrbView v, uint32_t n, PrbBatch src, const float* __restrict__ prio, InsertPlan plan)
{
    __shared__ unsigned long long s_cursor;
    if (threadIdx.x == 0) s_cursor = v.state->cursor;
    __syncthreads();
    const uint64_t cursor = s_cursor;

    if (blockIdx.x == 0) {
        insert_tree(v, n, prio, cursor);
    } else {
        const uint32_t n_tasks = plan.first_task[PRB_NUM_FIELDS];
        const uint32_t copy_ctas = gridDim.x - 1, c = blockIdx.x - 1;
        const uint32_t t_lo = (uint32_t)(((uint64_t)c * n_tasks) / copy_ctas);
        const uint32_t t_hi = (uint32_t)(((uint64_t)(c + 1) * n_tasks) / copy_ctas);
        int f = 0;
        for (uint32_t t = t_lo; t < t_hi; ++t) {
            while (t >= plan.first_task[f + 1]) ++f;
            copy_task(v, plan, f, src, n, cursor, t - plan.first_task[f]);
        }
    }

    // The last CTA to finish publishes the new cursor and fill count.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int done = atomicAdd(&v.state->insert_ticket, 1u);
        if (done == gridDim.x - 1) {
            const uint64_t N = v.capacity;
            uint64_t c = cursor + n;
            if (c >= N) c -= N;
            v.state->cursor = c;
            const uint64_t fill = v.state->fill + n;
            v.state->fill = fill > N ? N : fill;
            v.state->insert_ticket = 0;
        }
    }
}

}  // namespace

int prb_launch_insert(const PrbView& v, uint32_t n, const PrbBatch& src, const float* d_prio, cudaStream_t s)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
            sm_count = 148;
    }
    InsertPlan plan;
    uint32_t next = 0;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        plan.first_task[f] = next;
        plan.chunks[f] = 0;
        plan.chunk[f] = 0;
        if (v.field_bytes[f] == 0 || src.ptr[f] == nullptr) continue;
        const uint32_t W = v.field_bytes[f] / v.field_vec[f];
        if (v.field_vec[f] == 16 && W >= kRowMode) {
            plan.chunks[f] = (W + kChunk - 1) / kChunk;
            plan.chunk[f] = (W + plan.chunks[f] - 1) / plan.chunks[f];
            next += n * plan.chunks[f];
        } else {
            const uint64_t total = (uint64_t)n * W;
            next += (uint32_t)((total + kTile - 1) / kTile);
        }
    }
    plan.first_task[PRB_NUM_FIELDS] = next;
    const uint32_t one_wave = (uint32_t)sm_count * kCtasPerSm - 1;     // CTA 0 is the tree CTA
    const uint32_t copy_ctas = next < one_wave ? next : one_wave;
    prb_insert_kernel<<<copy_ctas + 1, kThreads, 0, s>>>(v, n, src, d_prio, plan);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
