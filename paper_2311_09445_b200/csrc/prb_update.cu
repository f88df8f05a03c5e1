// Batched priority update (PEARL Section V-A, "priority update"; on the critical path after
// the Learner, Eq. 7).  The paper applies a change Delta along the root-leaf path under a
// mutex; here the leaf is SET and the ancestors are re-summed, so the result does not depend
// on scheduling (see prb_update_team in prb_tree.cuh for the steps).
//
// One CTA, or eight CTAs of one thread-block cluster that share the deep levels: the batch is at most
// a few thousand entries and the work is a chain of dependent L2 round trips, one per level below
// the top of the tree, which is staged in shared memory.
#include "prb_tree.cuh"

namespace {

__global__ void __launch_bounds__(1024)
prb_update_kernel(const __grid_constant__ PrbView v, uint32_t B, uint32_t n2, const int32_t* __restrict__ idx,
                  const float* __restrict__ val, int raw, float alpha, float eps, uint32_t stale,
                  uint32_t ins_n, const float* __restrict__ ins_prio, uint32_t ticket_total)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned long long s_cursor, s_fill;
    PrbTeam team;
    team.rank = threadIdx.x;
    team.size = blockDim.x;
    team.whole_cta = true;
    team.part = blockIdx.x;          // CTAs of one cluster share the work (one CTA: the whole of it)
    team.parts = gridDim.x;
    PrbTop top;
    if (v.top_levels) top.mem = reinterpret_cast<float*>(smem + prb_update_smem_bytes(n2));
    if (team.part == 0) prb_top_begin(v, top, team.rank, team.size);
    unsigned long long fill, cursor = 0;
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
        if (threadIdx.x == 0) prb_publish_if_last(v, ins_n, cursor, fill, ticket_total);
    } else {
        fill = v.state->fill;
        if (stale) cursor = v.state->cursor;
    }
    prb_update_team(v, team, B, n2, idx, val, raw, alpha, eps, fill, smem, ins_n, ins_prio, cursor, pre, stale, top);
}

// Priority retrieval: one thread per entry.
__global__ void prb_get_priorities_kernel(const __grid_constant__ PrbView v, uint32_t B, const int32_t* __restrict__ idx,
                                          float* __restrict__ out)
{
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int32_t i = idx[b];
    if (i < 0 || (unsigned long long)i >= v.state->fill) { out[b] = 0.0f; atomicOr(&v.state->status, PEARL_ST_BAD_INDEX); return; }
    out[b] = __ldcg(v.level[v.depth] + i);
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

int prb_launch_update(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                      float alpha, float eps, cudaStream_t s, uint32_t stale,
                      uint32_t ins_n, const float* ins_prio, uint32_t ticket_total)
{
    if (ins_n && B > PEARL_UPDATE_SUBBATCH) return -1;
    static bool big_smem[kPrbMaxDevices];
    const int dev = prb_current_device();
    if (!big_smem[dev]) {
        if (cudaFuncSetAttribute(prb_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(prb_update_smem_bytes(PEARL_UPDATE_SUBBATCH) + kPrbTopFloats * sizeof(float))) != cudaSuccess)
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
        cfg.dynamicSmemBytes = prb_update_smem_bytes(n2) + v.top_floats * sizeof(float);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = ctas;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, prb_update_kernel, v, b, n2, d_idx + first, d_val + first, raw, alpha, eps, stale,
                               ins_n, ins_prio, ticket_total) != cudaSuccess)
            return -1;
        ++launches;
    }
    return launches;
}
