// Batched priority update (PEARL Section V-A, "priority update"; on the critical path after
// the Learner, Eq. 7).  The paper applies a change Delta along the root-leaf path under a
// mutex; here the leaf is SET and the ancestors are re-summed, so the result does not depend
// on scheduling (see prb_tree_team in prb_tree.cuh for the steps).
//
// One CTA: the batch is at most a few thousand entries and the work is a chain of dependent
// L2 round trips.
#include "prb_tree.cuh"

namespace {

__global__ void __launch_bounds__(1024)
prb_update_kernel(const __grid_constant__ PrbView v, const __grid_constant__ PrbTreeWork work)
{
    extern __shared__ __align__(16) unsigned char smem[];
    PrbTeam team;
    team.rank = threadIdx.x;
    team.size = blockDim.x;
    team.whole_cta = true;
    prb_tree_team(v, team, work, 0, v.state->fill, smem);
}

}  // namespace

int prb_launch_update(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                      float alpha, float eps, cudaStream_t s)
{
    PrbTreeWork w;
    w.B = B; w.n2 = 2; w.idx = d_idx; w.val = d_val; w.raw = raw; w.alpha = alpha; w.eps = eps;
    w.n = 0; w.prio = nullptr; w.forward = 0;
    while (w.n2 < B) w.n2 <<= 1;
    const uint32_t threads = w.n2 < 64 ? 64 : (w.n2 > 1024 ? 1024 : w.n2);
    const uint32_t fwd = prb_fwd_plan(v, &w, threads, 200 * 1024);
    const size_t smem = fwd ? fwd : prb_tree_smem_bytes(w.n2, v.fanout, threads);
    static bool big_smem = false;
    if (smem > 48 * 1024 && !big_smem) {
        if (cudaFuncSetAttribute(prb_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
            return -1;
        big_smem = true;
    }
    prb_update_kernel<<<1, threads, smem, s>>>(v, w);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
