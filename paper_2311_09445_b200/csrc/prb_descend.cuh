// The descent of one stratum by one thread, the stratified target and the Philox stream: shared by
// the sample kernels (prb_sample.cu) and the tree kernel that samples ahead (prb_update.cu).
#pragma once
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

#ifdef __CUDACC__

// Philox4x32-10 (Salmon et al., SC'11), first output word only.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

// Eq. 1's target of stratum k of B (one draw per equal segment of [0, total), Schaul et al.):
// x_k = (k + u_k) * (total / B) in binary64, two rounded operations, clamped to the binary64 just below
// total; u_k = word 0 of Philox4x32-10(counter = (k, 0, call_lo, call_hi), key = (seed_lo, seed_hi)) * 2^-32.
__device__ __forceinline__ double prb_stratum_target(uint32_t k, uint32_t B, double total, unsigned long long calls, uint64_t seed)
{
    const double seg = __ddiv_rn(total, (double)B);
    const uint32_t r0 = philox4x32_10_word0(k, 0u, (uint32_t)calls, (uint32_t)(calls >> 32), (uint32_t)seed, (uint32_t)(seed >> 32));
    const double u = __dmul_rn((double)r0, 2.3283064365386963e-10);     // * 2^-32, exact
    double x = __dmul_rn(__dadd_rn((double)k, u), seg);
    if (x >= total) x = __longlong_as_double(__double_as_longlong(total) - 1);   // next binary64 below total
    return x;
}

// The K children of one node into registers.  global: from global memory, through the read-only path (no
// kernel that walks the tree writes it); else from this CTA's shared memory.
template <int K>
__device__ __forceinline__ void prb_load_children(const float* src, bool global, float (&c)[K])
{
    if (K == 2) {
        const float2 t = global ? __ldg(reinterpret_cast<const float2*>(src)) : *reinterpret_cast<const float2*>(src);
        c[0] = t.x; c[1] = t.y;
    } else {
#pragma unroll
        for (int q = 0; q < K / 4; ++q) {
            const float4 t = global ? __ldg(reinterpret_cast<const float4*>(src) + q) : reinterpret_cast<const float4*>(src)[q];
            c[4 * q] = t.x; c[4 * q + 1] = t.y; c[4 * q + 2] = t.z; c[4 * q + 3] = t.w;
        }
    }
}

// One thread walks target x from the root to a leaf (Eq. 1 as Section V-A carries it out): per level the
// K children of the node, their left-to-right binary32 prefix sums one after another, and the first
// child whose prefix exceeds the binary64 target -- the count of prefixes the target has passed.  Levels
// 1 .. top_levels are read from s_top (level l at top_off[l]), the others from global memory.
template <int K>
__device__ __forceinline__ void prb_descend_alone(const PrbView& v, uint32_t top_levels, const uint32_t* top_off, const float* s_top,
                                                  double x, uint32_t& leaf, float& p_leaf, unsigned& flags)
{
    uint64_t g = 0;
    float chosen = 0.0f;
    for (uint32_t l = 1; l <= v.depth; ++l) {
        float c[K];
        const bool staged = l <= top_levels;
        if (!PRB_IN_BOUNDS(v, g * K + K <= v.level_alloc[l])) { flags |= PEARL_ST_INTERNAL; g = 0; }
        prb_load_children<K>(staged ? s_top + top_off[l] + (uint32_t)g * K : v.level[l] + g * K, !staged, c);
        int j = -1, last_pos = -1;
        float run = 0.0f, before_j = 0.0f, before_last = 0.0f;
#pragma unroll
        for (int q = 0; q < K; ++q) {
            const float before = run;                          // prefix q-1 (0 in front of the first child)
            run = (q == 0) ? c[0] : __fadd_rn(run, c[q]);
            if (j < 0 && !(x >= (double)run)) { j = q; before_j = before; chosen = c[q]; }
            if (c[q] > 0.0f) { last_pos = q; before_last = before; }
        }
        if (j < 0) {
            // the target has passed every prefix (possible only by binary32 rounding): last positive child
            flags |= PEARL_ST_CLAMPED;
            if (last_pos >= 0) { j = last_pos; before_j = before_last; }
            else { j = 0; before_j = 0.0f; flags |= PEARL_ST_INTERNAL; }
            chosen = 0.0f;
#pragma unroll
            for (int q = 0; q < K; ++q) if (q == j) chosen = c[q];
        }
        if (j > 0) x = __dsub_rn(x, (double)before_j);
        g = g * K + (uint64_t)j;
    }
    p_leaf = chosen;
    leaf = (uint32_t)g;
}

#endif  // __CUDACC__
