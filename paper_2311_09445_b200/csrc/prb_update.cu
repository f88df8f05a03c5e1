// Batched priority update (PEARL Section V-A, "priority update"; on the critical path after
// the Learner, Eq. 7).  The paper applies a change Delta along the root-leaf path under a
// mutex; here the leaf is SET and the ancestors are re-summed, so the result does not depend
// on scheduling: entries are sorted by (index, batch position), the last entry of every run of
// equal indices is the winner ("last writer wins"), winners write their leaves, and then each
// level is re-summed from its children in fixed left-to-right order, deepest level first.
// Because the sorted leaf indices stay sorted after dropping low-order digits, the first entry
// of every run of equal ancestors recomputes that ancestor: no parent is written twice and no
// lock is taken.
//
// One CTA (the batch is at most a few thousand entries and the work is a chain of dependent
// L2 round trips): keys are sorted with a bitonic network in shared memory.
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

namespace {

constexpr unsigned long long kInvalidKey = ~0ull;

// p = (|delta| + eps)^alpha from IEEE basic operations only (binary64, every operation rounded
// once, no fused multiply-add), so that a CPU restatement reproduces it bit for bit:
//   y = |delta| + eps (binary32);  y = m 2^E, m in (sqrt(1/2), sqrt(2)];  t = (m-1)/(m+1);
//   ln m = 2t (1 + t^2/3 + ... + t^24/25);  z = alpha (E ln2 + ln m);  k = rint(z / ln2);
//   r = (z - k ln2_hi) - k ln2_lo;  exp r = sum_{n<=14} r^n/n!;  p = (binary32)(exp r * 2^k).
// Returns false for an invalid entry (non-finite delta, or a result outside binary32).
__device__ bool priority_pow(float delta, float eps, float alpha, float& p)
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

// keys: (index << 32) | batch position, kInvalidKey for skipped entries; vals: priority by batch position.
__global__ void __launch_bounds__(1024)
prb_update_kernel(const __grid_constant__ PrbView v, uint32_t B, uint32_t n2, const int32_t* __restrict__ idx, const float* __restrict__ val,
                  int raw, float alpha, float eps)
{
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);
    float* vals = reinterpret_cast<float*>(smem + (size_t)n2 * sizeof(unsigned long long));
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    const unsigned long long fill = v.state->fill;

    unsigned flags = 0;
    for (uint32_t b = tid; b < n2; b += nt) {
        unsigned long long key = kInvalidKey;
        if (b < B) {
            const int32_t i = idx[b];
            float p = 0.0f;
            bool ok_p;
            if (raw) { p = val[b]; ok_p = prb_valid_priority(p); }
            else ok_p = priority_pow(val[b], eps, alpha, p);
            if (i < 0 || (unsigned long long)i >= fill) flags |= PEARL_ST_BAD_INDEX;
            else if (!ok_p) flags |= PEARL_ST_BAD_PRIORITY;
            else key = ((unsigned long long)(uint32_t)i << 32) | b;
            vals[b] = p;
        }
        keys[b] = key;
    }
    if (flags) atomicOr(&v.state->status, flags);
    __syncthreads();

    // Indices that come straight from a stratified sample are already in order; sort only if needed.
    int unsorted = 0;
    for (uint32_t b = tid; b + 1 < n2; b += nt) unsorted |= (keys[b] > keys[b + 1]);
    unsorted = __syncthreads_or(unsorted);

    // bitonic sort, ascending
    for (uint32_t k = 2; unsorted && k <= n2; k <<= 1) {
        for (uint32_t j = k >> 1; j > 0; j >>= 1) {
            for (uint32_t t = tid; t < (n2 >> 1); t += nt) {
                const uint32_t lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));   // element with bit j clear
                const uint32_t hi = lo | j;
                const unsigned long long a = keys[lo], c = keys[hi];
                const bool up = (lo & k) == 0;
                if ((a > c) == up) { keys[lo] = c; keys[hi] = a; }
            }
            __syncthreads();
        }
    }

    // winners write the leaves
    float* leaves = v.level[v.depth];
    for (uint32_t s = tid; s < n2; s += nt) {
        const unsigned long long key = keys[s];
        if (key == kInvalidKey) continue;
        const uint32_t i = (uint32_t)(key >> 32);
        const bool last = (s + 1 == n2) || ((uint32_t)(keys[s + 1] >> 32) != i);
        if (last) leaves[i] = vals[(uint32_t)key];
    }
    __syncthreads();

    // re-sum the ancestors, deepest level first
    const uint32_t K = v.fanout, lg = v.log2_fanout;
    for (int l = (int)v.depth - 1; l >= 0; --l) {
        const uint32_t sh = lg * (v.depth - (uint32_t)l);
        const float* child = v.level[l + 1];
        float* par = v.level[l];
        for (uint32_t s = tid; s < n2; s += nt) {
            const unsigned long long key = keys[s];
            if (key == kInvalidKey) continue;
            const uint32_t a = (uint32_t)(key >> 32) >> sh;
            const bool first = (s == 0) || (((uint32_t)(keys[s - 1] >> 32) >> sh) != a);
            if (first) par[a] = prb_sum_children_dyn(child + (uint64_t)a * K, K);
        }
        __syncthreads();
    }
}

}  // namespace

int prb_launch_update(const PrbView& v, uint32_t B, const int32_t* d_idx, const float* d_val, int raw,
                      float alpha, float eps, cudaStream_t s)
{
    uint32_t n2 = 2;
    while (n2 < B) n2 <<= 1;
    const uint32_t threads = n2 < 64 ? 64 : (n2 > 1024 ? 1024 : n2);
    const size_t smem = (size_t)n2 * (sizeof(unsigned long long) + sizeof(float));
    if (smem > 48 * 1024) {
        static bool raised = false;
        if (!raised) {
            if (cudaFuncSetAttribute(prb_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess)
                return -1;
            raised = true;
        }
    }
    prb_update_kernel<<<1, threads, smem, s>>>(v, B, n2, d_idx, d_val, raw, alpha, eps);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
