// Stratified priority sampling, importance-sampling weights and the gather of the sampled
// transitions, in one kernel.
//
// Priority sampling is Eq. 1 of PEARL (Section II-A) carried out as Section V-A describes it:
// "traversing the tree performing prefix sum from root to leaf".  A group of K lanes (K = the
// fanout) owns one stratum: lane j loads child j, so a child group is one 8..128-byte request;
// the left-to-right binary32 prefix sums are formed by K-1 broadcast-and-add steps (the same
// association as the stored parent), a ballot counts the prefixes the binary64 target has
// passed, and that count is the child to enter.  The read of the sampled rows is Listing 2's
// `D_storage[sampled_indices]`.  Stratification, the Philox stream and the weights follow the
// prioritized-replay reference the paper cites (Schaul et al.).
//
// CTA layout: a CTA serves G consecutive strata.  When rows are long (Atari-shaped) G = 1 and
// S CTAs share one stratum: each repeats the cheap descent (L2 reads) and copies one chunk of
// the stratum's rows, so the HBM-bound copy is spread evenly over all SMs without a second
// launch.  The CTA that finishes last normalises the weights by the batch maximum and bumps
// the sample-call counter; nothing ever waits on another CTA.
#include "prb_internal.cuh"
#include "../../include/pearl_prb.h"

namespace {

constexpr int kThreads = 256;
constexpr uint32_t kTile = kThreads * 8;   // granules per row chunk in row mode
constexpr uint32_t kRowMode = 512;         // rows of at least this many granules are split into chunks

struct SamplePlan {
    uint32_t G;                              // strata per CTA
    uint32_t S;                              // CTAs per stratum group (parts); > 1 only if G == 1
    uint32_t part_first[PRB_NUM_FIELDS];     // row mode: parts [part_first, part_first + parts) copy the chunks
    uint32_t parts[PRB_NUM_FIELDS];          // 0 = flat mode (copied by part 0)
};

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

template <int K>
__device__ __forceinline__ void descend(const PrbView& v, double x, uint32_t lane, uint32_t& leaf, float& p_leaf,
                                        unsigned& flags)
{
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const unsigned gshift = (K == 32) ? 0u : ((threadIdx.x & 31u) / K) * K;
    const unsigned gmask = (K == 32) ? FULL : ((1u << (K & 31)) - 1u);
    uint64_t g = 0;
    float c = 0.0f;
    int j = 0;
    for (uint32_t l = 1; l <= v.depth; ++l) {
        c = __ldg(v.level[l] + g * K + lane);
        float acc = __shfl_sync(FULL, c, 0, K);
#pragma unroll
        for (int i = 1; i < K; ++i) {
            const float ci = __shfl_sync(FULL, c, i, K);
            if ((int)lane >= i) acc = __fadd_rn(acc, ci);
        }
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

// Row mode: this CTA (part `part` of its stratum) copies one chunk of the sampled row of field f.
__device__ __forceinline__ void gather_row_chunk(const PrbView& v, int f, unsigned char* out, const SamplePlan& plan,
                                                 uint32_t part, uint32_t k0, uint32_t leaf)
{
    if (part < plan.part_first[f] || part >= plan.part_first[f] + plan.parts[f]) return;
    const uint32_t W = v.field_bytes[f] / 16u;
    const uint32_t e0 = (part - plan.part_first[f]) * kTile;
    const uint32_t cnt = min(W - e0, kTile);
    prb_copy_span16<8>(reinterpret_cast<uint4*>(out) + (uint64_t)k0 * W + e0,
                       reinterpret_cast<const uint4*>(v.store[f]) + (uint64_t)leaf * W + e0, cnt);
}

// Flat mode: the rows of all strata of this CTA, granule by granule.
template <typename T>
__device__ __forceinline__ void gather_flat(const PrbView& v, int f, unsigned char* out, uint32_t k0,
                                            uint32_t n_strata, const uint32_t* s_idx)
{
    const uint32_t W = v.field_bytes[f] / sizeof(T);
    const uint64_t dbase = (uint64_t)k0 * W;
    prb_copy_mapped<T>(reinterpret_cast<T*>(out), reinterpret_cast<const T*>(v.store[f]), 0u, n_strata * W,
                       [=](uint32_t e) { const uint32_t r = e / W; return (uint64_t)s_idx[r] * W + (e - r * W); },
                       [=](uint32_t e) { return dbase + e; });
}

template <int K>
__global__ void __launch_bounds__(kThreads)
prb_sample_kernel(PrbView v, uint32_t B, float beta, uint64_t seed, int32_t* __restrict__ out_idx,
                  float* __restrict__ out_w, PrbBatch dst, SamplePlan plan)
{
    constexpr int kGroups = kThreads / K;         // lane groups in a CTA
    __shared__ uint32_t s_idx[kGroups];
    __shared__ double s_wraw[kGroups];
    __shared__ unsigned long long s_calls, s_fill;
    __shared__ float s_total;
    __shared__ unsigned int s_last;

    const uint32_t tid = threadIdx.x;
    if (tid == 0) {
        s_calls = v.state->sample_calls;
        s_fill = v.state->fill;
        s_total = __ldg(v.level[0]);
    }
    __syncthreads();
    const float total32 = s_total;
    const unsigned long long calls = s_calls;
    const bool empty = (s_fill == 0) || !(total32 > 0.0f);

    const uint32_t group = blockIdx.x / plan.S;
    const uint32_t part = blockIdx.x - group * plan.S;
    const uint32_t k0 = group * plan.G;
    const uint32_t n_strata = min(plan.G, B - k0);

    if (!empty) {
        // ---- targets and descents: one K-lane group per stratum ----
        const uint32_t gi = tid / K, lane = tid % K;
        const uint32_t warp_first_group = (tid / 32u) * (32u / K);
        if (warp_first_group < n_strata) {          // warp-uniform: whole warps take part in the shuffles
            const uint32_t k = min(k0 + gi, B - 1);  // surplus groups repeat a valid stratum and write nothing
            const double total = (double)total32;
            const double seg = __ddiv_rn(total, (double)B);
            const uint32_t r0 = philox4x32_10_word0(k, 0u, (uint32_t)calls, (uint32_t)(calls >> 32),
                                                    (uint32_t)seed, (uint32_t)(seed >> 32));
            const double u = __dmul_rn((double)r0, 2.3283064365386963e-10);     // * 2^-32, exact
            double x = __dmul_rn(__dadd_rn((double)k, u), seg);
            if (x >= total) x = __longlong_as_double(__double_as_longlong(total) - 1);   // next binary64 below total
            uint32_t leaf; float p; unsigned flags = 0;
            descend<K>(v, x, lane, leaf, p, flags);
            if (lane == 0 && gi < n_strata) {
                s_idx[gi] = leaf;
                const double scaled = __ddiv_rn(__dmul_rn((double)s_fill, (double)p), total);
                const double wr = pow(scaled, -(double)beta);
                s_wraw[gi] = wr;
                if (part == 0) {
                    out_idx[k] = (int32_t)leaf;
                    v.wraw[k] = wr;
                    if (flags) atomicOr(&v.state->status, flags);
                }
            }
        }
        __syncthreads();
        if (part == 0 && tid == 0) {
            double m = s_wraw[0];
            for (uint32_t i = 1; i < n_strata; ++i) m = fmax(m, s_wraw[i]);
            atomicMax(&v.state->wmax_bits, (unsigned long long)__double_as_longlong(m));
        }

        // ---- gather: Data Storage rows of this CTA's strata ----
#pragma unroll 1
        for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
            if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0) continue;
            if (plan.parts[f] > 0) { gather_row_chunk(v, f, dst.ptr[f], plan, part, k0, s_idx[0]); continue; }
            if (part != 0) continue;
            switch (v.field_vec[f]) {
            case 16: gather_flat<uint4>(v, f, dst.ptr[f], k0, n_strata, s_idx); break;
            case 8: gather_flat<uint2>(v, f, dst.ptr[f], k0, n_strata, s_idx); break;
            case 4: gather_flat<uint32_t>(v, f, dst.ptr[f], k0, n_strata, s_idx); break;
            case 2: gather_flat<uint16_t>(v, f, dst.ptr[f], k0, n_strata, s_idx); break;
            default: gather_flat<uint8_t>(v, f, dst.ptr[f], k0, n_strata, s_idx); break;
            }
        }
    }

    // ---- the last CTA to finish normalises the weights and advances the call counter ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = (atomicAdd(&v.state->sample_ticket, 1u) == gridDim.x - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        if (empty) {
            if (tid == 0) atomicOr(&v.state->status, PEARL_ST_EMPTY);
        } else {
            const double wmax = __longlong_as_double((long long)__ldcg(&v.state->wmax_bits));
            if (out_w != nullptr)
                for (uint32_t k = tid; k < B; k += kThreads) out_w[k] = (float)__ddiv_rn(__ldcg(v.wraw + k), wmax);
        }
        __syncthreads();
        if (tid == 0) {
            if (!empty) v.state->sample_calls = calls + 1;
            v.state->wmax_bits = 0ull;
            v.state->sample_ticket = 0u;
        }
    }
}

}  // namespace

int prb_launch_sample(const PrbView& v, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w,
                      const PrbBatch& dst, cudaStream_t s)
{
    SamplePlan plan;
    plan.S = 0;
    bool row_mode = false;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        plan.part_first[f] = 0;
        plan.parts[f] = 0;
        if (dst.ptr[f] == nullptr || v.field_bytes[f] == 0) continue;
        const uint32_t W = v.field_bytes[f] / v.field_vec[f];
        if (v.field_vec[f] == 16 && W >= kRowMode) {
            row_mode = true;
            plan.part_first[f] = plan.S;
            plan.parts[f] = (W + kTile - 1) / kTile;
            plan.S += plan.parts[f];
        }
    }
    if (row_mode) {
        plan.G = 1;
    } else {
        plan.S = 1;
        plan.G = kThreads / v.fanout;
    }
    const uint32_t groups = (B + plan.G - 1) / plan.G;
    const uint32_t grid = groups * plan.S;
    switch (v.fanout) {
    case 2: prb_sample_kernel<2><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
    case 4: prb_sample_kernel<4><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
    case 8: prb_sample_kernel<8><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
    case 16: prb_sample_kernel<16><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
    default: prb_sample_kernel<32><<<grid, kThreads, 0, s>>>(v, B, beta, seed, d_idx, d_w, dst, plan); break;
    }
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
