// Host side of libpearl_prb: handle, device-memory layout, argument checks and the C ABI.
// Every step of the replay path runs in the kernels of prb_insert.cu / prb_sample.cu /
// prb_update.cu; this file only places memory and enqueues.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "../../include/pearl_prb.h"
#include "prb_internal.cuh"

namespace {

constexpr uint64_t kAlign = 256;

inline uint64_t align_up(uint64_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

inline uint32_t granule_of(uint32_t bytes)
{
    uint32_t g = 16;
    while (g > 1 && bytes % g != 0) g >>= 1;
    return g;
}

// Offsets (bytes from the slab base) of every region of a buffer.
struct Layout {
    uint32_t depth;
    uint64_t level_alloc[PRB_MAX_LEVELS];
    uint64_t off_state;
    uint64_t off_level[PRB_MAX_LEVELS];
    uint64_t off_min;                         // the min-tree's levels 0 .. depth-1, laid out like the sum tree's (0: no min-tree)
    uint64_t off_wraw;
    uint64_t off_handoff[kPrbHandoffs];
    uint64_t off_zero_end;                    // [0, off_zero_end) is zeroed at creation
    uint64_t off_store[PRB_NUM_FIELDS];
    uint64_t off_stage_in[PRB_NUM_FIELDS];    // staging of the *_host calls: inputs ...
    uint64_t off_stage_prio, off_stage_idx, off_stage_td;
    uint64_t off_stage_out[PRB_NUM_FIELDS];   // ... and outputs
    uint64_t off_stage_out_idx, off_stage_out_w;
    uint32_t field_bytes[PRB_NUM_FIELDS];     // a row of the store
    uint32_t out_bytes[PRB_NUM_FIELDS];       // a row as a sample hands it out
    uint32_t field_pitch[PRB_NUM_FIELDS];     // bytes from one slot's field to the next slot's (see PrbView)
    uint32_t stack;                           // frame-deduplicated layout: frames per observation (0: plain layout)
    uint64_t total;
};

bool valid_fanout(uint32_t k) { return k == 2 || k == 4 || k == 8 || k == 16 || k == 32; }

bool make_layout(uint64_t capacity, uint32_t fanout, const pearl_layout_t* lay, uint32_t max_batch, Layout* L, uint32_t stack = 0,
                 uint32_t options = 0)
{
    if (options & ~PEARL_OPT_MIN_TREE) return false;
    if (!lay || !valid_fanout(fanout) || capacity < 1 || capacity > (1ull << 30) || max_batch < 1 ||
        max_batch > (1u << 20))
        return false;
    if (stack > 16 || (stack && (lay->obs_bytes == 0 || capacity <= stack || (uint64_t)lay->obs_bytes * stack > 0xFFFFFFFFull)))
        return false;
    L->stack = stack;
    uint32_t D = 1;
    uint64_t span = fanout;
    while (span < capacity) { span *= fanout; ++D; }
    if (D >= PRB_MAX_LEVELS) return false;
    L->depth = D;
    uint64_t nodes[PRB_MAX_LEVELS];
    nodes[D] = capacity;
    for (int l = (int)D - 1; l >= 0; --l) nodes[l] = (nodes[l + 1] + fanout - 1) / fanout;
    for (uint32_t l = 0; l <= D; ++l)
        L->level_alloc[l] = (l == 0) ? 1 : (nodes[l] + fanout - 1) / fanout * fanout;

    // (with frames, lay->obs_bytes is the size of one frame)
    L->field_bytes[F_OBS] = lay->obs_bytes;
    L->field_bytes[F_NEXT_OBS] = stack ? 0 : lay->obs_bytes;
    L->field_bytes[F_ACT] = lay->act_bytes;
    L->field_bytes[F_REW] = 4;
    L->field_bytes[F_DONE] = 1;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) L->out_bytes[f] = L->field_bytes[f];
    if (stack) L->out_bytes[F_OBS] = L->out_bytes[F_NEXT_OBS] = lay->obs_bytes * stack;
    // A field that is copied granule by granule (anything but rows of at least 512 16-byte granules,
    // which move as bulk copies) is indexed with 32-bit granule numbers within one batch.
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        const uint32_t g = L->field_bytes[f] ? granule_of(L->field_bytes[f]) : 1;
        const uint64_t W = L->field_bytes[f] / g;
        if (!(g == 16 && W >= 512) && (uint64_t)max_batch * W >= (1ull << 32)) return false;
    }

    uint64_t at = 0;
    L->off_state = at; at = align_up(at + sizeof(PrbState));
    for (uint32_t l = 0; l <= D; ++l) { L->off_level[l] = at; at = align_up(at + L->level_alloc[l] * sizeof(float)); }
    L->off_min = 0;
    if (options & PEARL_OPT_MIN_TREE) { L->off_min = at; at = align_up(at + (L->off_level[D] - L->off_level[0])); }
    L->off_wraw = at; at = align_up(at + (uint64_t)max_batch * sizeof(double));
    for (uint32_t j = 0; j < kPrbHandoffs; ++j) { L->off_handoff[j] = at; at = align_up(at + prb_handoff_bytes(max_batch)); }
    L->off_zero_end = at;
    // Short rows (every field below the bulk-copy threshold, the record at most 512 bytes, no frames): one
    // padded record per transition, fields at offsets aligned to their copy granules, the record a multiple
    // of 64 bytes.  Otherwise one array per field.
    uint64_t record = 0;
    bool records = stack == 0;
    uint64_t field_off[PRB_NUM_FIELDS];
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        const uint32_t g = L->field_bytes[f] ? granule_of(L->field_bytes[f]) : 1;
        if (g == 16 && L->field_bytes[f] / g >= 512) records = false;
        record = (record + g - 1) / g * g;
        field_off[f] = record;
        record += L->field_bytes[f];
    }
    record = (record + 63) / 64 * 64;
    if (record > 512) records = false;
    if (records) {
        for (int f = 0; f < PRB_NUM_FIELDS; ++f) { L->off_store[f] = at + field_off[f]; L->field_pitch[f] = (uint32_t)record; }
        at = align_up(at + capacity * record);
    } else {
        for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
            L->off_store[f] = at;
            L->field_pitch[f] = L->field_bytes[f];
            at = align_up(at + capacity * L->field_bytes[f]);
        }
    }
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) { L->off_stage_in[f] = at; at = align_up(at + (uint64_t)max_batch * L->field_bytes[f]); }
    L->off_stage_prio = at; at = align_up(at + (uint64_t)max_batch * 4);
    L->off_stage_idx = at; at = align_up(at + (uint64_t)max_batch * 4);
    L->off_stage_td = at; at = align_up(at + (uint64_t)max_batch * 4);
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) { L->off_stage_out[f] = at; at = align_up(at + (uint64_t)max_batch * L->out_bytes[f]); }
    L->off_stage_out_idx = at; at = align_up(at + (uint64_t)max_batch * 4);
    L->off_stage_out_w = at; at = align_up(at + (uint64_t)max_batch * 4);
    L->total = at;
    return true;
}

}  // namespace

namespace {
void destroy_fork(PrbFork& f)
{
    if (f.fork) cudaEventDestroy(f.fork);
    if (f.join) cudaEventDestroy(f.join);
    if (f.side) cudaStreamDestroy(f.side);
    f = PrbFork{nullptr, nullptr, nullptr};
    cudaGetLastError();
}
}  // namespace

constexpr uint64_t kPackBytes = 256 * 1024;

struct pearl_prb {
    Layout lay;
    PrbView view;
    unsigned char* base;
    bool owns_slab;
    int device;
    cudaStream_t stream;
    uint32_t max_batch;
    uint64_t launches;
    PrbFork fork = PrbFork{nullptr, nullptr, nullptr};   // side stream and events of pearl_prb_update_insert with long rows
    // pearl_prb_sample_streamed: one stream and one event per sub-batch, created with the handle
    PrbSubStreams subs = PrbSubStreams{{nullptr, nullptr, nullptr, nullptr}, {nullptr, nullptr, nullptr, nullptr}, nullptr};
    uint32_t streamed_subs = 0;          // sub-batches of the last streamed call (0: none yet)
    // Small batches of the *_host calls travel packed: all arrays of a call in one pinned buffer, one
    // copy each way (2 x kPackBytes of pinned host memory; nullptr: every array is copied by itself).
    unsigned char* pin = nullptr;
    unsigned char* pin_dev = nullptr;    // the same memory as the device sees it (mapped; nullptr if it cannot be mapped)
    cudaEvent_t pin_read = nullptr;      // the last host-to-device copy out of `pin` has been made
    // A sample of long rows inside a stream capture is two kernels: the descents on fork.side, the row
    // copy on the caller's stream (see sample_two_kernels below).
    cudaEvent_t desc_done = nullptr;             // the descents of the running two-kernel sample are done
    cudaEvent_t relay_done = nullptr;            // ... and so is the relay behind them (see sample_two_kernels)
    cudaEvent_t gather_done[kPrbHandoffs] = {};   // the row copy that read hand-off area j is done
    unsigned long long gather_capture[kPrbHandoffs] = {};    // the capture gather_done[j] was last recorded in (0: none)
    unsigned long long side_capture = 0;         // the capture fork.side has last been made part of (0: none)
    bool main_touched = true;                    // since fork.side last waited for the caller's stream, that stream
                                                 // has been given work that reads or writes the tree or the state
    uint32_t handoff_next = 0;
    unsigned long long after_forked_tree = 0;    // the capture in which the last call was an update + insertion whose tree kernel ran on fork.side (0: it was not)
    unsigned long long main_last_gather = 0;     // the capture in which the last kernel given to the caller's stream was such a row copy (0: it was not)
    ~pearl_prb()
    {
        destroy_fork(fork);
        for (uint32_t i = 0; i < kPrbMaxSubBatches; ++i) {
            if (subs.done[i]) cudaEventDestroy(subs.done[i]);
            if (subs.stream[i]) cudaStreamDestroy(subs.stream[i]);
        }
        if (subs.fork) cudaEventDestroy(subs.fork);
        if (pin_read) cudaEventDestroy(pin_read);
        if (desc_done) cudaEventDestroy(desc_done);
        if (relay_done) cudaEventDestroy(relay_done);
        for (uint32_t j = 0; j < kPrbHandoffs; ++j) if (gather_done[j]) cudaEventDestroy(gather_done[j]);
        if (pin) cudaFreeHost(pin);
        cudaGetLastError();
    }
};

namespace {

inline bool misaligned(const void* p, uint32_t granule) { return ((uintptr_t)p & (granule - 1)) != 0; }

// (outputs: the pointers are a sample's outputs, whose rows are out_bytes long; else an insertion's inputs)
int check_batch_ptrs(const pearl_prb* h, const void* const ptrs[PRB_NUM_FIELDS], bool outputs = false)
{
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        const uint32_t row = outputs ? h->lay.out_bytes[f] : h->view.field_bytes[f];
        if (ptrs[f] && row && misaligned(ptrs[f], h->view.field_vec[f])) return PEARL_ERR_ALIGN;
    }
    return PEARL_OK;
}

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(true)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline unsigned char* at(const pearl_prb* h, uint64_t off) { return h->base + off; }

// The identifier of the stream capture the handle's stream is part of; 0 if it is not capturing.
unsigned long long capture_of(cudaStream_t s)
{
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    unsigned long long id = 0;
    if (cudaStreamGetCaptureInfo(s, &st, &id) != cudaSuccess) { cudaGetLastError(); return 0; }
    return st == cudaStreamCaptureStatusActive ? (id ? id : 1ull) : 0ull;
}

// A sample of long rows as two kernels, inside a stream capture (a captured step is replayed many
// times, and there the time of the call is what counts, not the time of its host code).
// The descents -- chains of dependent L2 reads that keep HBM idle -- read and write nothing of the
// caller's: the tree, the state and a hand-off area of the slab (leaf indices and priorities; the
// weights are formed by the row copy's spare warps).  So they are launched on the handle's
// second stream, where they are ordered after the tree work that stream already holds (the tree kernel
// of the update + insertion before them) but not after the rows the caller's stream is still copying:
// in a captured step they run beside the insertion's row copy, and in back-to-back samples beside the
// row copy of the sample before.  The caller's stream then waits for them and runs the indexed row
// copy, which also hands indices and weights to the caller.  Everything the caller can see is written
// on the caller's stream, in order.  The second stream waits for the caller's stream first whenever
// that stream has been given tree or state work since (main_touched), and once at the start of every
// capture; the hand-off areas are used in turn, an area not before the row copy that read it last.
int sample_two_kernels(pearl_prb* h, unsigned long long capture, uint32_t B, float beta, uint64_t seed, int32_t* d_idx,
                       float* d_w, const PrbBatch& dst, int uniform, int buffer_norm)
{
    cudaStream_t main = h->stream, side = h->fork.side;
    const uint32_t j = h->handoff_next;
    if (h->side_capture != capture || h->main_touched) {
        if (cudaEventRecord(h->fork.fork, main) != cudaSuccess || cudaStreamWaitEvent(side, h->fork.fork, 0) != cudaSuccess) return -1;
        h->side_capture = capture;
        h->main_touched = false;
    }
    if (h->gather_capture[j] == capture && cudaStreamWaitEvent(side, h->gather_done[j], 0) != cudaSuccess) return -1;
    unsigned char* area = h->view.handoff[j];
    const int k1 = prb_launch_descend(h->view, B, seed, area, side, uniform, buffer_norm);
    if (k1 < 0) return -1;
    // The row copy is launched as a programmatic dependent of what precedes it on the caller's stream, and an
    // event wait joins the descents to that: it could then start before the descents' writes are flushed.  So
    // the event it waits for is recorded behind a relay -- an empty kernel on a third stream that depends on
    // the descents in full -- and not behind the descents themselves; the next call's descents, on the
    // second stream, do not wait for the relay.
    cudaStream_t third = h->subs.stream[0];
    if (cudaEventRecord(h->desc_done, side) != cudaSuccess || cudaStreamWaitEvent(third, h->desc_done, 0) != cudaSuccess) return -1;
    if (prb_launch_relay(third) < 0) return -1;
    if (cudaEventRecord(h->relay_done, third) != cudaSuccess || cudaStreamWaitEvent(main, h->relay_done, 0) != cudaSuccess) return -1;
    const int k2 = prb_launch_gather(h->view, B, beta, area, d_idx, d_w, dst, main, h->main_last_gather == capture);
    if (k2 < 0) return -1;
    if (cudaEventRecord(h->gather_done[j], main) != cudaSuccess) return -1;
    h->gather_capture[j] = capture;
    h->handoff_next = (j + 1u) % kPrbHandoffs;
    h->main_last_gather = capture;
    h->after_forked_tree = 0;
    return k1 + k2 + 1;
}

bool finite_nonneg(float x) { return isfinite(x) && x >= 0.0f; }

}  // namespace

extern "C" {

uint64_t pearl_prb_slab_bytes(uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout, uint32_t max_batch)
{
    Layout L;
    if (!make_layout(capacity, fanout, layout, max_batch, &L)) return 0;
    return L.total;
}

uint64_t pearl_prb_slab_bytes_frames(uint64_t capacity, uint32_t fanout, uint32_t frame_bytes, uint32_t stack, uint32_t act_bytes,
                                     uint32_t max_batch)
{
    Layout L;
    const pearl_layout_t lay = { frame_bytes, act_bytes };
    if (stack < 1 || !make_layout(capacity, fanout, &lay, max_batch, &L, stack)) return 0;
    return L.total;
}

uint64_t pearl_prb_slab_bytes_opts(uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout, uint32_t frame_stack,
                                   uint32_t options, uint32_t max_batch)
{
    Layout L;
    if (!make_layout(capacity, fanout, layout, max_batch, &L, frame_stack, options)) return 0;
    return L.total;
}

static int create_common(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout, uint32_t stack,
                         uint32_t max_batch, int device, void* cuda_stream, void* slab, uint64_t slab_bytes, uint32_t options = 0);

int pearl_prb_create_opts(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout, uint32_t frame_stack,
                          uint32_t options, uint32_t max_batch, int device, void* cuda_stream, void* slab, uint64_t slab_bytes)
{
    return create_common(out, capacity, fanout, layout, frame_stack, max_batch, device, cuda_stream, slab, slab_bytes, options);
}

int pearl_prb_create(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout,
                     uint32_t max_batch, int device, void* cuda_stream, void* slab, uint64_t slab_bytes)
{
    return create_common(out, capacity, fanout, layout, 0, max_batch, device, cuda_stream, slab, slab_bytes);
}

int pearl_prb_create_frames(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, uint32_t frame_bytes, uint32_t stack,
                            uint32_t act_bytes, uint32_t max_batch, int device, void* cuda_stream, void* slab, uint64_t slab_bytes)
{
    const pearl_layout_t lay = { frame_bytes, act_bytes };
    if (stack < 1) return PEARL_ERR_BAD_ARG;
    return create_common(out, capacity, fanout, &lay, stack, max_batch, device, cuda_stream, slab, slab_bytes);
}

static int create_common(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout, uint32_t stack,
                         uint32_t max_batch, int device, void* cuda_stream, void* slab, uint64_t slab_bytes, uint32_t options)
{
    if (!out || !layout) return PEARL_ERR_NULL;
    if (!valid_fanout(fanout)) return PEARL_ERR_BAD_FANOUT;
    if (max_batch < 1 || max_batch > (1u << 20)) return PEARL_ERR_BAD_BATCH;
    Layout L;
    if (!make_layout(capacity, fanout, layout, max_batch, &L, stack, options)) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return PEARL_ERR_CUDA;

    pearl_prb* h = new (std::nothrow) pearl_prb();
    if (!h) return PEARL_ERR_OOM;
    h->lay = L;
    h->device = device;
    h->stream = (cudaStream_t)cuda_stream;
    h->max_batch = max_batch;
    h->launches = 0;
    if (cudaStreamCreateWithFlags(&h->fork.side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->fork.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->fork.join, cudaEventDisableTiming) != cudaSuccess) {
        delete h;
        return PEARL_ERR_CUDA;
    }
    for (uint32_t i = 0; i < kPrbMaxSubBatches; ++i) {
        if (cudaStreamCreateWithFlags(&h->subs.stream[i], cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->subs.done[i], cudaEventDisableTiming) != cudaSuccess) {
            delete h;
            return PEARL_ERR_CUDA;
        }
    }
    if (cudaEventCreateWithFlags(&h->subs.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->desc_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->relay_done, cudaEventDisableTiming) != cudaSuccess) { delete h; return PEARL_ERR_CUDA; }
    for (uint32_t j = 0; j < kPrbHandoffs; ++j)
        if (cudaEventCreateWithFlags(&h->gather_done[j], cudaEventDisableTiming) != cudaSuccess) { delete h; return PEARL_ERR_CUDA; }
    if (cudaHostAlloc((void**)&h->pin, 2 * kPackBytes, cudaHostAllocMapped) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->pin_read, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();                 // (not fatal: the host calls then copy array by array)
        if (h->pin) cudaFreeHost(h->pin);
        h->pin = nullptr;
    }
    if (h->pin && cudaHostGetDevicePointer((void**)&h->pin_dev, h->pin, 0) != cudaSuccess) { cudaGetLastError(); h->pin_dev = nullptr; }
    if (slab) {
        if (slab_bytes < L.total || ((uintptr_t)slab & (kAlign - 1))) { delete h; return slab_bytes < L.total ? PEARL_ERR_OOM : PEARL_ERR_ALIGN; }
        h->base = (unsigned char*)slab;
        h->owns_slab = false;
    } else {
        void* p = nullptr;
        if (cudaMalloc(&p, L.total) != cudaSuccess) { cudaGetLastError(); delete h; return PEARL_ERR_OOM; }
        h->base = (unsigned char*)p;
        h->owns_slab = true;
    }
    if (cudaMemsetAsync(h->base, 0, L.off_zero_end, h->stream) != cudaSuccess) {
        if (h->owns_slab) cudaFree(h->base);
        delete h;
        return PEARL_ERR_CUDA;
    }
    PrbView& v = h->view;
    memset(&v, 0, sizeof(v));
    v.state = (PrbState*)at(h, L.off_state);
    if (cudaMemsetAsync(&v.state->pmin_bits, 0xFF, sizeof(unsigned long long), h->stream) != cudaSuccess) {
        if (h->owns_slab) cudaFree(h->base);
        delete h;
        return PEARL_ERR_CUDA;
    }
    for (uint32_t l = 0; l <= L.depth; ++l) {
        v.level[l] = (float*)at(h, L.off_level[l]);
        v.level_alloc[l] = (uint32_t)L.level_alloc[l];
    }
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        v.store[f] = at(h, L.off_store[f]);
        v.field_bytes[f] = L.field_bytes[f];
        v.field_pitch[f] = L.field_pitch[f];
        v.field_vec[f] = L.field_bytes[f] ? granule_of(L.field_bytes[f]) : 1;
    }
    v.min_off = L.off_min ? (L.off_min - L.off_level[0]) / sizeof(float) : 0;
    v.stack = L.stack;
    if (v.stack) v.field_vec[F_NEXT_OBS] = v.field_vec[F_OBS];      // rebuilt from the same frames
    v.wraw = (double*)at(h, L.off_wraw);
    for (uint32_t j = 0; j < kPrbHandoffs; ++j) v.handoff[j] = at(h, L.off_handoff[j]);
    v.capacity = capacity;
    v.fanout = fanout;
    v.log2_fanout = 0;
    while ((1u << v.log2_fanout) < fanout) ++v.log2_fanout;
    v.depth = L.depth;
    v.max_batch = max_batch;
    // the levels that fit a CTA's staging area (the leaves are never staged)
    v.top_levels = 0;
    v.top_floats = 0;
    for (uint32_t l = 1; l < L.depth; ++l) {
        const uint64_t end = (uint64_t)(v.level[l] - v.level[1]) + v.level_alloc[l];
        if (end > kPrbTopFloats) break;
        v.top_levels = l;
        v.top_off[l] = (uint32_t)(v.level[l] - v.level[1]);
        v.top_floats = (uint32_t)((end + 3) / 4 * 4);
    }
    *out = h;
    return PEARL_OK;
}

int pearl_prb_destroy(pearl_prb_t* h)
{
    if (!h) return PEARL_ERR_NULL;
    DeviceGuard guard(h->device);
    int rc = PEARL_OK;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) rc = PEARL_ERR_CUDA;
    if (h->fork.side && cudaStreamSynchronize(h->fork.side) != cudaSuccess) rc = PEARL_ERR_CUDA;
    for (uint32_t i = 0; i < kPrbMaxSubBatches; ++i)
        if (h->subs.stream[i] && cudaStreamSynchronize(h->subs.stream[i]) != cudaSuccess) rc = PEARL_ERR_CUDA;
    destroy_fork(h->fork);
    if (h->owns_slab && cudaFree(h->base) != cudaSuccess) rc = PEARL_ERR_CUDA;
    delete h;
    return rc;
}

int pearl_prb_insert(pearl_prb_t* h, uint32_t n, const void* d_obs, const void* d_act, const float* d_rew,
                     const void* d_next_obs, const uint8_t* d_done, const float* d_prio)
{
    if (!h) return PEARL_ERR_NULL;
    if (n == 0 || n > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (n > h->view.capacity) return PEARL_ERR_TOO_MANY;
    if (h->view.stack && (d_next_obs || !d_done)) return PEARL_ERR_BAD_ARG;     // one frame per transition (d_obs); markers live in d_done
    const void* ptrs[PRB_NUM_FIELDS] = { d_obs, d_next_obs, d_act, d_rew, d_done };
    int rc = check_batch_ptrs(h, ptrs);
    if (rc != PEARL_OK) return rc;
    if (d_prio && misaligned(d_prio, 4)) return PEARL_ERR_ALIGN;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    PrbBatch b;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) b.ptr[f] = (unsigned char*)ptrs[f];
    const int k = prb_launch_insert(h->view, n, b, d_prio, h->stream);
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    return PEARL_OK;
}

static int check_sample_args(const pearl_prb_t* h, uint32_t B, float beta, const int32_t* d_idx, const float* d_w,
                             const void* const ptrs[PRB_NUM_FIELDS])
{
    if (!h || !d_idx) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (!finite_nonneg(beta)) return PEARL_ERR_BAD_ARG;
    int rc = check_batch_ptrs(h, ptrs, true);
    if (rc != PEARL_OK) return rc;
    if (misaligned(d_idx, 4) || (d_w && misaligned(d_w, 4))) return PEARL_ERR_ALIGN;
    return PEARL_OK;
}

static int sample_common(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w, void* d_obs,
                         void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done, int uniform, uint32_t n_sub = 1,
                         int buffer_norm = 0)
{
    const void* ptrs[PRB_NUM_FIELDS] = { d_obs, d_next_obs, d_act, d_rew, d_done };
    int rc = check_sample_args(h, B, beta, d_idx, d_w, ptrs);
    if (rc != PEARL_OK) return rc;
    if (n_sub < 1 || n_sub > kPrbMaxSubBatches || n_sub > B) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    PrbBatch b;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) b.ptr[f] = (unsigned char*)ptrs[f];
    // Inside a capture a sample of long rows is two kernels (sample_two_kernels above) -- unless the call
    // before it was an update + insertion whose tree kernel the descents would have to follow: that kernel
    // ends with the row copy beside it, nothing is left for the descents to hide behind, and the one-kernel
    // form, whose descents are the prologue of the copy, is shorter by a launch.
    const unsigned long long capture = (n_sub == 1 && prb_sample_has_long_rows(h->view, b)) ? capture_of(h->stream) : 0ull;
    int k;
    if (capture && h->after_forked_tree != capture) {
        k = sample_two_kernels(h, capture, B, beta, seed, d_idx, d_w, b, uniform, buffer_norm);
    } else {
        k = prb_launch_sample(h->view, B, beta, seed, d_idx, d_w, b, h->stream, uniform, n_sub, &h->subs, buffer_norm);
        h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    }
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    if (n_sub > 1) h->streamed_subs = n_sub;
    return PEARL_OK;
}

int pearl_prb_sample(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w, void* d_obs,
                     void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    return sample_common(h, B, beta, seed, d_idx, d_w, d_obs, d_act, d_rew, d_next_obs, d_done, 0);
}

int pearl_prb_sample_buffer_norm(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w, void* d_obs,
                                 void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    return sample_common(h, B, beta, seed, d_idx, d_w, d_obs, d_act, d_rew, d_next_obs, d_done, 0, 1, 1);
}

int pearl_prb_sample_streamed(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, uint32_t n_sub, int32_t* d_idx, float* d_w,
                              void* d_obs, void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    return sample_common(h, B, beta, seed, d_idx, d_w, d_obs, d_act, d_rew, d_next_obs, d_done, 0, n_sub);
}

int pearl_prb_wait_sub_batch(pearl_prb_t* h, uint32_t sub_batch, void* cuda_stream)
{
    if (!h) return PEARL_ERR_NULL;
    if (sub_batch >= h->streamed_subs) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    return cudaStreamWaitEvent((cudaStream_t)cuda_stream, h->subs.done[sub_batch], 0) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int pearl_prb_sample_uniform(pearl_prb_t* h, uint32_t B, uint64_t seed, int32_t* d_idx, float* d_w, void* d_obs,
                             void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    if (h && h->view.stack) return PEARL_ERR_BAD_ARG;      // (a uniform draw could name a marker or a slot without history)
    return sample_common(h, B, 0.0f, seed, d_idx, d_w, d_obs, d_act, d_rew, d_next_obs, d_done, 1);
}

static int update_common(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_val, int raw, float alpha,
                         float eps, uint32_t stale = 0)
{
    if (!h || !d_idx || !d_val) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (!raw && (!finite_nonneg(alpha) || !finite_nonneg(eps))) return PEARL_ERR_BAD_ARG;
    if (misaligned(d_idx, 4) || misaligned(d_val, 4)) return PEARL_ERR_ALIGN;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    if (stale > h->view.capacity) return PEARL_ERR_BAD_ARG;
    const int k = prb_launch_update(h->view, B, d_idx, d_val, raw, alpha, eps, h->stream, stale);
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    return PEARL_OK;
}

int pearl_prb_update(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_td, float alpha, float eps)
{
    return update_common(h, B, d_idx, d_td, 0, alpha, eps);
}

int pearl_prb_update_priorities(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_prio)
{
    return update_common(h, B, d_idx, d_prio, 1, 0.0f, 0.0f);
}

int pearl_prb_update_delta(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_delta)
{
    return update_common(h, B, d_idx, d_delta, 2, 0.0f, 0.0f);
}

int pearl_prb_update_after_insert(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_td, float alpha,
                                  float eps, uint32_t inserted)
{
    return update_common(h, B, d_idx, d_td, 0, alpha, eps, inserted);
}

int pearl_prb_get_priorities(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, float* d_out)
{
    if (!h || !d_idx || !d_out) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (misaligned(d_idx, 4) || misaligned(d_out, 4)) return PEARL_ERR_ALIGN;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    const int k = prb_launch_get_priorities(h->view, B, d_idx, d_out, h->stream);
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    return PEARL_OK;
}

static int check_update_insert_args(const pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_td, float alpha,
                                    float eps, uint32_t n, const void* const ptrs[PRB_NUM_FIELDS], const float* d_prio)
{
    if (!h || !d_idx || !d_td) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (n == 0 || n > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (n > h->view.capacity) return PEARL_ERR_TOO_MANY;
    if (!finite_nonneg(alpha) || !finite_nonneg(eps)) return PEARL_ERR_BAD_ARG;
    if (h->view.stack && (ptrs[F_NEXT_OBS] || !ptrs[F_DONE])) return PEARL_ERR_BAD_ARG;
    int rc = check_batch_ptrs(h, ptrs);
    if (rc != PEARL_OK) return rc;
    if ((d_prio && misaligned(d_prio, 4)) || misaligned(d_idx, 4) || misaligned(d_td, 4)) return PEARL_ERR_ALIGN;
    return PEARL_OK;
}

int pearl_prb_update_insert(pearl_prb_t* h, uint32_t B, const int32_t* d_idx, const float* d_td, float alpha, float eps,
                            uint32_t n, const void* d_obs, const void* d_act, const float* d_rew, const void* d_next_obs,
                            const uint8_t* d_done, const float* d_prio)
{
    const void* ptrs[PRB_NUM_FIELDS] = { d_obs, d_next_obs, d_act, d_rew, d_done };
    int rc = check_update_insert_args(h, B, d_idx, d_td, alpha, eps, n, ptrs, d_prio);
    if (rc != PEARL_OK) return rc;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    PrbBatch b;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) b.ptr[f] = (unsigned char*)ptrs[f];
    bool forked = false;
    const int k = prb_launch_insert(h->view, n, b, d_prio, h->stream, B, d_idx, d_td, 0, alpha, eps, &h->fork, &forked);
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    if (forked) {
        // the tree work went to the second stream, which waited for this one first; what this stream got
        // is the row copy, which touches neither the tree nor the state the descents read
        h->side_capture = capture_of(h->stream);
        h->main_touched = false;
        h->main_last_gather = 0;
        h->after_forked_tree = h->side_capture;
    } else {
        h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    }
    return PEARL_OK;
}

int pearl_prb_step(pearl_prb_t* h, uint32_t B_upd, const int32_t* d_upd_idx, const float* d_td, float alpha, float eps,
                   uint32_t n, const void* d_new_obs, const void* d_new_act, const float* d_new_rew, const void* d_new_next_obs,
                   const uint8_t* d_new_done, const float* d_new_prio, uint32_t B, float beta, uint64_t seed, int32_t* d_idx,
                   float* d_w, void* d_obs, void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    const void* in[PRB_NUM_FIELDS] = { d_new_obs, d_new_next_obs, d_new_act, d_new_rew, d_new_done };
    const void* out[PRB_NUM_FIELDS] = { d_obs, d_next_obs, d_act, d_rew, d_done };
    // (n == 0: an iteration without new transitions -- update, then sample)
    int rc = check_update_insert_args(h, B_upd, d_upd_idx, d_td, alpha, eps, n ? n : 1u, in, d_new_prio);
    if (rc != PEARL_OK) return rc;
    rc = check_sample_args(h, B, beta, d_idx, d_w, out);
    if (rc != PEARL_OK) return rc;
    // (both calls' arguments have been checked: nothing is enqueued unless both go through)
    rc = n ? pearl_prb_update_insert(h, B_upd, d_upd_idx, d_td, alpha, eps, n, d_new_obs, d_new_act, d_new_rew, d_new_next_obs,
                                     d_new_done, d_new_prio)
           : pearl_prb_update(h, B_upd, d_upd_idx, d_td, alpha, eps);
    if (rc != PEARL_OK) return rc;
    return pearl_prb_sample(h, B, beta, seed, d_idx, d_w, d_obs, d_act, d_rew, d_next_obs, d_done);
}

// ---- host-buffer forms ---------------------------------------------------------------------

namespace {

// Offsets of up to seven arrays packed one after another, each start 16-byte aligned.
struct Packing {
    uint64_t off[PRB_NUM_FIELDS + 3];
    uint64_t bytes[PRB_NUM_FIELDS + 3];
    uint64_t total = 0;
    void add(int slot, uint64_t nbytes)
    {
        off[slot] = total;
        bytes[slot] = nbytes;
        total = (total + nbytes + 15) / 16 * 16;
    }
};

// Host -> pinned buffer -> device arena in one copy; dev[i] = where array i landed (nullptr if absent).
// The pinned buffer is written only after the copy that last read it has been made.
int pack_to_device(pearl_prb* h, const Packing& pk, const void* const* src, int count, unsigned char* arena, void** dev)
{
    if (cudaEventSynchronize(h->pin_read) != cudaSuccess) return PEARL_ERR_CUDA;
    for (int i = 0; i < count; ++i) {
        dev[i] = nullptr;
        if (!src[i] || pk.bytes[i] == 0) continue;
        memcpy(h->pin + pk.off[i], src[i], pk.bytes[i]);
        dev[i] = arena + pk.off[i];
    }
    if (cudaMemcpyAsync(arena, h->pin, pk.total, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaEventRecord(h->pin_read, h->stream) != cudaSuccess)
        return PEARL_ERR_CUDA;
    return PEARL_OK;
}

}  // namespace

int pearl_prb_insert_host(pearl_prb_t* h, uint32_t n, const void* h_obs, const void* h_act, const float* h_rew,
                          const void* h_next_obs, const uint8_t* h_done, const float* h_prio)
{
    if (!h) return PEARL_ERR_NULL;
    if (n == 0 || n > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (n > h->view.capacity) return PEARL_ERR_TOO_MANY;
    if (h->view.stack && (h_next_obs || !h_done)) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    const void* src[PRB_NUM_FIELDS + 1] = { h_obs, h_next_obs, h_act, h_rew, h_done, h_prio };
    void* dev[PRB_NUM_FIELDS + 1];
    Packing pk;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) pk.add(f, src[f] ? (uint64_t)n * h->view.field_bytes[f] : 0);
    pk.add(PRB_NUM_FIELDS, h_prio ? (uint64_t)n * 4 : 0);
    if (h->pin && pk.total <= kPackBytes) {
        // small batch: one copy; the caller's arrays are free on return, the work is left on the stream
        int rc = pack_to_device(h, pk, src, PRB_NUM_FIELDS + 1, at(h, h->lay.off_stage_in[0]), dev);
        if (rc != PEARL_OK) return rc;
        return pearl_prb_insert(h, n, dev[F_OBS], dev[F_ACT], (const float*)dev[F_REW], dev[F_NEXT_OBS],
                                (const uint8_t*)dev[F_DONE], (const float*)dev[PRB_NUM_FIELDS]);
    }
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        dev[f] = nullptr;
        const uint64_t bytes = (uint64_t)n * h->view.field_bytes[f];
        if (!src[f] || bytes == 0) continue;
        dev[f] = at(h, h->lay.off_stage_in[f]);
        if (cudaMemcpyAsync(dev[f], src[f], bytes, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    }
    float* d_prio = h_prio ? (float*)at(h, h->lay.off_stage_prio) : nullptr;
    if (h_prio && cudaMemcpyAsync(d_prio, h_prio, (uint64_t)n * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess)
        return PEARL_ERR_CUDA;
    int rc = pearl_prb_insert(h, n, dev[F_OBS], dev[F_ACT], (const float*)dev[F_REW], dev[F_NEXT_OBS],
                              (const uint8_t*)dev[F_DONE], d_prio);
    if (rc != PEARL_OK) return rc;
    // (copies from pinned memory are asynchronous: the caller's arrays are free once the stream has drained)
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int pearl_prb_sample_host(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, int32_t* h_idx, float* h_w, void* h_obs,
                          void* h_act, float* h_rew, void* h_next_obs, uint8_t* h_done)
{
    if (!h || !h_idx) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    void* dst[PRB_NUM_FIELDS + 2] = { h_obs, h_next_obs, h_act, h_rew, h_done, h_idx, h_w };
    void* dev[PRB_NUM_FIELDS + 2];
    Packing pk;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) pk.add(f, dst[f] ? (uint64_t)B * h->lay.out_bytes[f] : 0);
    pk.add(PRB_NUM_FIELDS, (uint64_t)B * 4);
    pk.add(PRB_NUM_FIELDS + 1, h_w ? (uint64_t)B * 4 : 0);
    if (h->pin && pk.total <= kPackBytes) {
        // small batch: the kernel writes its outputs packed, one copy brings them to the pinned buffer
        unsigned char* arena = at(h, h->lay.off_stage_out[0]);
        unsigned char* pin_out = h->pin + kPackBytes;
        for (int i = 0; i < PRB_NUM_FIELDS + 2; ++i) dev[i] = (dst[i] && pk.bytes[i]) ? arena + pk.off[i] : nullptr;
        int rc = pearl_prb_sample(h, B, beta, seed, (int32_t*)dev[PRB_NUM_FIELDS], (float*)dev[PRB_NUM_FIELDS + 1], dev[F_OBS],
                                  dev[F_ACT], (float*)dev[F_REW], dev[F_NEXT_OBS], (uint8_t*)dev[F_DONE]);
        if (rc != PEARL_OK) return rc;
        if (cudaMemcpyAsync(pin_out, arena, pk.total, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
            cudaStreamSynchronize(h->stream) != cudaSuccess)
            return PEARL_ERR_CUDA;
        for (int i = 0; i < PRB_NUM_FIELDS + 2; ++i)
            if (dev[i]) memcpy(dst[i], pin_out + pk.off[i], pk.bytes[i]);
        return PEARL_OK;
    }
    for (int f = 0; f < PRB_NUM_FIELDS; ++f)
        dev[f] = (dst[f] && h->lay.out_bytes[f]) ? at(h, h->lay.off_stage_out[f]) : nullptr;
    int32_t* d_idx = (int32_t*)at(h, h->lay.off_stage_out_idx);
    float* d_w = h_w ? (float*)at(h, h->lay.off_stage_out_w) : nullptr;
    int rc = pearl_prb_sample(h, B, beta, seed, d_idx, d_w, dev[F_OBS], dev[F_ACT], (float*)dev[F_REW],
                              dev[F_NEXT_OBS], (uint8_t*)dev[F_DONE]);
    if (rc != PEARL_OK) return rc;
    if (cudaMemcpyAsync(h_idx, d_idx, (uint64_t)B * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (h_w && cudaMemcpyAsync(h_w, d_w, (uint64_t)B * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        if (!dev[f]) continue;
        if (cudaMemcpyAsync(dst[f], dev[f], (uint64_t)B * h->lay.out_bytes[f], cudaMemcpyDeviceToHost, h->stream) != cudaSuccess)
            return PEARL_ERR_CUDA;
    }
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int pearl_prb_update_host(pearl_prb_t* h, uint32_t B, const int32_t* h_idx, const float* h_td, float alpha, float eps)
{
    if (!h || !h_idx || !h_td) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    if (h->pin && (uint64_t)B * 8 + 16 <= kPackBytes) {
        const void* src[2] = { h_idx, h_td };
        void* dev[2];
        Packing pk;
        pk.add(0, (uint64_t)B * 4);
        pk.add(1, (uint64_t)B * 4);
        int rc = pack_to_device(h, pk, src, 2, at(h, h->lay.off_stage_in[0]), dev);
        if (rc != PEARL_OK) return rc;
        return pearl_prb_update(h, B, (const int32_t*)dev[0], (const float*)dev[1], alpha, eps);
    }
    int32_t* d_idx = (int32_t*)at(h, h->lay.off_stage_idx);
    float* d_td = (float*)at(h, h->lay.off_stage_td);
    if (cudaMemcpyAsync(d_idx, h_idx, (uint64_t)B * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (cudaMemcpyAsync(d_td, h_td, (uint64_t)B * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    int rc = pearl_prb_update(h, B, d_idx, d_td, alpha, eps);
    if (rc != PEARL_OK) return rc;
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

namespace {

inline bool long_field(const pearl_prb* h, int f)
{
    return h->view.field_vec[f] == 16 && h->view.field_bytes[f] / 16u >= 512u;
}

// A step of long rows through host buffers with the two directions of the host link busy at once.
// The new transitions' long rows travel host -> device on a second stream while the caller's stream runs the
// tree kernel (update + the insertion's tree work, which needs the new priorities only), the descents and the
// row copy of every stratum that drew none of the new slots, and sends those rows device -> host.  When the
// new rows have arrived and are in the store (the insertion's row kernel, second stream), the rest follows on
// the caller's stream: rows of strata that drew new slots, indices, weights, short fields.  The first, large
// device -> host copy carried whatever the output staging held for those few strata: their rows are copied
// again, one by one, at the end.  Results are those of the three calls.
int step_host_duplex(pearl_prb* h, uint32_t B_upd, const int32_t* h_upd_idx, const float* h_td, float alpha, float eps, uint32_t n,
                     const void* const src[PRB_NUM_FIELDS], const float* h_new_prio, uint32_t B, float beta, uint64_t seed,
                     int32_t* h_idx, float* h_w, void* const dst[PRB_NUM_FIELDS])
{
    const Layout& L = h->lay;
    cudaStream_t main = h->stream, up = h->subs.stream[1];
    PrbBatch in_b, out_b;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        in_b.ptr[f] = (src[f] && h->view.field_bytes[f]) ? at(h, L.off_stage_in[f]) : nullptr;
        out_b.ptr[f] = (dst[f] && L.out_bytes[f]) ? at(h, L.off_stage_out[f]) : nullptr;
    }
    int32_t* d_idx = (int32_t*)at(h, L.off_stage_out_idx);
    float* d_w = h_w ? (float*)at(h, L.off_stage_out_w) : nullptr;
    int32_t* d_uidx = (int32_t*)at(h, L.off_stage_idx);
    float* d_td = (float*)at(h, L.off_stage_td);
    float* d_prio = h_new_prio ? (float*)at(h, L.off_stage_prio) : nullptr;
    auto to_dev = [](void* d, const void* s, uint64_t bytes, cudaStream_t st) {
        return cudaMemcpyAsync(d, s, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    };
    auto to_host = [](void* d, const void* s, uint64_t bytes, cudaStream_t st) {
        return cudaMemcpyAsync(d, s, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };
    // the second stream starts where the caller's stream is (the staging areas may still be in use by its work)
    if (cudaEventRecord(h->subs.fork, main) != cudaSuccess || cudaStreamWaitEvent(up, h->subs.fork, 0) != cudaSuccess) return PEARL_ERR_CUDA;
    // (the tree kernel's few inputs are handed to the copy engine first: it serves copies in the order they were issued)
    if (!to_dev(d_uidx, h_upd_idx, (uint64_t)B_upd * 4, main) || !to_dev(d_td, h_td, (uint64_t)B_upd * 4, main)) return PEARL_ERR_CUDA;
    if (d_prio && !to_dev(d_prio, h_new_prio, (uint64_t)n * 4, main)) return PEARL_ERR_CUDA;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f)
        if (in_b.ptr[f] && !to_dev(in_b.ptr[f], src[f], (uint64_t)n * h->view.field_bytes[f], up)) return PEARL_ERR_CUDA;      // (read by the row kernel only)
    unsigned char* area = h->view.handoff[0];
    int k = prb_launch_update(h->view, B_upd, d_uidx, d_td, 0, alpha, eps, main, 0, n, d_prio, in_b.ptr[F_DONE]);
    if (k != 1) return PEARL_ERR_CUDA;
    if (prb_launch_descend(h->view, B, seed, area, main, 0, 0) != 1) return PEARL_ERR_CUDA;
    if (prb_launch_gather(h->view, B, beta, area, d_idx, d_w, out_b, main, false, 1, n) != 1) return PEARL_ERR_CUDA;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f)
        if (out_b.ptr[f] && long_field(h, f) && !to_host(dst[f], out_b.ptr[f], (uint64_t)B * L.out_bytes[f], main)) return PEARL_ERR_CUDA;
    if (prb_launch_insert(h->view, n, in_b, d_prio, up, 0, nullptr, nullptr, 0, 0.0f, 0.0f, nullptr, nullptr, true) != 1) return PEARL_ERR_CUDA;
    if (cudaEventRecord(h->subs.done[1], up) != cudaSuccess || cudaStreamWaitEvent(main, h->subs.done[1], 0) != cudaSuccess) return PEARL_ERR_CUDA;
    if (prb_launch_gather(h->view, B, beta, area, d_idx, d_w, out_b, main, false, 2, n) != 1) return PEARL_ERR_CUDA;
    h->launches += 5;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    // (the cursor comes back with the batch: into the handle's pinned buffer where there is one -- no call
    // leaves its second half in use -- so that the copy call itself does not wait for the stream)
    unsigned long long cursor_here = 0;
    unsigned long long* cursor_at = h->pin ? (unsigned long long*)(h->pin + 2 * kPackBytes - 16) : &cursor_here;
    if (!to_host(h_idx, d_idx, (uint64_t)B * 4, main) || (h_w && !to_host(h_w, d_w, (uint64_t)B * 4, main))) return PEARL_ERR_CUDA;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f)
        if (out_b.ptr[f] && !long_field(h, f) && !to_host(dst[f], out_b.ptr[f], (uint64_t)B * L.out_bytes[f], main)) return PEARL_ERR_CUDA;
    if (!to_host(cursor_at, &h->view.state->cursor, sizeof(unsigned long long), main)) return PEARL_ERR_CUDA;
    if (cudaStreamSynchronize(main) != cudaSuccess) return PEARL_ERR_CUDA;
    const unsigned long long cursor = *cursor_at;
    // the strata that drew one of the new slots: their long rows were written after the large copy
    const uint64_t N = h->view.capacity;
    const uint64_t lo = cursor >= n ? cursor - n : cursor + N - n;
    bool again = false;
    for (uint32_t s = 0; s < B; ++s) {
        if (h_idx[s] < 0) continue;
        const uint64_t i = (uint64_t)h_idx[s];
        if ((i >= lo ? i - lo : i + N - lo) >= n) continue;
        for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
            const uint64_t row = L.out_bytes[f];
            if (out_b.ptr[f] && long_field(h, f) && !to_host((unsigned char*)dst[f] + s * row, out_b.ptr[f] + s * row, row, main)) return PEARL_ERR_CUDA;
        }
        again = true;
    }
    if (again && cudaStreamSynchronize(main) != cudaSuccess) return PEARL_ERR_CUDA;
    return PEARL_OK;
}

}  // namespace

// One iteration through host buffers as one call.  A small step (all inputs, and all outputs, within 256 KB
// each) makes no copy call at all: the inputs are gathered in the handle's pinned buffer, which the device
// sees mapped, the kernels read them from there and write the sampled batch into its second half, and the
// one synchronisation of the step is the wait for that.  A larger step with long rows both ways (8 KB and
// more, plain layout, at most PEARL_UPDATE_SUBBATCH updates) runs with both directions of the host link busy
// at once (step_host_duplex above); any other is the three host calls.
int pearl_prb_step_host(pearl_prb_t* h, uint32_t B_upd, const int32_t* h_upd_idx, const float* h_td, float alpha, float eps,
                        uint32_t n, const void* h_new_obs, const void* h_new_act, const float* h_new_rew, const void* h_new_next_obs,
                        const uint8_t* h_new_done, const float* h_new_prio, uint32_t B, float beta, uint64_t seed, int32_t* h_idx,
                        float* h_w, void* h_obs, void* h_act, float* h_rew, void* h_next_obs, uint8_t* h_done)
{
    if (!h || !h_upd_idx || !h_td || !h_idx) return PEARL_ERR_NULL;
    if (B_upd == 0 || B_upd > h->max_batch || n > h->max_batch || B == 0 || B > h->max_batch) return PEARL_ERR_BAD_BATCH;
    if (n > h->view.capacity) return PEARL_ERR_TOO_MANY;
    if (!finite_nonneg(alpha) || !finite_nonneg(eps) || !finite_nonneg(beta)) return PEARL_ERR_BAD_ARG;
    if (n && h->view.stack && (h_new_next_obs || !h_new_done)) return PEARL_ERR_BAD_ARG;
    const void* src[PRB_NUM_FIELDS + 3] = { h_new_obs, h_new_next_obs, h_new_act, h_new_rew, h_new_done, h_new_prio, h_upd_idx, h_td };
    void* dst[PRB_NUM_FIELDS + 2] = { h_obs, h_next_obs, h_act, h_rew, h_done, h_idx, h_w };
    Packing in, out;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) in.add(f, src[f] ? (uint64_t)n * h->view.field_bytes[f] : 0);
    in.add(PRB_NUM_FIELDS, h_new_prio ? (uint64_t)n * 4 : 0);
    in.add(PRB_NUM_FIELDS + 1, (uint64_t)B_upd * 4);
    in.add(PRB_NUM_FIELDS + 2, (uint64_t)B_upd * 4);
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) out.add(f, dst[f] ? (uint64_t)B * h->lay.out_bytes[f] : 0);
    out.add(PRB_NUM_FIELDS, (uint64_t)B * 4);
    out.add(PRB_NUM_FIELDS + 1, h_w ? (uint64_t)B * 4 : 0);
    if (!(h->pin_dev && in.total <= kPackBytes && out.total <= kPackBytes)) {
        bool long_in = false, long_out = false;
        for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
            long_in = long_in || (src[f] && long_field(h, f));
            long_out = long_out || (dst[f] && long_field(h, f));
        }
        if (n && h->view.stack == 0 && B_upd <= PEARL_UPDATE_SUBBATCH && long_in && long_out) {
            const void* ins[PRB_NUM_FIELDS] = { h_new_obs, h_new_next_obs, h_new_act, h_new_rew, h_new_done };
            DeviceGuard guard(h->device);
            if (!guard.ok) return PEARL_ERR_CUDA;
            return step_host_duplex(h, B_upd, h_upd_idx, h_td, alpha, eps, n, ins, h_new_prio, B, beta, seed, h_idx, h_w, dst);
        }
        int rc = pearl_prb_update_host(h, B_upd, h_upd_idx, h_td, alpha, eps);
        if (rc != PEARL_OK) return rc;
        rc = n ? pearl_prb_insert_host(h, n, h_new_obs, h_new_act, h_new_rew, h_new_next_obs, h_new_done, h_new_prio) : PEARL_OK;
        if (rc != PEARL_OK) return rc;
        return pearl_prb_sample_host(h, B, beta, seed, h_idx, h_w, h_obs, h_act, h_rew, h_next_obs, h_done);
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    // the pinned buffer may still be the source of a copy an earlier *_host call left on the stream
    if (cudaEventSynchronize(h->pin_read) != cudaSuccess) return PEARL_ERR_CUDA;
    void* din[PRB_NUM_FIELDS + 3];
    void* dout[PRB_NUM_FIELDS + 2];
    for (int i = 0; i < PRB_NUM_FIELDS + 3; ++i) {
        din[i] = nullptr;
        if (!src[i] || in.bytes[i] == 0) continue;
        memcpy(h->pin + in.off[i], src[i], in.bytes[i]);
        din[i] = h->pin_dev + in.off[i];
    }
    for (int i = 0; i < PRB_NUM_FIELDS + 2; ++i) dout[i] = (dst[i] && out.bytes[i]) ? h->pin_dev + kPackBytes + out.off[i] : nullptr;
    int rc = pearl_prb_step(h, B_upd, (const int32_t*)din[PRB_NUM_FIELDS + 1], (const float*)din[PRB_NUM_FIELDS + 2], alpha, eps, n,
                            din[F_OBS], din[F_ACT], (const float*)din[F_REW], din[F_NEXT_OBS], (const uint8_t*)din[F_DONE],
                            (const float*)din[PRB_NUM_FIELDS], B, beta, seed, (int32_t*)dout[PRB_NUM_FIELDS],
                            (float*)dout[PRB_NUM_FIELDS + 1], dout[F_OBS], dout[F_ACT], (float*)dout[F_REW], dout[F_NEXT_OBS],
                            (uint8_t*)dout[F_DONE]);
    if (rc != PEARL_OK) return rc;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    for (int i = 0; i < PRB_NUM_FIELDS + 2; ++i)
        if (dout[i]) memcpy(dst[i], h->pin + kPackBytes + out.off[i], out.bytes[i]);
    return PEARL_OK;
}

// ---- sampling with static scratch --------------------------------------------------------------
// Scratch of the sample kernel (raw importance-sampling weights) for callers that cannot
// allocate: a fixed array in the library image instead of the handle's slab.  In host code the
// name below is only a stand-in for the symbol; the device address comes from
// cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) double g_static_wraw[PEARL_STATIC_SCRATCH_MAX_BATCH];

namespace {
constexpr int kMaxDevices = 64;
double* g_static_wraw_addr[kMaxDevices];   // per device ordinal; nullptr until the first call there

// Device address of g_static_wraw on `device` (which must be current); nullptr on failure.
double* static_wraw_on(int device)
{
    if (device < 0 || device >= kMaxDevices) return nullptr;
    if (g_static_wraw_addr[device] == nullptr) {
        double* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_static_wraw) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        g_static_wraw_addr[device] = p;
    }
    return g_static_wraw_addr[device];
}
}  // namespace

int pearl_prb_sample_static_scratch(pearl_prb_t* h, uint32_t B, float beta, uint64_t seed, int32_t* d_idx, float* d_w,
                                    void* d_obs, void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done)
{
    if (!h || !d_idx) return PEARL_ERR_NULL;
    if (B == 0 || B > h->max_batch || B > PEARL_STATIC_SCRATCH_MAX_BATCH) return PEARL_ERR_BAD_BATCH;
    if (!finite_nonneg(beta)) return PEARL_ERR_BAD_ARG;
    const void* ptrs[PRB_NUM_FIELDS] = { d_obs, d_next_obs, d_act, d_rew, d_done };
    int rc = check_batch_ptrs(h, ptrs);
    if (rc != PEARL_OK) return rc;
    if (misaligned(d_idx, 4) || (d_w && misaligned(d_w, 4))) return PEARL_ERR_ALIGN;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    double* scratch = static_wraw_on(h->device);
    if (!scratch) return PEARL_ERR_CUDA;
    PrbView v = h->view;          // same tree, store and state; only the scratch pointer differs
    v.wraw = scratch;
    PrbBatch b;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) b.ptr[f] = (unsigned char*)ptrs[f];
    const int k = prb_launch_sample(v, B, beta, seed, d_idx, d_w, b, h->stream);
    if (k < 0) return PEARL_ERR_CUDA;
    h->launches += (uint64_t)k;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    return PEARL_OK;
}

// ---- synchronisation and read-back ---------------------------------------------------------

int pearl_prb_sync(pearl_prb_t* h, uint32_t* status_bits)
{
    if (!h) return PEARL_ERR_NULL;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    uint32_t st = 0;
    if (cudaMemcpyAsync(&st, &h->view.state->status, 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (cudaMemsetAsync(&h->view.state->status, 0, 4, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (status_bits) *status_bits = st;
    return PEARL_OK;
}

int pearl_prb_info(pearl_prb_t* h, uint64_t* fill, uint64_t* cursor, uint64_t* sample_calls, uint32_t* depth)
{
    if (!h) return PEARL_ERR_NULL;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    PrbState st;
    if (cudaMemcpyAsync(&st, h->view.state, sizeof(st), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (fill) *fill = st.fill;
    if (cursor) *cursor = st.cursor;
    if (sample_calls) *sample_calls = st.sample_calls;
    if (depth) *depth = h->view.depth;
    return PEARL_OK;
}

int pearl_prb_max_priority(pearl_prb_t* h, float* out)
{
    if (!h || !out) return PEARL_ERR_NULL;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    unsigned int bits = 0;
    if (cudaMemcpyAsync(&bits, &h->view.state->max_prio_bits, 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    memcpy(out, &bits, 4);
    return PEARL_OK;
}

uint64_t pearl_prb_level_alloc(pearl_prb_t* h, uint32_t level)
{
    if (!h || level > h->view.depth) return 0;
    return h->lay.level_alloc[level];
}

int pearl_prb_read_level(pearl_prb_t* h, uint32_t level, float* h_dst, uint64_t count)
{
    if (!h || !h_dst) return PEARL_ERR_NULL;
    if (level > h->view.depth || count > h->lay.level_alloc[level]) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    if (cudaMemcpyAsync(h_dst, h->view.level[level], count * sizeof(float), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess)
        return PEARL_ERR_CUDA;
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int pearl_prb_read_min_level(pearl_prb_t* h, uint32_t level, float* h_dst, uint64_t count)
{
    if (!h || !h_dst) return PEARL_ERR_NULL;
    if (h->view.min_off == 0 || level >= h->view.depth || count > h->lay.level_alloc[level]) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    if (cudaMemcpyAsync(h_dst, h->view.level[level] + h->view.min_off, count * sizeof(float), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess)
        return PEARL_ERR_CUDA;
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int pearl_prb_read_rows(pearl_prb_t* h, const int32_t* h_idx, uint32_t n, void* h_obs, void* h_act, float* h_rew,
                        void* h_next_obs, uint8_t* h_done)
{
    if (!h || !h_idx) return PEARL_ERR_NULL;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    void* dst[PRB_NUM_FIELDS] = { h_obs, h_next_obs, h_act, h_rew, h_done };
    for (uint32_t k = 0; k < n; ++k)
        if (h_idx[k] < 0 || (uint64_t)h_idx[k] >= h->view.capacity) return PEARL_ERR_BAD_ARG;
    const uint32_t S = h->view.stack;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) {
        const uint64_t fb = h->view.field_bytes[f];
        if (!dst[f] || fb == 0 || (S && f == F_OBS)) continue;
        for (uint32_t k = 0; k < n; ++k) {
            if (cudaMemcpyAsync((unsigned char*)dst[f] + k * fb, h->view.store[f] + (uint64_t)h_idx[k] * h->view.field_pitch[f], fb,
                                cudaMemcpyDeviceToHost, h->stream) != cudaSuccess)
                return PEARL_ERR_CUDA;
        }
    }
    if (S && (h_obs || h_next_obs)) {
        // frames: both observations are rebuilt the way a sample rebuilds them -- frame b steps back comes
        // from slot i - min(b, c), c the distance back to the nearest episode-start marker (or to slot 0
        // while the ring has not wrapped)
        PrbState st;
        if (cudaMemcpyAsync(&st, h->view.state, sizeof(st), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
        unsigned char* marks = (unsigned char*)malloc((size_t)n * S + 1);
        if (!marks) return PEARL_ERR_OOM;
        const uint64_t N = h->view.capacity, F = h->view.field_bytes[F_OBS];
        for (uint32_t k = 0; k < n; ++k)
            for (uint32_t d = 1; d <= S; ++d) {
                const uint64_t j = ((uint64_t)h_idx[k] + N - d) % N;
                if (cudaMemcpyAsync(marks + (size_t)k * S + (d - 1), h->view.store[F_DONE] + j, 1, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) {
                    free(marks);
                    return PEARL_ERR_CUDA;
                }
            }
        if (cudaStreamSynchronize(h->stream) != cudaSuccess) { free(marks); return PEARL_ERR_CUDA; }
        for (uint32_t k = 0; k < n; ++k) {
            const uint64_t i = (uint64_t)h_idx[k];
            uint32_t c = S;
            for (uint32_t d = 1; d <= S; ++d) {
                if (st.fill < N && i < d) { c = d - 1; break; }
                if (marks[(size_t)k * S + (d - 1)] & kPrbEpisodeStart) { c = d; break; }
            }
            for (uint32_t pos = 0; pos < S; ++pos) {
                const uint32_t b_next = S - 1 - pos, b_obs = S - pos;
                const uint64_t j_next = (i + N - (b_next < c ? b_next : c)) % N, j_obs = (i + N - (b_obs < c ? b_obs : c)) % N;
                if (h_next_obs && cudaMemcpyAsync((unsigned char*)h_next_obs + ((uint64_t)k * S + pos) * F, h->view.store[F_OBS] + j_next * F, F,
                                                  cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) { free(marks); return PEARL_ERR_CUDA; }
                if (h_obs && cudaMemcpyAsync((unsigned char*)h_obs + ((uint64_t)k * S + pos) * F, h->view.store[F_OBS] + j_obs * F, F,
                                             cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) { free(marks); return PEARL_ERR_CUDA; }
            }
        }
        free(marks);
    }
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

// ---- checkpoint and resume -----------------------------------------------------------------------
namespace {

constexpr uint64_t kImageHeaderBytes = 256;
struct ImageHeader {
    char magic[8];                    // "PEARLPRB"
    uint32_t version;
    uint32_t fanout;
    uint64_t capacity;
    uint32_t field_bytes[PRB_NUM_FIELDS];
    uint32_t field_pitch[PRB_NUM_FIELDS];
    uint32_t stack;
    uint32_t min_tree;
    uint64_t tree_bytes;              // state, sum tree, min-tree: slab bytes [off_state, off_wraw)
    uint64_t store_bytes;             // Data Storage: slab bytes [off_zero_end, off_stage_in[0])
};
static_assert(sizeof(ImageHeader) <= kImageHeaderBytes, "the image header has 256 bytes");

void fill_image_header(const pearl_prb* h, unsigned char out[kImageHeaderBytes])
{
    memset(out, 0, kImageHeaderBytes);
    ImageHeader hd;
    memset(&hd, 0, sizeof(hd));
    memcpy(hd.magic, "PEARLPRB", 8);
    hd.version = 1;
    hd.fanout = h->view.fanout;
    hd.capacity = h->view.capacity;
    for (int f = 0; f < PRB_NUM_FIELDS; ++f) { hd.field_bytes[f] = h->lay.field_bytes[f]; hd.field_pitch[f] = h->lay.field_pitch[f]; }
    hd.stack = h->lay.stack;
    hd.min_tree = h->lay.off_min ? 1u : 0u;
    hd.tree_bytes = h->lay.off_wraw - h->lay.off_state;
    hd.store_bytes = h->lay.off_stage_in[0] - h->lay.off_zero_end;
    memcpy(out, &hd, sizeof(hd));
}

// Copies the part of image range [offset, offset + bytes) that lies in the image's part [part_at, part_at + part_bytes),
// which is slab range [slab_at, ...), in the direction given.
int copy_image_part(pearl_prb* h, uint64_t offset, unsigned char* host, uint64_t bytes, uint64_t part_at, uint64_t part_bytes,
                    uint64_t slab_at, bool to_host)
{
    const uint64_t lo = offset > part_at ? offset : part_at;
    const uint64_t hi = (offset + bytes) < (part_at + part_bytes) ? (offset + bytes) : (part_at + part_bytes);
    if (lo >= hi) return PEARL_OK;
    unsigned char* dev = at(h, slab_at + (lo - part_at));
    unsigned char* hp = host + (lo - offset);
    const cudaError_t e = to_host ? cudaMemcpyAsync(hp, dev, hi - lo, cudaMemcpyDeviceToHost, h->stream)
                                  : cudaMemcpyAsync(dev, hp, hi - lo, cudaMemcpyHostToDevice, h->stream);
    return e == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

int image_transfer(pearl_prb* h, uint64_t offset, unsigned char* host, uint64_t bytes, bool to_host)
{
    unsigned char mine[kImageHeaderBytes];
    fill_image_header(h, mine);
    const uint64_t tree_bytes = h->lay.off_wraw - h->lay.off_state, store_bytes = h->lay.off_stage_in[0] - h->lay.off_zero_end;
    const uint64_t total = kImageHeaderBytes + tree_bytes + store_bytes;
    if (offset > total || bytes > total - offset) return PEARL_ERR_BAD_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return PEARL_ERR_CUDA;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PEARL_ERR_CUDA;
    if (offset < kImageHeaderBytes && bytes > 0) {
        const uint64_t n = (offset + bytes < kImageHeaderBytes ? offset + bytes : kImageHeaderBytes) - offset;
        if (to_host) memcpy(host, mine + offset, n);
        else if (offset != 0 || n != kImageHeaderBytes || memcmp(host, mine, kImageHeaderBytes) != 0) return PEARL_ERR_BAD_ARG;
    }
    int rc = copy_image_part(h, offset, host, bytes, kImageHeaderBytes, tree_bytes, h->lay.off_state, to_host);
    if (rc == PEARL_OK)
        rc = copy_image_part(h, offset, host, bytes, kImageHeaderBytes + tree_bytes, store_bytes, h->lay.off_zero_end, to_host);
    if (rc != PEARL_OK) return rc;
    if (!to_host) { h->main_touched = true; h->main_last_gather = 0; h->after_forked_tree = 0; }
    return cudaStreamSynchronize(h->stream) == cudaSuccess ? PEARL_OK : PEARL_ERR_CUDA;
}

}  // namespace

uint64_t pearl_prb_image_bytes(pearl_prb_t* h)
{
    if (!h) return 0;
    return kImageHeaderBytes + (h->lay.off_wraw - h->lay.off_state) + (h->lay.off_stage_in[0] - h->lay.off_zero_end);
}

int pearl_prb_export(pearl_prb_t* h, uint64_t offset, void* h_dst, uint64_t bytes)
{
    if (!h || !h_dst) return PEARL_ERR_NULL;
    return image_transfer(h, offset, (unsigned char*)h_dst, bytes, true);
}

int pearl_prb_import(pearl_prb_t* h, uint64_t offset, const void* h_src, uint64_t bytes)
{
    if (!h || !h_src) return PEARL_ERR_NULL;
    return image_transfer(h, offset, (unsigned char*)h_src, bytes, false);
}

uint64_t pearl_prb_kernel_launches(pearl_prb_t* h) { return h ? h->launches : 0; }

const char* pearl_prb_error_string(int code)
{
    switch (code) {
    case PEARL_OK: return "ok";
    case PEARL_ERR_NULL: return "a required pointer is NULL";
    case PEARL_ERR_BAD_FANOUT: return "fanout must be 2, 4, 8, 16 or 32";
    case PEARL_ERR_BAD_BATCH: return "batch is 0 or exceeds the maximum";
    case PEARL_ERR_TOO_MANY: return "more rows than the capacity";
    case PEARL_ERR_ALIGN: return "a pointer is misaligned for its row size";
    case PEARL_ERR_OOM: return "out of device memory or slab too small";
    case PEARL_ERR_BAD_ARG: return "a scalar argument is out of range or not finite";
    case PEARL_ERR_CUDA: return "a CUDA runtime call failed";
    default: return "unknown error";
    }
}

}  // extern "C"
