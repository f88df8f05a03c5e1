/*
 * pearl_prb.h -- C ABI of the B200-native Prioritized Replay Buffer.
 *
 * The buffer is the Replay Manager + Data Storage pair of PEARL (arXiv 2311.09445):
 * a K-ary sum tree over transition priorities (Section V-A) next to a struct-of-arrays
 * store of the transitions {state, action, reward, next state, done} (Section II-A).
 * The four operations are the requests the host runtime sends to the Replay Manager in
 * the paper's training protocol (Section IV, Listing 2): insertion, priority sampling
 * (Eq. 1) followed by the read of the sampled rows, and priority update.
 *
 * Conventions
 *   - Every `d_*` argument is a DEVICE pointer owned by the caller, every `h_*` argument a
 *     HOST pointer owned by the caller.  The library never frees or keeps them.
 *   - Batches are dense and row-major: row k of a field with `fb` bytes per row starts at
 *     byte k*fb.  A field pointer must be aligned to the largest power of two (<= 16) that
 *     divides fb, otherwise PEARL_ERR_ALIGN.
 *   - Calls validate their host-visible arguments, enqueue kernels on the handle's stream
 *     and return; they are ordered by that stream.  The ring cursor, the fill count, the
 *     sample-call counter and the status word live in device memory.
 *   - Return value: PEARL_OK or a negative PEARL_ERR_* (nothing was enqueued).  Conditions
 *     found on the device never trap; they set PEARL_ST_* bits in a device status word that
 *     pearl_prb_sync() returns and clears.
 *   - One handle is used from one host thread at a time.
 */
#ifndef PEARL_PRB_H_
#define PEARL_PRB_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pearl_prb pearl_prb_t;

/* Row sizes of the two caller-defined fields; reward is one binary32 and done one byte. */
typedef struct pearl_layout {
    uint32_t obs_bytes;   /* bytes of one observation (state and next state alike), may be 0 */
    uint32_t act_bytes;   /* bytes of one action, may be 0 */
} pearl_layout_t;

#define PEARL_OK 0
#define PEARL_ERR_NULL (-1)        /* a required pointer is NULL */
#define PEARL_ERR_BAD_FANOUT (-2)  /* fanout not in {2, 4, 8, 16, 32} */
#define PEARL_ERR_BAD_BATCH (-3)   /* batch is 0 or larger than max_batch */
#define PEARL_ERR_TOO_MANY (-4)    /* insert of more rows than the capacity */
#define PEARL_ERR_ALIGN (-5)       /* a field pointer is misaligned for its row size */
#define PEARL_ERR_OOM (-6)         /* allocation failed or the slab is too small */
#define PEARL_ERR_BAD_ARG (-7)     /* a scalar argument is out of range or not finite */
#define PEARL_ERR_CUDA (-8)        /* a CUDA runtime call failed */

#define PEARL_ST_BAD_INDEX 1u      /* update: index < 0 or >= fill count; entry skipped */
#define PEARL_ST_BAD_PRIORITY 2u   /* NaN/Inf/negative priority or non-finite TD error; update skips
                                      the entry, insert stores the row with priority 0 */
#define PEARL_ST_EMPTY 4u          /* sample on an empty buffer or a non-positive total; outputs untouched */
#define PEARL_ST_CLAMPED 8u        /* a descent met residual >= last prefix sum and took the last positive child */
#define PEARL_ST_INTERNAL 16u      /* inconsistent tree met during a descent, or a bounded wait ran out.
                                      Every wait on the device (a bulk copy's completion, the grid barrier of
                                      a large update) gives up after a fixed number of polls instead of
                                      hanging.  After a copy that gave up, rows of that call are missing or
                                      partial.  After an update of more than 1024 entries that gave up, the
                                      tree is not consistent: leaves named by the batch may hold the marker
                                      bit pattern 0x80000000|entry instead of a priority, and parents may not
                                      equal the sum of their children; every later update of more than 1024
                                      entries on that buffer raises the bit again and does nothing.  Treat the
                                      buffer as lost: destroy it and build a new one.  No correct run raises
                                      this bit. */
#define PEARL_ST_STALE 32u         /* update_after_insert: the index was overwritten since it was sampled; entry skipped */

/* The largest update batch one thread block handles.  A batch of more than 1024 priorities or TD
 * errors is applied by one launch of many co-resident thread blocks (a cooperative launch; the last
 * valid entry of a repeated index still wins); a batch of changes (pearl_prb_update_delta) of any
 * size, or any batch on a device without cooperative launches, by one thread block per sub-batch of
 * at most this many entries, sub-batches in batch order, one launch each.  The result is that of
 * the whole batch either way. */
#define PEARL_UPDATE_SUBBATCH 4096u

/* Bytes of device memory a buffer of this geometry needs (tree, storage, scratch and the
 * staging areas of the *_host calls).  0 if the arguments are invalid. */
uint64_t pearl_prb_slab_bytes(uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout,
                              uint32_t max_batch);

/* Creates a buffer of `capacity` slots (1 .. 2^30) with a sum tree of the given fanout
 * (Section V-A: the tree is parameterised by depth and fanout).  Depth D is the smallest
 * D >= 1 with fanout^D >= capacity; level 0 is the root, level D the leaves; each level is a
 * binary32 array zero-padded to a multiple of the fanout.
 *   device       CUDA device ordinal that owns the memory.
 *   cuda_stream  a cudaStream_t (NULL = the legacy default stream) on which every call enqueues.
 *   slab         optional caller-owned device memory of at least pearl_prb_slab_bytes() bytes,
 *                256-byte aligned; NULL lets the library allocate (and free in destroy).
 * The tree, the state and the scratch area are zeroed on the stream.  Besides the slab a handle
 * owns five more streams with their events (the tree kernel of a long-row update_insert, the
 * sub-batches of pearl_prb_sample_streamed; all joined back into cuda_stream before a call's work
 * is over) and 512 KB of pinned host memory for the *_host calls (without it they copy array by
 * array).  Returns PEARL_ERR_OOM if the slab is too small, and PEARL_ERR_BAD_ARG for a geometry out
 * of range -- which includes a row whose size is not a multiple of 16 bytes (or is below 8 KB) when
 * max_batch such rows hold 2^32 or more copy granules (the largest power of two, at most 16, that
 * divides the row size): pad such rows to a multiple of 16 bytes or lower max_batch. */
int pearl_prb_create(pearl_prb_t** out, uint64_t capacity, uint32_t fanout,
                     const pearl_layout_t* layout, uint32_t max_batch, int device,
                     void* cuda_stream, void* slab, uint64_t slab_bytes);

/* A buffer whose Data Storage keeps ONE frame per transition instead of two stacked observations (the
 * paper's Pong workload, Table III, has 84 x 84 observations and a DQN state stacks the last few; Section
 * VI-C: Data Storage traffic is what dominates).  The paper describes no such layout; the one used here:
 *   - an observation is `stack` frames (1..16) of frame_bytes each, oldest first; a sample hands out obs and
 *     next_obs rows of stack * frame_bytes bytes, as a buffer created with pearl_prb_create would;
 *   - consecutive ring slots hold consecutive steps of ONE trajectory.  Each slot stores the newest frame
 *     of its transition's next observation: the insertion calls take that frame per transition in
 *     d_obs (rows of frame_bytes), d_next_obs must be NULL and d_done must be given;
 *   - an episode begins with a marker slot: bit 1 (value 2) of its done byte is set, its frame is the
 *     episode's first frame, its other fields are not used, and its leaf is 0 whatever priority is given,
 *     so it is never sampled.  Bit 0 of done keeps its meaning;
 *   - for a sampled slot i the frame b steps back is that of slot i - min(b, c), c being the distance back
 *     to the nearest marker (or to slot 0 while the ring has not wrapped): what lies before the episode
 *     repeats its first frame.  next_obs = frames stack-1 .. 0 steps back, obs = frames stack .. 1 steps back;
 *   - an insertion also clears the leaves of the `stack` slots that follow the new cursor -- once the ring
 *     has wrapped they are the oldest transitions, whose history the insertion overwrites -- and an update
 *     that names one of them is skipped and raises PEARL_ST_STALE;
 *   - pearl_prb_sample_uniform is refused (PEARL_ERR_BAD_ARG): a uniform draw could name a marker.
 * Everything else -- tree, sampling, weights, updates, status bits -- is as for pearl_prb_create.  For
 * stack = 4 the store is an eighth of the plain layout's and an insertion writes an eighth of the bytes.
 * capacity must exceed stack. */
uint64_t pearl_prb_slab_bytes_frames(uint64_t capacity, uint32_t fanout, uint32_t frame_bytes, uint32_t stack,
                                     uint32_t act_bytes, uint32_t max_batch);
int pearl_prb_create_frames(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, uint32_t frame_bytes,
                            uint32_t stack, uint32_t act_bytes, uint32_t max_batch, int device, void* cuda_stream,
                            void* slab, uint64_t slab_bytes);

/* Creation with options.  frame_stack = 0 gives pearl_prb_create's layout; frame_stack >= 1 that of
 * pearl_prb_create_frames (layout->obs_bytes is then the size of one frame).  `options` is a sum of PEARL_OPT_*
 * bits (unknown bits: PEARL_ERR_BAD_ARG; pearl_prb_slab_bytes_opts returns 0).
 *   PEARL_OPT_MIN_TREE  the buffer keeps, beside the sum tree, a min-tree of the same shape (Section V-A
 *       describes the sum tree only; a min-tree is what prioritized-replay implementations use for the
 *       weight normalisation of Schaul et al., Algorithm 1): node (l, a), l < depth, holds the smallest
 *       positive leaf below it, 0 if there is none; the leaves serve both trees.  Every call that writes
 *       the sum tree re-derives the min-tree's nodes above the written leaves in the same passes (the
 *       min-tree costs one more array of the size of the inner levels, and an update or insertion about
 *       one more read per level).  pearl_prb_sample_buffer_norm then reads the minimum at the root
 *       instead of scanning the leaves; its results are the same either way (the minimum of a set does
 *       not depend on the order it is taken in). */
#define PEARL_OPT_MIN_TREE 1u
uint64_t pearl_prb_slab_bytes_opts(uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout,
                                   uint32_t frame_stack, uint32_t options, uint32_t max_batch);
int pearl_prb_create_opts(pearl_prb_t** out, uint64_t capacity, uint32_t fanout, const pearl_layout_t* layout,
                          uint32_t frame_stack, uint32_t options, uint32_t max_batch, int device,
                          void* cuda_stream, void* slab, uint64_t slab_bytes);

/* Synchronises the handle's streams, frees library-owned memory, streams, events and the handle. */
int pearl_prb_destroy(pearl_prb_t* prb);

/* Insertion (Section V-A: "priority retrievals followed by priority updates"; Listing 2: the
 * collected experiences are added to the Data Storage and insertion requests sent to the RM).
 * Writes n transitions to ring slots cursor .. cursor+n-1 (mod capacity), sets their leaves to
 * d_prio and re-sums the ancestors; then cursor += n (mod capacity), fill = min(fill+n, capacity).
 * d_prio gives each new transition's priority; with d_prio == NULL every new transition takes the
 * largest priority written so far by any call (1 if none yet), the usual default of prioritized
 * replay (Schaul et al.), so that it is replayed at least once.  d_obs/d_next_obs: n rows of obs_bytes;
 * d_act: n rows of act_bytes; d_rew: n binary32; d_done: n bytes; a NULL field pointer leaves
 * that field of the slots unwritten.  1 <= n <= min(max_batch, capacity). */
int pearl_prb_insert(pearl_prb_t* prb, uint32_t n, const void* d_obs, const void* d_act,
                     const float* d_rew, const void* d_next_obs, const uint8_t* d_done,
                     const float* d_prio);

/* Priority sampling (Eq. 1, Section V-A) + the Data Storage read of the sampled rows
 * (Listing 2: sampled_data = D_storage[sampled_indices]).
 * The range [0, total) is cut into B equal strata; stratum k draws
 *   x_k = (k + u_k) * total / B,  u_k = word 0 of Philox4x32-10(counter = (k, 0, call_lo, call_hi),
 *   key = (seed_lo, seed_hi)) * 2^-32,
 * where `call` counts this handle's earlier successful sample calls.  A root-to-leaf traversal
 * finds the leaf i_k whose prefix interval holds x_k (binary32 left-to-right child prefix sums,
 * binary64 target).  Outputs, each of B entries:
 *   d_idx   leaf indices (int32);
 *   d_w     importance-sampling weights (fill * p_i / total)^(-beta), divided by their maximum
 *           over the batch (may be NULL);
 *   d_obs, d_act, d_rew, d_next_obs, d_done   the gathered rows (each may be NULL to skip it).
 * 1 <= B <= max_batch; beta finite and >= 0. */
int pearl_prb_sample(pearl_prb_t* prb, uint32_t B, float beta, uint64_t seed, int32_t* d_idx,
                     float* d_w, void* d_obs, void* d_act, float* d_rew, void* d_next_obs,
                     uint8_t* d_done);

/* Uniform replay (the toolkit's other replay mode, Section III-B: set_replay(size, mode, fanout)):
 * B independent draws i_k = floor(u_k * fill) from the transitions stored, u_k from the same Philox
 * stream and call counter as pearl_prb_sample; the tree is not read.  d_w (may be NULL) is filled
 * with 1; the gathered rows as in pearl_prb_sample.  An empty buffer raises PEARL_ST_EMPTY. */
int pearl_prb_sample_uniform(pearl_prb_t* prb, uint32_t B, uint64_t seed, int32_t* d_idx, float* d_w,
                             void* d_obs, void* d_act, float* d_rew, void* d_next_obs, uint8_t* d_done);

/* Priority update (Section V-A).  For b = 0 .. B-1 in batch order: p_b = (|d_td[b]| + eps)^alpha
 * and leaf[d_idx[b]] <- p_b, so the last valid entry of a repeated index wins; then every
 * ancestor of a written leaf is recomputed as the left-to-right binary32 sum of its children,
 * deepest level first.  The power is evaluated in binary64 from IEEE basic operations only, so
 * it is reproducible bit for bit.  1 <= B <= max_batch;
 * alpha, eps finite and >= 0. */
int pearl_prb_update(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx, const float* d_td,
                     float alpha, float eps);

/* As pearl_prb_update, with the priorities given directly (no power). */
int pearl_prb_update_priorities(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx,
                                const float* d_prio);

/* The paper's own form of the priority update (Section V-A, "priority update": the inputs are the
 * indices and the change Delta of each priority).  Entry by entry in batch order the leaf becomes
 * leaf + Delta, one binary32 addition, so that repeated indices accumulate in batch order; an
 * entry whose Delta is not finite, or whose sum is negative or not finite, is skipped with
 * BAD_PRIORITY and leaves the leaf as it was.  Where the paper adds Delta to every node of the
 * root-leaf path under a mutex, the ancestors here are re-summed from their children as after any
 * other write: the same tree up to rounding, every parent still the sum of its children, and no
 * lock.  Arguments and errors as for pearl_prb_update_priorities. */
int pearl_prb_update_delta(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx, const float* d_delta);

/* Priority update that arrives after an insertion (Section IV-C, "Replay-Collision-Free
 * Scheduling": the insertion index is compared against the sampled indices, so that the Learner's
 * update does not contaminate a transition the Actors wrote in the meantime).  `inserted`
 * transitions have been inserted since d_idx was sampled; they occupy the ring slots
 * cursor-inserted .. cursor-1 (mod capacity).  An entry naming one of them is skipped and raises
 * PEARL_ST_STALE; everything else is pearl_prb_update.  The sequence sample, insert,
 * update_after_insert leaves the same tree as sample, update, insert.  inserted <= capacity. */
int pearl_prb_update_after_insert(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx, const float* d_td,
                                  float alpha, float eps, uint32_t inserted);

/* Priority retrieval (Section V-A): d_out[b] = the priority stored at d_idx[b], for b < B.  An
 * index outside [0, fill) yields 0 and raises PEARL_ST_BAD_INDEX.  1 <= B <= max_batch. */
int pearl_prb_get_priorities(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx, float* d_out);

/* Priority update followed by insertion, in one call.  The result is exactly that of
 * pearl_prb_update(prb, B, d_idx, d_td, alpha, eps) followed by pearl_prb_insert(prb, n, ...): the
 * update's tree work is done first, the insertion's tree work after it, by the same thread blocks,
 * while other thread blocks already copy the new rows into the Data Storage (an update touches
 * the tree only, so the two do not conflict).  Short rows: one launch (update batches of 1024 entries
 * and more: the update's launch, then the insertion's).  Rows of 8 KB and more: the
 * tree work is a kernel of its own on a second stream of the handle, beside the kernel that copies
 * the rows; the handle's stream continues when both are done (capturable in a CUDA graph).  This
 * is the overlap of the paper's training
 * protocol, where insertion runs beside the priority update (Section IV-C; Eq. 7:
 * T_itr = T_samp + max(T_ins, T_upd + T_learner)).  Arguments and errors as for the two calls. */
int pearl_prb_update_insert(pearl_prb_t* prb, uint32_t B, const int32_t* d_idx, const float* d_td,
                            float alpha, float eps, uint32_t n, const void* d_obs, const void* d_act,
                            const float* d_rew, const void* d_next_obs, const uint8_t* d_done,
                            const float* d_prio);

/* One iteration of the training protocol as one call (Listing 2; Section IV-C, Eq. 7): the priority
 * update for the batch the Learner has just finished with and the insertion of the transitions the
 * Actors have collected meanwhile -- exactly pearl_prb_update_insert(prb, B_upd, d_upd_idx, d_td, alpha,
 * eps, n, d_new_*...) -- followed by the sample of the next batch -- exactly pearl_prb_sample(prb, B,
 * beta, seed, d_idx, d_w, d_obs ...): same results, same state, same status bits as the two calls.
 * What the one call buys is one host call per iteration with all arguments checked before anything is
 * enqueued; the kernels are those of the two calls (for rows of 8 KB and more: the tree kernel beside the
 * copy of the new rows, then the sample).  d_upd_idx may be the d_idx of the previous step: it is read
 * before d_idx is written.
 * n == 0 stands for an iteration without new transitions (update, then sample; the d_new_* are not read).
 * Arguments and errors as for the two calls; nothing is enqueued if any argument is refused. */
int pearl_prb_step(pearl_prb_t* prb, uint32_t B_upd, const int32_t* d_upd_idx, const float* d_td, float alpha,
                   float eps, uint32_t n, const void* d_new_obs, const void* d_new_act, const float* d_new_rew,
                   const void* d_new_next_obs, const uint8_t* d_new_done, const float* d_new_prio, uint32_t B,
                   float beta, uint64_t seed, int32_t* d_idx, float* d_w, void* d_obs, void* d_act, float* d_rew,
                   void* d_next_obs, uint8_t* d_done);

/* pearl_prb_sample with the weights normalised as in the prioritized-replay paper the toolkit
 * follows (Schaul et al., Algorithm 1: w_j = (N P(j))^-beta / max_i w_i, the maximum over the whole
 * memory): the divisor is the weight of the smallest positive priority stored,
 * (N p_min / total)^-beta, found by a scan of the leaves in a launch of its own before the sample
 * -- or, in a buffer created with PEARL_OPT_MIN_TREE, read from the root of its min-tree.
 * Weights are then at most 1 and do not depend on which other transitions the batch holds.  PEARL
 * itself does not say how the weights are normalised.  Everything else as pearl_prb_sample. */
int pearl_prb_sample_buffer_norm(pearl_prb_t* prb, uint32_t B, float beta, uint64_t seed, int32_t* d_idx,
                                 float* d_w, void* d_obs, void* d_act, float* d_rew, void* d_next_obs,
                                 uint8_t* d_done);

/* pearl_prb_sample issued as n_sub (1..4, <= B) sub-batches of consecutive strata -- sub-batch i is
 * strata [i*B/n_sub, (i+1)*B/n_sub) -- each a launch of its own on a stream of the handle, so that
 * the Learner can start on the first sub-batch while the others are still being gathered (the
 * paper's overlap of computation and communication by sub-batches on several streams, Section IV-C).
 * Outputs, and the state left behind, are those of pearl_prb_sample.  The handle's stream continues
 * when all sub-batches are done; the weights are normalised by the maximum of the whole batch and
 * final only then.  pearl_prb_wait_sub_batch makes `cuda_stream` (a cudaStream_t) wait until the
 * indices and gathered rows of sub-batch `sub_batch` of the most recent streamed call are in place
 * (PEARL_ERR_BAD_ARG if there is no such sub-batch).  n_sub == 1 is pearl_prb_sample. */
int pearl_prb_sample_streamed(pearl_prb_t* prb, uint32_t B, float beta, uint64_t seed, uint32_t n_sub,
                              int32_t* d_idx, float* d_w, void* d_obs, void* d_act, float* d_rew,
                              void* d_next_obs, uint8_t* d_done);
int pearl_prb_wait_sub_batch(pearl_prb_t* prb, uint32_t sub_batch, void* cuda_stream);

/* Host-buffer forms of the three calls (the paper's host runtime exchanges requests and data
 * with the Replay Manager over PCIe, Section IV-A).  They copy their inputs to the device and
 * their outputs back on the handle's stream; sample_host returns after the stream has drained,
 * insert_host and update_host once their host buffers may be reused.  A call whose arrays come to
 * at most 256 KB travels packed -- the arrays are gathered in a pinned buffer of the handle and cross
 * PCIe in one copy (insert_host and update_host then leave their work on the stream and return at
 * once); a larger call copies array by array, asynchronously if the caller's memory is pinned, and
 * returns when the stream has drained.  Output pointers of sample_host other than h_idx may be NULL. */
int pearl_prb_insert_host(pearl_prb_t* prb, uint32_t n, const void* h_obs, const void* h_act,
                          const float* h_rew, const void* h_next_obs, const uint8_t* h_done,
                          const float* h_prio);
int pearl_prb_sample_host(pearl_prb_t* prb, uint32_t B, float beta, uint64_t seed, int32_t* h_idx,
                          float* h_w, void* h_obs, void* h_act, float* h_rew, void* h_next_obs,
                          uint8_t* h_done);
int pearl_prb_update_host(pearl_prb_t* prb, uint32_t B, const int32_t* h_idx, const float* h_td,
                          float alpha, float eps);

/* pearl_prb_step through host buffers: the update for the previous batch, the insertion of the new
 * transitions and the sample of the next batch, with every array in host memory (Section IV-A: the host
 * runtime exchanges requests and data with the Replay Manager over PCIe).  Returns when the sampled batch is
 * in the caller's arrays.  A step whose inputs and whose outputs come to at most 256 KB each makes no copy
 * call: the inputs are gathered in a pinned buffer of the handle that the device reads in place, the kernels
 * write the batch into that buffer, and the step's one synchronisation is the wait for them.  A larger step
 * that inserts and samples rows of 8 KB and more (plain layout, n >= 1, B_upd <= PEARL_UPDATE_SUBBATCH) keeps
 * both directions of the host link busy at once: the new rows travel to the device on a stream of the handle
 * while the caller's stream updates the tree (the new priorities included), draws the batch, and sends back
 * the rows of every stratum that drew none of the new slots; the rest -- rows of strata that did, indices,
 * weights, short fields -- follows when the new rows are stored.  The copies overlap only if the caller's
 * arrays are pinned (page-locked) memory; with pageable memory the step is correct and serial.  Any other
 * large step is pearl_prb_update_host, pearl_prb_insert_host and pearl_prb_sample_host one after the other.
 * Results are those of the three calls whichever way the step travels.
 * Arguments and errors as for pearl_prb_step, with host pointers. */
int pearl_prb_step_host(pearl_prb_t* prb, uint32_t B_upd, const int32_t* h_upd_idx, const float* h_td, float alpha,
                        float eps, uint32_t n, const void* h_new_obs, const void* h_new_act, const float* h_new_rew,
                        const void* h_new_next_obs, const uint8_t* h_new_done, const float* h_new_prio, uint32_t B,
                        float beta, uint64_t seed, int32_t* h_idx, float* h_w, void* h_obs, void* h_act, float* h_rew,
                        void* h_next_obs, uint8_t* h_done);

/* Largest batch pearl_prb_sample_static_scratch accepts. */
#define PEARL_STATIC_SCRATCH_MAX_BATCH 4096u

/* pearl_prb_sample with its per-call scratch in library-owned static device memory.
 * (The paper has no counterpart; this exists for callers that cannot allocate.)
 *
 * Who needs it: code that runs where device allocation is off the table -- a plug-in inside a
 * framework whose memory pool has already claimed the whole GPU, so that a cudaMalloc would fail
 * or fragment it; a real-time control or serving loop whose rules forbid allocator calls after
 * start-up.  Such a caller hands in the same inputs and outputs as pearl_prb_sample, and the
 * kernel's scratch (the batch's raw, un-normalised importance-sampling weights, one binary64 per
 * stratum) lives in a fixed 32 KiB array that is part of the library image: every GPU on which
 * the library runs this call holds that array until the process exits, whether or not it is used
 * again.  The call itself performs no cudaMalloc/cudaFree and calls no allocating routine.
 *
 * Arguments, outputs, ordering on the handle's stream and error codes are those of
 * pearl_prb_sample, except that B > PEARL_STATIC_SCRATCH_MAX_BATCH returns PEARL_ERR_BAD_BATCH
 * ("batch is 0 or exceeds the maximum") and nothing is enqueued.
 *
 * Set-up: the first call on each device looks up the array's device address (one runtime query,
 * made with that device current, remembered afterwards).  Make that first call outside any
 * stream capture.
 *
 * Sharing: all handles and all streams of a device use the same array, and it keeps whatever the
 * last call left in it.  Nothing in it has to start at zero -- every entry the kernel reads was
 * written earlier in the same call -- so it is not cleared.  Two of these calls that overlap on
 * one GPU (different streams, or different handles on different streams) race on the array and
 * produce wrong weights; keep them ordered on one stream or serialise them yourself. */
int pearl_prb_sample_static_scratch(pearl_prb_t* prb, uint32_t B, float beta, uint64_t seed,
                                    int32_t* d_idx, float* d_w, void* d_obs, void* d_act,
                                    float* d_rew, void* d_next_obs, uint8_t* d_done);

/* Waits for the stream; returns the accumulated PEARL_ST_* bits in *status_bits (may be NULL)
 * and clears them. */
int pearl_prb_sync(pearl_prb_t* prb, uint32_t* status_bits);

/* Read-back for tests and checkpoints; each synchronises the stream.  Any output may be NULL. */
int pearl_prb_info(pearl_prb_t* prb, uint64_t* fill, uint64_t* cursor, uint64_t* sample_calls,
                   uint32_t* depth);
/* The largest priority written so far by insert or update calls (0 if none). */
int pearl_prb_max_priority(pearl_prb_t* prb, float* h_out);
/* Copies the first `count` entries (padding included) of tree level `level` (0 = root). */
int pearl_prb_read_level(pearl_prb_t* prb, uint32_t level, float* h_dst, uint64_t count);
/* The same for level `level` < depth of the min-tree (PEARL_ERR_BAD_ARG without PEARL_OPT_MIN_TREE). */
int pearl_prb_read_min_level(pearl_prb_t* prb, uint32_t level, float* h_dst, uint64_t count);
/* Number of entries of a level including its zero padding; 0 for an invalid level. */
uint64_t pearl_prb_level_alloc(pearl_prb_t* prb, uint32_t level);
/* Copies stored rows h_idx[0..n) (slot numbers < capacity) to host arrays. */
int pearl_prb_read_rows(pearl_prb_t* prb, const int32_t* h_idx, uint32_t n, void* h_obs,
                        void* h_act, float* h_rew, void* h_next_obs, uint8_t* h_done);

/* Checkpoint and resume.  The image of a buffer is a 256-byte header (geometry: capacity, fanout, row sizes,
 * frame stack, options) followed by its persistent device memory as it lies in the slab: the state (ring
 * cursor, fill count, call counter, running maximum, pending status bits), the sum tree (and the min-tree
 * of a buffer that keeps one), and the Data Storage.  The paper keeps replay memory for the length of a
 * training run (Section IV); a run that is to survive a restart needs it back bit for bit, because the
 * sampled indices depend on every priority and on the call counter.
 *   pearl_prb_image_bytes  the size of the image.
 *   pearl_prb_export       waits for the stream, then copies bytes [offset, offset + bytes) of the image to
 *                          h_dst (so a large image can be written out piece by piece).
 *   pearl_prb_import       copies bytes [offset, offset + bytes) of an image into the buffer.  A piece that
 *                          covers any of the header must cover all of it; the header is then compared with
 *                          this buffer's geometry: PEARL_ERR_BAD_ARG if they differ (nothing is copied).
 *                          The caller imports the whole image, the header first, before the next call
 *                          that uses the buffer; after that the buffer behaves exactly as the exported one
 *                          did: same samples for the same seeds, same tree, same rows.  Waits for the stream.
 * PEARL_ERR_BAD_ARG for a range outside the image. */
uint64_t pearl_prb_image_bytes(pearl_prb_t* prb);
int pearl_prb_export(pearl_prb_t* prb, uint64_t offset, void* h_dst, uint64_t bytes);
int pearl_prb_import(pearl_prb_t* prb, uint64_t offset, const void* h_src, uint64_t bytes);

/* Number of kernels this handle has launched so far. */
uint64_t pearl_prb_kernel_launches(pearl_prb_t* prb);

/* A short English name for a PEARL_ERR_* code. */
const char* pearl_prb_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* PEARL_PRB_H_ */
