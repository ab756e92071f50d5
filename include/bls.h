/*
 * bls.h - C ABI of the B200 bounded-lag-synchronous (BLS) embedding lookup.
 *
 * One GPU emulates P logical ranks.  Every rank owns a partition of T embedding
 * tables (all resident in device memory) and a row block of b = B/P samples of
 * the batch.  One iteration of the path is
 *   (1) route   every rank sorts the row IDs it needs by owner rank: alltoallv
 *               send counts / displacements and a stably packed send buffer;
 *   (2) lookup  every owner gathers the requested rows and sum-pools them per
 *               bag with fp32 accumulation;
 *   (3) return  the pooled vectors are written straight into the requester's
 *               output layout out[src][s][t][:];
 * and iterations are kept in a ring of k_max+1 slots driven by per-rank
 * progress counters in device memory, so that ranks may be up to k iterations
 * apart.
 *
 * Conventions
 *   - All `const void*`/`int32_t*` data arguments are DEVICE pointers unless the
 *     argument is documented as "host".  The library allocates no device
 *     memory: the caller provides one workspace (bls_plan_bytes) and keeps
 *     tables, workspace and per-iteration inputs alive as documented.
 *   - All work is enqueued on the CUDA stream given to bls_plan; calls return
 *     without synchronising unless stated.
 *   - Bags are ordered (src, t, s): flat bag index g = (src*T + t)*b + s.
 *     `offsets` is int32 [P*T*b + 1], exclusive prefix of bag lengths starting
 *     at 0; `ids` is int32 [offsets[last]], row numbers into table t.
 *   - Errors are return codes.  Conditions detected on the device (bad ID,
 *     capacity exceeded, bounded wait expired) are latched in a device status
 *     word and reported by bls_status(); the device never traps.
 */
#ifndef BLS_H
#define BLS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bls_plan bls_plan_t;          /* opaque, host memory */

typedef enum {
    BLS_OK = 0,
    BLS_EINVAL = 1,     /* bad argument / malformed offsets */
    BLS_ENOSPC = 2,     /* workspace or per-rank ID capacity too small */
    BLS_ECUDA = 3,      /* a CUDA runtime call failed */
    BLS_ERANGE = 4,     /* an ID outside [0, rows) was seen (it was replaced by row 0) */
    BLS_ETIMEOUT = 5,   /* a bounded device-side wait gave up */
    BLS_ESTATE = 6      /* call order violated, k > k_max, or k changed mid-flight */
} bls_status_t;

typedef enum { BLS_F32 = 0, BLS_BF16 = 1, BLS_F16 = 2 } bls_dtype_t;

/* Table placement (Section I leaves the partitioning strategy open):
 *   TABLE_RR   owner(t, id) = t mod P, owner-local row = id
 *   ROW_BLOCK  owner(t, id) = id / ceil(rows_t / P), owner-local row = id - owner*ceil(rows_t/P) */
typedef enum { BLS_PART_TABLE_RR = 0, BLS_PART_ROW_BLOCK = 1 } bls_part_t;

/* One embedding table: row-major [rows][dim] of `dtype`, device memory, base
 * 16-byte aligned, dim*sizeof(dtype) one of 16,32,64,128,256,512 bytes.  All
 * tables of a plan share dim and dtype.  Borrowed for the plan's lifetime. */
typedef struct {
    const void *weight;
    int64_t rows;
    int32_t dim;
    int32_t dtype;               /* bls_dtype_t */
} bls_table_t;

/* Device pointers to the routing artefacts and output of one iteration's slot
 * (for parity checks and for consumers of the output).
 *   sendcounts/sdispls  [P][P] indexed [src][dst]   (alltoallv arguments of the request leg)
 *   recvcounts/rdispls  [P][P] indexed [dst][src]   (valid once the owners have answered the iteration:
 *                       bls_counters reports served > iter; with a bound >= 1 that may be one
 *                       step after the step that issued it)
 *   sendbuf             rank src's packed send buffer starts at sendbuf + src*sendbuf_stride;
 *                       owner-local rows, sorted by dst, ties in original order
 *   sub_start           rank src's array starts at sub_start + src*sub_stride and has sub_entries
 *                       entries: the start position (in src's send buffer) of every sub-bag, from
 *                       which bag boundaries are rebuilt.  Table-wise (sub_bag_major = 0): ordered
 *                       (dst, table, sample) plus one terminal entry; the length of a sub-bag is the
 *                       difference to the next entry.  Row-wise (sub_bag_major = 1): ordered
 *                       (table, sample, dst) plus P terminal entries (one per dst); the length of
 *                       sub-bag (t, s, dst) is entry[(t*b+s+1)*P + dst] - entry[(t*b+s)*P + dst]
 *   out                 fp32 [P][b][T][dim], the requester layout */
typedef struct {
    const int32_t *sendcounts, *sdispls, *recvcounts, *rdispls;
    const int32_t *sendbuf;
    int64_t sendbuf_stride;
    const int32_t *sub_start;
    int64_t sub_stride;
    int64_t subbags_per_rank;
    int64_t sub_entries;
    int32_t sub_bag_major;
    const float *out;
} bls_route_view_t;

/* ---- plan (Section III-B "Initialisation": buffers are created and registered
 * once and then reused circularly; the bound is passed at initialisation) ---- */

/* Workspace size in bytes for the given shape.  host call, no GPU work.
 * max_ids_per_rank: capacity of one rank's send buffer (IDs per rank per iteration). */
bls_status_t bls_plan_bytes(const bls_table_t *tables /*host*/, int T, int part, int P,
                            int local_batch, int k_max, int64_t max_ids_per_rank, size_t *bytes /*host*/);

/* Build a plan inside `workspace` (device, 256-byte aligned, `bytes` long, borrowed
 * until bls_destroy).  Enqueues the initialisation of counters and descriptors on
 * `cuda_stream` (a cudaStream_t; NULL = default stream).  P <= 32, k_max <= 15. */
bls_status_t bls_plan(const bls_table_t *tables /*host*/, int T, int part, int P, int local_batch,
                      int k_max, int64_t max_ids_per_rank, void *workspace, size_t bytes,
                      void *cuda_stream, bls_plan_t **plan /*host out*/);

void bls_destroy(bls_plan_t *plan);          /* frees host-side state (incl. the copy streams and timing
                                                events it created); the workspace stays the caller's;
                                                does not synchronise */

/* ---- the synchronous decomposition (bound 0 == plain alltoallv, Section III-D) ----
 * bls_route:  step (1) for every rank for iteration `iter` (must be the next
 *             unissued iteration, with nothing outstanding).  ids/offsets are
 *             borrowed until the call's work has run.
 * bls_lookup: steps (2)+(3) for that iteration; afterwards bls_view(iter).out
 *             holds the result until the next iteration is issued. */
bls_status_t bls_route(bls_plan_t *plan, int64_t iter, const int32_t *ids, const int32_t *offsets,
                       int64_t n_ids);
bls_status_t bls_lookup(bls_plan_t *plan, int64_t iter);

/* ---- the BLS loop (Section IV, Listing 2) ----
 * bls_step: issue the next iteration t with bound k (0 <= k <= k_max, the same k
 *           until everything outstanding has been drained).  Ranks that are not
 *           held back by an injected stall route, serve and complete whatever
 *           the counters allow; the call makes sure iteration t-k is complete on
 *           every rank (the oldest request is waited for once more than k are
 *           outstanding) and hands it back: *out = its fp32 [P][b][T][dim] block
 *           inside the ring, *out_iter = t-k; or *out = NULL, *out_iter = -1
 *           during the first k steps of a loop (iteration t-k does not exist, or belongs
 *           to an earlier loop that has been drained).  `*out` stays valid until the next bls_step/bls_drain
 *           call on the stream.  ids/offsets of iteration t are borrowed until
 *           k further steps (or the drain) have run.
 *           With k >= 1, table-wise placement, no injected delays and iterations of about
 *           a million lookups or more (bls_set_overlap), a step works in overlapped mode (the
 *           paper's Table I: communication of one batch beside computation of another):
 *           the requesters post iteration t while the owners answer iteration t-1, the
 *           router enqueued on a second stream beside the gather-pool kernel.  The
 *           plan's stream waits for that second stream before the call returns control of
 *           it, so the caller sees one ordered stream.  In this mode the owners are one
 *           iteration behind the requesters after a step (bls_status reports a lag of 1)
 *           and the first bls_drain call enqueues the last answer.  Results are the same
 *           bit for bit in both modes.
 *           Small table-wise iterations without injected delays (below about 256 K lookups,
 *           below a million when bags hold four IDs or fewer on average;
 *           bls_set_fused) are ONE kernel launch: every block routes a tile of one
 *           (requester, table) chunk and answers it at once, the last block publishes the
 *           iteration for all ranks.  Same routing artefacts, same sums, bit for bit.
 * bls_drain: Listing 2's final loop, one outstanding iteration per call, oldest
 *           first; *out = NULL once nothing is outstanding. */
bls_status_t bls_step(bls_plan_t *plan, int k, const int32_t *ids, const int32_t *offsets,
                      int64_t n_ids, const float **out /*host out*/, int64_t *out_iter /*host out*/);
bls_status_t bls_drain(bls_plan_t *plan, const float **out /*host out*/, int64_t *out_iter /*host out*/);

/* The same two calls with HOST input and output buffers: ids/offsets are copied
 * to a staging area of the ring (pinned memory recommended), and the iteration
 * handed back, if any, is copied to host_out (fp32 [P][b][T][dim]; may be NULL to
 * skip the copy).  The copies run asynchronously on two internal streams (upload of the
 * next iteration and download of the previous result overlap; with a bound k >= 1 - k >= 2 in
 * overlapped mode - and no injected delays the download of iteration t-k also runs beside the
 * kernels of iteration t, which work on other slots of the ring); the plan's stream waits for
 * them, so synchronising it, or enqueuing work on it, after the call sees host_out complete.
 * The host buffers must stay untouched until then. */
bls_status_t bls_step_host(bls_plan_t *plan, int k, const int32_t *ids /*host*/,
                           const int32_t *offsets /*host*/, int64_t n_ids,
                           float *host_out /*host*/, int64_t *out_iter /*host out*/);
bls_status_t bls_drain_host(bls_plan_t *plan, float *host_out /*host*/, int64_t *out_iter /*host out*/);

/* ---- inspection (bls_view, bls_counters, bls_status, bls_set_poison, bls_set_wait_limit,
 * bls_profile*, bls_set_tuning, bls_set_overlap, bls_set_fused, bls_set_ring: debugging and measurement aids with no counterpart in the paper) ---- */
/* Device pointers of the slot that holds iteration `iter` (must still be in the ring). */
bls_status_t bls_view(bls_plan_t *plan, int64_t iter, bls_route_view_t *view /*host out*/);
/* Synchronises the stream; copies the P per-rank counters to host arrays (may be NULL). */
bls_status_t bls_counters(bls_plan_t *plan, int64_t *posted, int64_t *served, int64_t *done);
/* Synchronises the stream and returns the first latched device condition (BLS_OK if none);
 * *max_lag (may be NULL) receives the largest distance ever seen between the newest
 * posted iteration and the oldest incomplete one. */
bls_status_t bls_status(bls_plan_t *plan, int64_t *max_lag /*host out*/);
/* Injected delay of rank `rank` before each of its iterations (Section V-E,
 * setting 2: a delay models a slowdown of any nature), in nanoseconds.  As in Listing 2's
 * loop the delay of iteration j + 1 starts when the rank has posted iteration j and has
 * at most k requests outstanding; the rank posts iteration j + 1 when the delay is over.
 * From the first injected delay on, the plan works with the persistent ring kernel (bls_set_ring). */
bls_status_t bls_set_stall(bls_plan_t *plan, int rank, int64_t ns);
/* The paper's random-delay setting: in addition to the fixed delay, rank `rank` is
 * delayed before each of its iterations by a time drawn uniformly from [0, max_ns]
 * (a counter-based draw from `seed`, the rank and the iteration number, so a run
 * can be repeated).  The seed is shared by all ranks of the plan. */
bls_status_t bls_set_random_stall(bls_plan_t *plan, int rank, int64_t max_ns, uint64_t seed);
/* The persistent ring kernel.  While delays are injected, every bls_step / bls_drain call is
 * ONE cooperative kernel launch in which each logical rank runs the loop of Listing 2 on its own
 * (Section III-C: initiation never synchronises two ranks): it spends its delay, completes the
 * requests that have arrived, posts as soon as the slot of its next iteration is free (every
 * rank has completed the iteration k + 1 before it), and blocks on its oldest request only while
 * more than k are outstanding; owners answer an iteration as soon as all ranks have posted it.
 * A scheduler warp publishes this work to the other blocks of the launch through a queue in the
 * workspace; the launch ends once the call's iteration (t - k, or the drained one) is complete
 * on every rank and nothing else can be done at that moment.  Results are the same bit for bit.
 * mode -1 (default): only while delays are injected; 0: also for iterations below about 128 K
 * lookups (one launch instead of three dependent ones), unless bls_set_overlap(1) was asked for;
 * 1: always.  Only between loops (nothing outstanding), else BLS_ESTATE. */
bls_status_t bls_set_ring(bls_plan_t *plan, int mode);
/* Time stamps (device clock, ns) of the last 1024 iterations, for the per-rank latency and
 * throughput the paper reports (Section V-C): for iterations first_iter .. first_iter + n_iter - 1
 * and every rank r, when r's post of the iteration was complete, when owner r had answered it,
 * and when r completed it.  Host arrays of n_iter * P entries indexed [i * P + r], any may be
 * NULL.  Synchronises the stream.  BLS_ESTATE if an iteration has not been issued yet or is more
 * than 1024 iterations old. */
bls_status_t bls_timeline(bls_plan_t *plan, int64_t first_iter, int n_iter, uint64_t *post_ns /*host out*/,
                          uint64_t *serve_ns /*host out*/, uint64_t *done_ns /*host out*/);
/* Overlapped mode of bls_step (see there): mode 0 (default) uses it for iterations of about a
 * million lookups or more (P * max_ids_per_rank >= 2^20; smaller ones are bound by the launch
 * rate and lose to the second stream's extra driver calls), 1 whenever it applies (bound >= 1,
 * table-wise placement, no injected delays, no hot-row staging, ring kernel not in use), -1 never.
 * May be called at any time. */
bls_status_t bls_set_overlap(bls_plan_t *plan, int mode);
/* One-launch iterations (see bls_step): mode 0 (default) uses the fused kernel when an iteration
 * holds fewer than about 256 K lookups (P * max_ids_per_rank < 2^18: below that the launches of a
 * wave cost more than the work in them; < 2^20 when max_ids_per_rank allows at most four IDs per bag on
 * average, where routing and answering a tile in one go stays ahead for longer), 1 whenever it applies (table-wise placement, no injected
 * delays, ring kernel and overlapped mode not in use, no hot-row staging, default tuning), -1 never.
 * May be called at any time. */
bls_status_t bls_set_fused(bls_plan_t *plan, int mode);
/* Debug aid: while enabled, the output slot an iteration is issued into is first filled
 * with 0xFF bytes (NaN), so that a bag that was not written, or a slot read before its data
 * arrived, shows up in the result.  Costs one pass over the slot per step. */
bls_status_t bls_set_poison(bls_plan_t *plan, int enable);
/* Upper limit of any single device-side wait (default 2 s).  In the ring kernel: after this long
 * without any progress (no rank changed state, no tile of work finished) the scheduler latches
 * BLS_ETIMEOUT and stops honouring injected delays, so the loop still completes with correct data;
 * after a second such period it ends the launch.  A worker block that finds no work for four
 * times the limit plus one second leaves.  Waits on mbarriers (bulk-copy gather variant, linear
 * layers) give up after 2 s of their own. */
bls_status_t bls_set_wait_limit(bls_plan_t *plan, int64_t ns);

/* Stage timing with CUDA events on the plan's stream.  While enabled, every
 * bls_step/bls_drain records events around its three stages (up to 1024 calls
 * are kept).  bls_profile_read synchronises the stream, adds up the recorded
 * calls into milliseconds per stage (gate + router kernels, the gather-pool-return
 * kernel including the commit done by its last block, anything after it), reports how
 * many calls were summed and how many kernels the plan has launched so far, and clears
 * the record.  Any pointer may be NULL.  A call served by the ring kernel is one launch: its
 * whole time is reported under the gather stage. */
bls_status_t bls_profile(bls_plan_t *plan, int enable);
bls_status_t bls_profile_read(bls_plan_t *plan, double *ms_route, double *ms_gather, double *ms_ring,
                              int64_t *calls, int64_t *kernels);

/* Tuning of the gather-pool kernel (results do not depend on it): bags_per_run =
 * consecutive sub-bags one lane group streams (0 = keep; default 4 to 24, about 160 rows'
 * worth for table-wise and 50 for row-wise placement), rows_in_flight = row loads per
 * batch, 4 or 8 (0 = keep; default 4).  16 or 32 (table-wise placement, rows of 64 bytes or
 * more) select the variant that stages rows in shared memory with the bulk-copy engine
 * (cp.async.bulk, one copy per row, 2 or 4 stages of 8 rows per lane group, completion
 * counted on an mbarrier with a bounded wait); measured slower than the default on the
 * benchmark workloads, kept as an option. */
bls_status_t bls_set_tuning(bls_plan_t *plan, int bags_per_run, int rows_in_flight);

/* ---- hot-row staging (optional; table-wise placement only) ----
 * Power-law ID distributions put most lookups on a few hundred rows per table.
 * After bls_hot_build the router marks, for every packed lookup, the slot of its
 * row in the table's hot list, and the gather kernel keeps the listed rows of the
 * table it is working on in shared memory.  Pooled results are unchanged (a staged
 * row is a copy of the table row).  The paper calls caching orthogonal to its
 * collective (Section II); this is an internal optimisation of step (2).
 *   bls_hot_bytes    size of the caller-provided device buffer for `rows_per_table` slots
 *   bls_hot_attach   hand over that buffer (device, 256-byte aligned, borrowed until
 *                    bls_destroy); rows_per_table * row bytes must fit in shared memory
 *                    (<= 200 KiB), nothing may be outstanding; synchronises the stream
 *   bls_hot_observe  add one batch of IDs (device, same layout as bls_step's) to the
 *                    per-row request counts; asynchronous
 *   bls_hot_build    select per table the most requested rows (at most rows_per_table,
 *                    cut at a count threshold) and switch staging on; asynchronous;
 *                    nothing may be outstanding
 *   bls_hot_view     device pointers to the lists: rows int32 [T][rows_per_table] in slot
 *                    order, count int32 [T] */
bls_status_t bls_hot_bytes(bls_plan_t *plan, int rows_per_table, size_t *bytes /*host*/);
bls_status_t bls_hot_attach(bls_plan_t *plan, int rows_per_table, void *buffer, size_t bytes);
bls_status_t bls_hot_observe(bls_plan_t *plan, const int32_t *ids, const int32_t *offsets, int64_t n_ids);
bls_status_t bls_hot_build(bls_plan_t *plan);
bls_status_t bls_hot_view(bls_plan_t *plan, const int32_t **rows /*host out*/, const int32_t **count /*host out*/,
                          int *rows_per_table /*host out*/);

const char *bls_strerror(int status);

/* ---- input generation helper (not part of the method) ----
 * Fill rows [0, rows) of table `t` with the counter-hash values used by the
 * synthetic workloads: SplitMix64 output number (t<<48 | row<<16 | c) + 1 for
 * `seed`, four 16-bit fields summed, minus 131070, times 1/sqrt((65536^2-1)/3)
 * in fp32, rounded to nearest even into `dtype`. */
bls_status_t bls_fill_hash_table(void *weight, int64_t rows, int32_t dim, int32_t dtype,
                                 uint64_t seed, int32_t t, void *cuda_stream);

/* ---- the collective on its own: BLS alltoallv of raw bytes (Section III-C) ----
 * P logical ranks exchange byte segments.  bls_a2a_post initiates request j: rank src's
 * segment for dst (sendcounts[src][dst] bytes at sendbuf + src*send_stride +
 * sdispls[src][dst]) is put into dst's receive buffer of slot j mod (k_max+1) at
 * rdispls[dst][src] = sum of the counts of lower-ranked sources, and the arrival is
 * counted; nothing waits.  bls_a2a_wait completes the OLDEST outstanding request (it
 * checks that every receiver counted P messages) and hands out its slot: *recv (device,
 * rank dst at dst*recv_stride), *recvcounts / *rdispls (device, int64 [P][P] indexed
 * [dst][src]), valid until k_max+1 further posts.  At most k_max+1 requests may be
 * outstanding (BLS_ESTATE otherwise): k_max = 0 is a plain alltoallv.
 *   workspace        device, 256-byte aligned, bls_a2a_bytes() long, borrowed
 *   sendbuf/sendcounts/sdispls  device; counts and displacements are int64 [P][P] in bytes
 *   max_segment_bytes host hint: the largest sendcounts entry.  It only sizes the launch:
 *                    a segment longer than the hint is still copied whole
 * A segment whose count or displacement leaves the sender's stride (BLS_EINVAL), or that no
 * longer fits behind the accepted segments of lower-ranked sources in the receiver's buffer
 * (BLS_ENOSPC), is rejected: it arrives as an empty segment (recvcounts 0), the receiver
 * counts one message fewer, and bls_a2a_wait's check then also latches BLS_ESTATE.
 * Asynchronous on the stream; device-detected conditions (segment outside the send
 * stride: BLS_EINVAL, receive capacity exceeded: BLS_ENOSPC) via bls_a2a_status, which
 * synchronises. */
typedef struct bls_a2a bls_a2a_t;
bls_status_t bls_a2a_bytes(int P, int k_max, int64_t max_bytes_per_rank, size_t *bytes /*host*/);
bls_status_t bls_a2a_create(int P, int k_max, int64_t max_bytes_per_rank, void *workspace, size_t bytes,
                            void *cuda_stream, bls_a2a_t **handle /*host out*/);
void bls_a2a_destroy(bls_a2a_t *handle);
bls_status_t bls_a2a_post(bls_a2a_t *handle, const void *sendbuf, int64_t send_stride,
                          const int64_t *sendcounts, const int64_t *sdispls, int64_t max_segment_bytes);
bls_status_t bls_a2a_wait(bls_a2a_t *handle, const void **recv /*host out*/, int64_t *recv_stride /*host out*/,
                          const int64_t **recvcounts /*host out*/, const int64_t **rdispls /*host out*/,
                          int64_t *request /*host out*/);
bls_status_t bls_a2a_status(bls_a2a_t *handle);

/* ---- the dense stages either side of the lookup (Section IV, Listing 1 / Listing 2) ----
 * Listing 1 runs the bottom MLP on the dense features between the alltoall and its wait, then
 * the feature interaction of its output with the pooled vectors and the top MLP; Listing 2 lets
 * those stages of batch j run beside the exchange of later batches (Table I).  These calls are
 * stand-ins for those stages with weights the caller provides (the paper takes them from the
 * reference DLRM and does not restate them); all buffers are DEVICE memory.
 *
 * An MLP is n_layers linear layers y = act(x W^T + bias): dims[0] inputs, dims[i+1] outputs of
 * layer i; weights[i] is bf16 [dims[i+1]][dims[i]] row-major, 16-byte aligned; bias[i] fp32
 * [dims[i+1]]; every dims[i] with i < n_layers is a multiple of 8.  Hidden layers use ReLU, the
 * last layer last_act (0 none, 1 ReLU, 2 logistic function).  Activations are bf16 between
 * layers, sums are fp32 (tensor cores: tcgen05.mma fed by TMA tile loads, accumulator in tensor
 * memory).  The workspace (bls_mlp_bytes, 256-byte aligned, borrowed until bls_mlp_destroy)
 * holds the hidden activations of up to max_rows rows; weights and biases are borrowed too.
 *   bls_mlp_forward  x bf16 [rows][ldx] (ldx a multiple of 8, >= dims[0], 16-byte aligned base)
 *                    -> y [rows][ldy]: bf16, or fp32 when y_fp32.  Asynchronous on cuda_stream;
 *                    calls that use the same handle must not overlap on the GPU.
 *   bls_interact     x bf16 [rows][ldx] (the bottom MLP's output, D columns used), pooled fp32
 *                    [rows][T][D] (a slot of the ring: out[src][s][t][:] is [rows = P*b][T][D])
 *                    -> r bf16 [rows][ldr]: the D values of x, then the dot products
 *                    <v_i, v_j>, i = 1..T, j < i, of v_0 = x and v_1..v_T = the pooled vectors
 *                    (strictly lower triangle, row-major), then zeros up to ldr
 *   bls_mlp_status   synchronises cuda_stream; BLS_ETIMEOUT if a bounded wait inside a kernel gave up */
typedef struct bls_mlp bls_mlp_t;
bls_status_t bls_mlp_bytes(int n_layers, const int *dims /*host*/, int max_rows, size_t *bytes /*host*/);
bls_status_t bls_mlp_create(int n_layers, const int *dims /*host*/, const void *const *weights /*host array of device ptrs*/,
                            const float *const *bias /*host array of device ptrs*/, int last_act, int max_rows,
                            void *workspace, size_t bytes, void *cuda_stream, bls_mlp_t **handle /*host out*/);
void bls_mlp_destroy(bls_mlp_t *handle);
bls_status_t bls_mlp_forward(bls_mlp_t *handle, const void *x, int ldx, int rows, void *y, int ldy, int y_fp32,
                             void *cuda_stream);
bls_status_t bls_interact(const void *x, int ldx, const float *pooled, int rows, int T, int D, void *r, int ldr,
                          void *cuda_stream);
bls_status_t bls_mlp_status(bls_mlp_t *handle, void *cuda_stream);

/* ---- allocation-free router (the paper has no counterpart: this entry point
 * exists for deployment reasons only) ----
 * Step (1) for table-wise round-robin placement, for callers that cannot
 * allocate device memory and therefore cannot provide a plan's workspace: code
 * embedded in a server or framework that owns all device memory, plugins that
 * receive fixed buffers, and loops where cudaMalloc's device-wide
 * synchronisation or its failure under a full pool is unacceptable.  The call
 * uses no workspace and calls no allocator: its only scratch (the start of each
 * (requester, table) chunk) lives in a 128 KiB static device array inside the
 * library, which every GPU that loads the library holds until the process exits.
 *
 *   table_rows  device, int64 [T]: table heights (for the ID range check)
 *   ids/offsets device, as everywhere else; n_ids = offsets[P*T*local_batch]
 *   sendcounts, sdispls  device out, int32 [P][P] indexed [src][dst]
 *   sendbuf     device out, int32 [P][cap]: rank src's packed send buffer at src*cap
 *   sub_start   device out, int32 [P][T*local_batch + 1], ordered (dst, table, sample)
 *   status      device out, one int32: 0, or an OR of 1 (malformed offsets or a table
 *               height below 1), 2 (cap too small), 4 (ID out of range, replaced by row 0)
 * Results are identical to bls_route + bls_view on a table-wise plan.
 *
 * Limits and rules: P * (T + 1) <= 32768, else BLS_ENOSPC.  The first call on a
 * device looks up the scratch array's device address (with that device current);
 * make that first call before any stream capture.  All calls on a device share
 * the array, which keeps the last call's contents; the part in use is cleared at
 * the start of each call.  Calls whose GPU work may overlap (other streams or
 * host threads) race on it: serialise them.  Asynchronous on `cuda_stream`. */
bls_status_t bls_route_table_rr_static(const int64_t *table_rows, int T, int P, int local_batch,
                                       const int32_t *ids, const int32_t *offsets, int64_t n_ids,
                                       int32_t *sendcounts, int32_t *sdispls, int32_t *sendbuf,
                                       int64_t cap, int32_t *sub_start, int32_t *status,
                                       void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BLS_H */
