/*
 * ec.h - eventually consistent collectives on one B200: C ABI.
 *
 * P simulated ranks live as buffers in one GPU's memory.  Every (rank, segment)
 * contribution carries an arrival notification (one bit).  The collectives
 * produce their result from whatever has arrived, report how much took part,
 * and fold late contributions in when they land.
 *
 * General rules for every entry point
 *   - extern "C"; returns int: EC_OK (0) or a negative EC_ERR_* code.  Nothing
 *     throws, exits, or synchronises the device.
 *   - "device" pointers are CUDA device addresses valid on the current device;
 *     "host" pointers are ordinary process memory.  The caller owns every buffer
 *     it passes; the library owns only its context objects (and a workspace it
 *     allocated itself when the caller passed none).
 *   - All device work is enqueued on `stream` (a cudaStream_t; NULL = the legacy
 *     default stream).  Buffers and notification words must stay valid and
 *     unmodified until that work has completed.  Notification words are read on
 *     the device when the kernel runs, so a producer may set bits in stream
 *     order right up to the call (Sec. II: data is written as soon as it exists and
 *     its arrival is looked at as late as possible).
 *   - A context is not thread-safe and expects its calls in one stream order;
 *     distinct contexts are independent.
 *
 * Notification words (Sec. II: data is usable once its notification is
 * visible): uint64 [S][W] on the device, W = ceil(P/64); the notification of
 * rank r for segment s is bit (r % 64) of word [s][r / 64].  Bits at or above P
 * are ignored.  Words are cumulative inside an epoch; a bit that is cleared
 * after its contribution was folded in is ignored (nothing is un-applied).
 * A contribution whose bit is 0 is never read.
 */
#ifndef EC_H_
#define EC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* ec_stream_t; /* the same type as cudaStream_t */

typedef enum {
    EC_F32 = 0,  /* fp32 in, fp32 accumulate, fp32 out */
    EC_BF16 = 1, /* raw bfloat16 bits in, widened exactly, fp32 accumulate, fp32 out */
    EC_I64 = 2,  /* int64 in/out; sum wraps modulo 2^64 */
    EC_F64 = 3   /* fp64 in/out (the element type of the paper's experiments) */
} ec_dtype_t;

typedef enum {
    EC_SUM = 0, /* the paper's "global sum" (Sec. IV-A) */
    EC_MAX = 1, /* acc = (x > acc) ? x : acc */
    EC_MIN = 2  /* acc = (x < acc) ? x : acc */
} ec_op_t;

typedef enum {
    EC_ORDER_FIXED = 0,   /* each apply folds its new ranks in ascending rank order: reproducible bits */
    EC_ORDER_PAIRWISE = 1, /* balanced tree over the rank index (float sum only): smaller rounding error; for P a power
                              of two this is the order of the hypercube allreduce of Sec. III-A (recursive doubling) */
    EC_ORDER_RING = 2      /* the order of the segmented pipelined ring (Sec. IV-A, Scatter-Reduce): the vector is cut
                              into P chunks of ceil(n/P) elements; chunk c is first sent by node c and reduced by nodes
                              c+1, c+2, ... in turn, so its fold runs over the ranks c, c+1, ..., P-1, 0, ..., c-1
                              (each apply folds its new ranks in that cyclic order).  segment_size must divide
                              ceil(n/P) (EC_ERR_INVALID otherwise) */
} ec_order_t;

enum {
    EC_OK = 0,
    EC_ERR_INVALID = -1,     /* NULL / zero / inconsistent argument */
    EC_ERR_UNSUPPORTED = -2, /* combination of dtype, op and order that is not implemented */
    EC_ERR_CUDA = -3,        /* a CUDA runtime call failed; see ec_last_cuda_error() */
    EC_ERR_STATE = -4,       /* call not allowed in the context's current state */
    EC_ERR_CAPACITY = -5     /* a size exceeds a stated limit or a workspace is too small */
};

#define EC_MAX_RANKS 1024 /* largest P any call accepts */

typedef struct ec_ctx ec_ctx_t;
typedef struct ec_kmeans ec_kmeans_t;

/* ------------------------------------------------------------------------- *
 * Eventually consistent allreduce.
 *
 * Follows the Scatter-Reduce stage of the segmented pipelined ring (Sec. IV-A):
 * the vector is cut into segments that are reduced independently, here all on
 * one device, so the P-1 ring steps of a segment collapse into one pass over
 * the P rank buffers.  The consistency rule is the paper's (Sec. II, Sec. III):
 * only notified contributions are used; the status output says how many ranks
 * are in each segment's result ("threshold" and "status" parameters); once
 * every notification has been seen the result is the complete reduction
 * (end of Sec. IV-A).
 *
 * n elements per rank, segments of segment_size elements (the last may be
 * short), S = ceil(n / segment_size).
 * ------------------------------------------------------------------------- */

/* Bytes of device workspace a context needs (two copies of the "already folded
 * in" words, 256-byte aligned).  0 on invalid arguments. */
size_t ec_allreduce_workspace_bytes(int P, size_t n, size_t segment_size);

/* Create a context.  `workspace` is device memory of at least
 * ec_allreduce_workspace_bytes() bytes, 256-byte aligned, owned by the caller
 * and kept alive until destroy; NULL lets the library cudaMalloc it (and free it
 * in destroy).  The workspace is cleared with a cudaMemsetAsync on the legacy
 * default stream followed by a stream synchronise, so init must not be called
 * during stream capture.  Pairwise order is accepted only for EC_SUM on a
 * floating dtype (else EC_ERR_UNSUPPORTED). */
int ec_allreduce_init(ec_ctx_t** ctx, int P, size_t n, ec_dtype_t dtype, ec_op_t op, size_t segment_size,
                      ec_order_t order, void* workspace, size_t workspace_bytes);

/* One apply = one round: fold every contribution that is notified now and was
 * not folded in by an earlier apply of this epoch.
 *
 *   rank_bufs      HOST array of P DEVICE pointers; rank r's vector of n elements
 *                  of the context's input type.  Read during the call (copied
 *                  into the launch), so it may be reused at once.
 *   P, n, dtype, op, segment_size
 *                  must equal the values given to init (EC_ERR_INVALID if not).
 *   arrival_mask   device uint64 [S][W]; NULL means everything has arrived.
 *   result         device, n elements of the output type (fp32 for EC_F32 and
 *                  EC_BF16, int64, fp64).  In/out across the applies of an epoch.
 *                  Must not alias a rank buffer.
 *   contrib_count  device uint32 [S], or NULL.  After the call contrib_count[s]
 *                  = number of ranks folded into segment s so far this epoch
 *                  (= popcount of the cumulative words restricted to bits < P).
 *
 * Per segment: if no rank was folded in before, the accumulator starts from the
 * operator's identity (+0.0; -inf / +inf; 0; INT64_MIN / INT64_MAX) and `result`
 * is not read; otherwise it starts from `result`.  The new ranks are folded in
 * ascending rank order (EC_ORDER_FIXED) or as a balanced tree whose root is then
 * added (EC_ORDER_PAIRWISE).  The first apply of an epoch writes the identity to
 * segments without any contribution, so `result` is fully defined after it;
 * later applies neither read nor write segments without new arrivals.
 *
 * 16-byte aligned pointers together with segment_size * sizeof(input element)
 * divisible by 16 take the 128-bit path; anything else is still correct through
 * an element-wise path.  One kernel launch, no allocation. */
int ec_allreduce_apply(ec_ctx_t* ctx, const void* const* rank_bufs, int P, size_t n, ec_dtype_t dtype,
                       ec_op_t op, size_t segment_size, const uint64_t* arrival_mask, void* result,
                       uint32_t* contrib_count, ec_stream_t stream);

/* Stale-synchronous apply (Sec. III-A, Algorithm 1 "allreduce_ssp").
 *
 * In the paper every process keeps, per communication step, the last contribution it received
 * together with the logical clock (iteration number) in which that contribution was computed, and
 * uses it instead of waiting as long as its clock is not below min_clock_accepted = clock - slack.
 * Here rank r's buffer plays the part of that dedicated receive memory: it holds whatever rank r
 * wrote last for a segment, and notif_clock says how old that is.
 *
 *   notif_clock    device uint32 [S][P]: clock of the contribution that rank_bufs[r] holds for
 *                  segment s; 0 = nothing received yet.  Read on the device when the kernel runs.
 *   clock, slack   the caller's current clock (>= 1) and the allowed staleness.
 *   result         device, n output elements, written in full: per segment the reduction, in
 *                  ascending rank order starting from the identity, of every contribution with
 *                  notif_clock >= clock - slack (slack = 0 is the classic synchronous allreduce).
 *   contrib_count  device uint32 [S] or NULL: number of contributions used.
 *   seg_clock      device uint32 [S] or NULL: the clock of the reduction = the smallest clock among
 *                  the contributions used (0 if none): Sec. III-A gives a reduction the smaller of
 *                  the clocks of what went into it.
 *   wait_count     device uint32 [S] or NULL: contributions that were too stale (or absent).  The
 *                  paper's process blocks on those; this call never waits - it reports them, and
 *                  the caller applies again once they have been refreshed.
 *
 * The call keeps no state: it neither reads nor changes what ec_allreduce_apply has folded in.
 * P, n, dtype, op, segment_size must equal the context's.  One kernel launch, no allocation. */
int ec_allreduce_ssp_apply(ec_ctx_t* ctx, const void* const* rank_bufs, int P, size_t n, ec_dtype_t dtype,
                           ec_op_t op, size_t segment_size, const uint32_t* notif_clock, uint32_t clock,
                           uint32_t slack, void* result, uint32_t* contrib_count, uint32_t* seg_clock,
                           uint32_t* wait_count, ec_stream_t stream);

/* Start a new epoch: forget which contributions were folded in (the counterpart
 * of resetting notifications, Sec. II / Sec. IV-B).  `result` is not touched; the
 * next apply overwrites it. */
int ec_allreduce_reset(ec_ctx_t* ctx, ec_stream_t stream);

/* One whole epoch from HOST memory (Sec. IV-B: a reset followed by an apply each
 * time more contributions have come in, here `rounds` of them).
 *
 *   host_rank_bufs  HOST array of P HOST pointers, n elements of the context's
 *                   dtype each; pinned memory makes the copies asynchronous.
 *   host_masks      HOST array of `rounds` HOST pointers, each a cumulative
 *                   notification mask uint64 [S][W] as in ec_allreduce_apply.
 *   host_result     HOST, n elements of the accumulator type; written.
 *   host_contrib_count  HOST uint32 [S] after the last round, or NULL.
 *   staging         DEVICE scratch of at least ec_allreduce_host_staging_bytes
 *                   (ctx, rounds) bytes, 256-byte aligned, owned by the caller;
 *                   it holds the uploaded buffers, masks, the result and counts.
 *
 * Everything is enqueued on `stream` (P + rounds uploads, `rounds` applies, the
 * read-back); the host arrays are valid once the stream has been synchronised.
 * Two calls on two streams need two staging areas and two contexts.  Errors as
 * in ec_allreduce_apply; EC_ERR_CAPACITY for a staging area that is too small or
 * misaligned. */
size_t ec_allreduce_host_staging_bytes(const ec_ctx_t* ctx, int rounds);
int ec_allreduce_epoch_host(ec_ctx_t* ctx, const void* const* host_rank_bufs, const uint64_t* const* host_masks,
                            int rounds, void* host_result, uint32_t* host_contrib_count, void* staging,
                            size_t staging_bytes, ec_stream_t stream);

/* Expert knob: elements of one segment handled per thread block (rounded to the
 * vector width) and threads per block (64..256, multiple of 32).  0 keeps the
 * current value.  Affects speed only, never results. */
int ec_allreduce_set_tile(ec_ctx_t* ctx, int threads, size_t tile_elems);

/* Expert knob: 1 = the tiles of the rank buffers are staged through shared memory
 * by bulk asynchronous copies (the default for up to 64 ranks, in every order;
 * EC_ERR_UNSUPPORTED for more ranks); 0 = they are read with direct
 * 128-bit loads.  Calls that cannot take the 128-bit path, and short segments,
 * use the direct kernels whatever the setting.  Affects speed only, never results. */
int ec_allreduce_set_path(ec_ctx_t* ctx, int path);

/* Free the context (and its workspace if the library allocated it).  The caller
 * makes sure no work of this context is still running. */
int ec_allreduce_destroy(ec_ctx_t* ctx);

/* ------------------------------------------------------------------------- *
 * Eventually consistent allgatherv.
 *
 * Every rank owns a fixed slot, as every chunk has a fixed place in the ring's
 * Allgather stage (Sec. IV-A) and every writer its own target and notification
 * in the AlltoAll (Sec. IV-B): displs is the exclusive prefix sum of the counts
 * of ALL ranks, arrived or not, and displs[P] the total.  Ranks whose bit is
 * set are copied into their slot; the slots of the others are left untouched
 * (a late rank is one more call with its bit set).  Stateless.
 *
 *   bufs           HOST array of P DEVICE pointers (rank r: counts[r] elements).
 *                  Entries of ranks that are not notified may be NULL.
 *   counts         device int64 [P], each >= 0.
 *   dtype          element type (sets the element size: 4, 2, 8, 8 bytes).
 *   arrival_mask   device uint64 [W], one bit per rank; NULL = all arrived.
 *   displs         device int64 [P+1], written.
 *   out            device, out_capacity_elems elements.
 *   status         device uint32, written: 0 = done; 1 = the total exceeds
 *                  out_capacity_elems or a count is negative - then displs is
 *                  still written but not a byte of `out`.
 * One kernel launch (prefix sum and copy fused), no allocation. */
int ec_allgatherv(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype,
                  const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity_elems,
                  uint32_t* status, ec_stream_t stream);

/* The other reading of "packed": only the ranks that have arrived get a slot, so the
 * arrived contributions are contiguous from out[0] on.  displs is the exclusive prefix sum
 * of (arrived ? counts[r] : 0); displs[P] = number of elements gathered.  Unlike the fixed-slot
 * form above, a rank that arrives later moves every slot behind it, so a later call rewrites
 * the whole output from the then-current notification word.  Same arguments and status rules. */
int ec_allgatherv_compact(const void* const* bufs, const int64_t* counts, int P, ec_dtype_t dtype,
                          const uint64_t* arrival_mask, int64_t* displs, void* out, size_t out_capacity_elems,
                          uint32_t* status, ec_stream_t stream);

/* ------------------------------------------------------------------------- *
 * Eventually consistent AlltoAll (Sec. IV-B): every rank writes its d-th block
 * into rank d's receive memory, each write with a notification of its own; the
 * receiver uses what has been notified and the collective is complete once all
 * P blocks of every receiver have arrived.
 *
 *   send_bufs      HOST array of P DEVICE pointers: rank s's P blocks of
 *                  block_bytes bytes, block d destined for rank d.
 *   recv_bufs      HOST array of P DEVICE pointers: rank d's P slots of
 *                  block_bytes bytes; slot s receives the block from rank s.
 *                  No receive buffer may be a send buffer.
 *   arrival_mask   device uint64 [P][W]: row d = destination, bit s = the block
 *                  from rank s has arrived; NULL = all.  Slots whose bit is
 *                  clear are left untouched (a late block is one more call with
 *                  its bit set).
 *   recv_count     device uint32 [P] or NULL: notified blocks per destination
 *                  (= P when that rank's AlltoAll is complete).
 * Stateless; one kernel launch; 128-bit copies when block_bytes and all pointers
 * are multiples of 16, byte-wise otherwise. */
int ec_alltoall(const void* const* send_bufs, void* const* recv_bufs, int P, size_t block_bytes,
                const uint64_t* arrival_mask, uint32_t* recv_count, ec_stream_t stream);

/* ------------------------------------------------------------------------- *
 * K-means driver: Lloyd iterations whose combine step is the allreduce above.
 * (The paper's iterative-convergent ML workload is a matrix factorisation on a
 * data set that is not available; K-means takes its place as the data-parallel
 * solver that tolerates missing contributions, Sec. I and Sec. III.)
 *
 * N points of D coordinates, row-major fp32 [N][D]; K centroids fp32 [K][D];
 * rank r owns points [r*N/P, (r+1)*N/P).  Per-rank partials are fp32
 * [P][K][D+4]: columns 0..D-1 the coordinate sums of the rank's points with that
 * label, column D their number, D+1..D+3 zero.  One iteration = assignment
 * (label = nearest centroid by squared Euclidean distance computed as
 * sum_d (x-c)^2 in fp32, lowest index on a tie), partials, one allreduce epoch
 * (reset + one apply, segment = one centroid row of D+4 elements, so a rank's
 * sums and count for a centroid arrive together; contributions that are not
 * notified are dropped for this iteration), centroid update (sum / points; a
 * centroid without points stays where it was).
 * Limits: 1 <= D <= 128 and D % 4 == 0; 1 <= K <= 1024; 1 <= P <= EC_MAX_RANKS.
 * ------------------------------------------------------------------------- */
size_t ec_kmeans_workspace_bytes(size_t N, int D, int K, int P);

/* points and init_centroids are device pointers; points must stay valid for the
 * life of the context (they are not copied), init_centroids are copied in on the
 * legacy default stream (synchronised before return).  workspace as for the
 * allreduce (NULL = library allocates). */
int ec_kmeans_init(ec_kmeans_t** km, const float* points, size_t N, int D, int K, int P,
                   const float* init_centroids, void* workspace, size_t workspace_bytes);

/* Assignment alone: labels[j] for the given device centroids [K][D]. */
int ec_kmeans_assign(ec_kmeans_t* km, const float* centroids, int32_t* labels, ec_stream_t stream);

/* Partials alone: device labels [N] -> device partials [P][K][D+4].  Sums are
 * accumulated in a fixed order (no floating-point atomics): same bits every run. */
int ec_kmeans_partials(ec_kmeans_t* km, const int32_t* labels, float* partials, ec_stream_t stream);

/* One full iteration on the context's own centroids.  arrival_mask: device
 * uint64 [K][W] for this iteration, NULL = all arrived.
 * The context keeps the labels and the per-rank sums between iterations; on the
 * tensor-core path (D = 16 or 32, K <= 256) an iteration after the first adds to
 * the sums only what changed - +x for the cluster a point joins, -x for the one
 * it leaves - and every 32nd iteration sums everything afresh, which bounds the
 * rounding the running sums collect (about 2^-24 of a sum per iteration; counts
 * stay exact).  Those iterations also skip the search of points whose label
 * provably cannot change (ec_kmeans_set_bounds below).  Results repeat bit for
 * bit from run to run either way. */
int ec_kmeans_iterate(ec_kmeans_t* km, const uint64_t* arrival_mask, ec_stream_t stream);

/* The same iteration with the combine step spread over several rounds: one allreduce epoch with
 * `rounds` applies (1..64) before the centroid update.  arrival_masks is a HOST array of `rounds`
 * DEVICE pointers to cumulative notification words [K][W] (an entry may be NULL = all arrived);
 * rows that are late in round 1 still count if a later round of the same iteration sees them. */
int ec_kmeans_iterate_rounds(ec_kmeans_t* km, const uint64_t* const* arrival_masks, int rounds, ec_stream_t stream);

/* Replace the context's centroids (device [K][D]); used for lock-step checks.  The next iteration
 * searches every point again (the distance bounds do not know how far the centroids were moved). */
int ec_kmeans_set_centroids(ec_kmeans_t* km, const float* centroids, ec_stream_t stream);

/* Copy out (device to device, on `stream`) whichever outputs are non-NULL:
 * centroids [K][D], labels [N] and reduced [K][D+4] and contrib_count [K] of the
 * last iteration. */
int ec_kmeans_get(ec_kmeans_t* km, float* centroids, int32_t* labels, float* reduced,
                  uint32_t* contrib_count, ec_stream_t stream);

/* Expert knob: on the tensor-core path every `every`-th iteration sums all points
 * afresh and the iterations in between only what changed (default 32; 1 = every
 * iteration sums everything, the running sums are not used).  The next iteration
 * after this call is a full one.  EC_ERR_INVALID for every < 1. */
int ec_kmeans_set_refresh(ec_kmeans_t* km, int every);

/* Distance bounds (on by default; tensor-core kernel only).  Between full passes the driver keeps, for every
 * point, an upper bound on the distance to its own centroid and a lower bound on the distance to every other
 * one, and for every centroid how far it has moved since.  A tile of 128 points whose bounds show that no label
 * can change is not read in that iteration (triangle inequality; all roundings directed, and a margin far above
 * the rounding of the exact form), so labels, sums and centroids are the same as without the bounds; only the
 * time changes: an iteration in which the centroids barely move reads 12 bytes per point instead of the points.
 * enable = 0 searches every tile in every iteration.  The paper has no counterpart (its K-means-like workloads
 * are not described at this level); the bounds are those of the textbook accelerations of Lloyd's algorithm. */
int ec_kmeans_set_bounds(ec_kmeans_t* km, int enable);

/* Expert knob: which kernel ec_kmeans_iterate / ec_kmeans_assign use.
 *   0  automatic: the fastest one that covers the shape (default); where both tensor-core kernels do, the kernel of 2
 *      for the assignment alone and for iterations that sum only changes, the kernel of 3 for an iteration that sums
 *      every point;
 *   1  fp32 fused kernel: candidate search by one FMA per (point, centroid, coordinate);
 *   2  tensor cores (D in {16, 32}, K <= 256): for K <= 128 the warp-specialised kernel - the fp32 points go from
 *      global to shared memory by bulk tensor copies and are multiplied as they lie (tcgen05, tf32) - otherwise
 *      the kernel of 3;
 *   3  tensor cores, register-staged form: points converted to bf16 by the threads, candidate search as a bf16 GEMM.
 * All decide every point whose two best candidates lie within the error bound of the search again
 * by the exact form sum_d (x-c)^2 in fp32, so labels do not depend on the choice; speed does.
 * ec_kmeans_tc_status reads a word that is nonzero if a bounded wait inside a tensor-core kernel ever gave up:
 * bit 0 - the kernel of 3 finished that tile in plain fp32 (results valid); bit 1 - the warp-specialised kernel
 * stopped early (the results of that call are not valid; the other bits say which wait it was).
 * EC_ERR_UNSUPPORTED if the shape is not covered by the requested kernel. */
int ec_kmeans_set_path(ec_kmeans_t* km, int path);

/* Copies (device to device, on `stream`) the driver's health word to `device_out`: 0 = fine; nonzero =
 * a bounded wait on the tensor core gave up at least once and the affected tiles were computed by the
 * exact form instead (results are still correct). */
int ec_kmeans_tc_status(ec_kmeans_t* km, uint32_t* device_out, ec_stream_t stream);

int ec_kmeans_destroy(ec_kmeans_t* km);

/* Per-rank partial sums for callers that are not allowed to allocate device
 * memory.  (An addition of this library; the paper has no counterpart.)
 *
 * Some callers cannot call cudaMalloc at the point where they need this step:
 * a serving process whose framework has claimed all device memory for its own
 * pool at start-up, so that a later cudaMalloc simply fails; a latency-critical
 * loop or a callback that must not block, while cudaMalloc and cudaFree
 * synchronise the whole device and take a process-wide lock; a plug-in whose
 * host forbids allocations outside its own allocator.  The context-based call
 * above needs a workspace (someone has to allocate it); this one needs none.
 *
 * It computes exactly what ec_kmeans_partials computes (same kernels, same
 * order of additions, same bits) from
 *   points    device fp32 [N][D]
 *   labels    device int32 [N]
 *   partials  device fp32 [P][K][D+4], written
 * with the same limits on N, D, K, P as the K-means driver.  The per-block
 * partial sums that the workspace would hold go to a fixed 8 MiB array inside
 * the library image (every GPU that loads the library holds those 8 MiB until
 * the process ends).  Shapes whose per-block sums need more than 8 MiB are
 * rejected with EC_ERR_CAPACITY before anything is launched (for the K-means
 * workload of the benchmark they need 2.4 MB).
 *
 * The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating
 * library routine.  The first call on each device looks up the device address
 * of the array and raises the kernel's shared-memory limit; make that first
 * call before starting any stream capture.  Host threads may make their first
 * calls at the same time: the set-up is serialised by a lock inside the library.
 * All calls on a device share the one array.  A call overwrites every element
 * it later reads, so no clearing is needed and nothing leaks from the previous
 * call; but two calls that run on the GPU at the same time (different streams,
 * different threads) race on it and give wrong sums - order them. */
int ec_kmeans_partials_static(const float* points, const int32_t* labels, size_t N, int D, int K, int P,
                              float* partials, ec_stream_t stream);

/* ------------------------------------------------------------------------- *
 * Matrix factorisation whose item gradients go through the stale-synchronous
 * allreduce (the experiment of Sec. V; the paper names the model and the
 * collective, the update rule here is the textbook one).
 *
 * r_ui ~ <p_u, q_i>, k = 32 or 64 factors.  Rank r owns the users
 * [r*U/P, (r+1)*U/P) with all their ratings; user factors are updated locally,
 * item factors are shared.  The ratings are given twice: by user (CSR over all
 * users: user_ptr int64 [U+1], user_item int32 [nnz], user_val fp32 [nnz]) and,
 * inside every rank's share, by item (rank_item_ptr int64 [P][I+1] = offsets
 * into item_user int32 [nnz] / item_val fp32 [nnz]).  All six arrays are DEVICE
 * memory owned by the caller and must stay valid until destroy.
 *
 * One ec_mf_iterate at clock t (the clock starts at 0 and is raised first; all
 * errors e_ui = r_ui - <p_u, q_i> are taken at the factors the call starts from):
 *   1. the contribution G_r[i] = sum over rank r's ratings of e_ui * p_u of a
 *      (rank, item segment) pair is recomputed if its bit in refresh_mask is set
 *      (device uint64 [S][W], S = ceil(I / segment_rows); NULL = all), if it was
 *      never computed, or if its clock is below t - slack (Algorithm 1: a
 *      contribution that is too stale is waited for); its clock becomes t.
 *      Otherwise the rank's buffer keeps what it delivered before.
 *   2. R = ec_allreduce_ssp_apply over the P buffers (sum, rank order).
 *   3. p_u += lr * (sum_i e_ui * q_i - lambda * p_u) for every user.
 *   4. q_i += lr * (R_i - lambda * q_i) for every item.
 * Sums run in storage order with a fixed shape, so results repeat bit for bit.
 * ------------------------------------------------------------------------- */
typedef struct ec_mf ec_mf_t;

/* Bytes of device workspace (factors, P gradient buffers, clocks, the allreduce's
 * words).  0 on invalid arguments (k other than 32 or 64, P > n_users, ...). */
size_t ec_mf_workspace_bytes(int n_users, int n_items, int k, int P, size_t segment_rows);

/* user_factors fp32 [U][k] and item_factors fp32 [I][k] (device) are copied.
 * workspace as in ec_allreduce_init (NULL: the library allocates it).  Must not
 * be called during stream capture (it synchronises the legacy default stream). */
int ec_mf_init(ec_mf_t** mf, int n_users, int n_items, int k, int P, const int64_t* user_ptr, const int32_t* user_item,
               const float* user_val, const int64_t* rank_item_ptr, const int32_t* item_user, const float* item_val,
               const float* user_factors, const float* item_factors, float lr, float lambda, size_t segment_rows,
               void* workspace, size_t workspace_bytes);

/* One iteration as described above: five launches on `stream`, no allocation. */
int ec_mf_iterate(ec_mf_t* mf, const uint64_t* refresh_mask, uint32_t slack, ec_stream_t stream);

/* Replace the factors (device to device copies on `stream`); clocks and the
 * delivered gradients are kept. */
int ec_mf_set_factors(ec_mf_t* mf, const float* user_factors, const float* item_factors, ec_stream_t stream);

/* Copy out (device pointers, any may be NULL): the factors, sse = sum of e_ui^2
 * over all ratings at the start of the last iteration (one double), the clock of
 * each segment of the last reduction uint32 [S] (the minimum over the ranks,
 * Sec. III-A), the clocks of all contributions uint32 [S][P], and the number of
 * contributions the last reduction found too stale uint32 [S] (always 0 here,
 * since step 1 refreshes them). */
int ec_mf_get(ec_mf_t* mf, float* user_factors, float* item_factors, double* sse, uint32_t* seg_clock,
              uint32_t* notif_clock, uint32_t* wait_count, ec_stream_t stream);

int ec_mf_destroy(ec_mf_t* mf);

/* ------------------------------------------------------------------------- *
 * Threshold variants of Reduce / Broadcast (Sec. III-B) as notification words,
 * and the threshold test on the status output (Sec. III: "threshold" and
 * "status" parameters).  host_mask is HOST memory, uint64 [S][W], written.
 * ------------------------------------------------------------------------- */

/* Eventually consistent Broadcast (Sec. III-B): the root ships only the leading share of its
 * vector that the threshold `data_fraction` names, i.e. the first ceil(data_fraction * S) segments
 * (the rule of ec_mask_data_fraction), into the receive buffer of every rank; the rest of every
 * receive buffer is not touched.  On one device the binomial tree of the paper collapses into one
 * pass that reads each delivered byte once and writes it P times.
 *
 *   src            device, n elements of `dtype`: the root's data.
 *   dst_bufs       HOST array of P DEVICE pointers (n elements each).  NULL = that rank receives
 *                  nothing.  dst_bufs[root] may be NULL or equal to src (nothing is copied for it);
 *                  no other buffer may overlap src (EC_ERR_INVALID).
 *   notify         device uint64 [S][W], written in full, or NULL: bit r of segment s is 1 iff
 *                  s was delivered and (dst_bufs[r] != NULL or r == root) - ready to be used as
 *                  the arrival mask of a consumer.
 *
 * 16-byte aligned pointers take the 128-bit path, anything else a byte-wise one.  One launch, no
 * allocation, stateless. */
int ec_bcast(const void* src, void* const* dst_bufs, int P, int root, size_t n, ec_dtype_t dtype,
             size_t segment_size, double data_fraction, uint64_t* notify, ec_stream_t stream);

/* Strategy 1 of Sec. III-B, less data from everybody: the first ceil(fraction * S) segments of every rank count as
 * arrived, the others do not.  0 <= fraction <= 1. */
int ec_mask_data_fraction(int P, size_t S, double fraction, uint64_t* host_mask);

/* Strategy 2 of Sec. III-B, all the data of fewer processes: the binomial spanning tree works in stages
 * that double the number of involved processes (stage k brings in ranks 2^k .. 2^(k+1)-1); whole
 * stages are added until at least fraction * P processes take part.  Ranks 0 .. *ranks_included-1
 * count as arrived for every segment.  The last stage alone adds half of the processes, so
 * fractions 0.75 and 1.0 select the same set, as the paper observes.  ranks_included may be NULL. */
int ec_mask_process_threshold(int P, size_t S, double fraction, uint64_t* host_mask, int* ranks_included);

/* The threshold test: *ready_segments (device word, written) = number of segments whose
 * contrib_count (device uint32 [S], as written by an apply) is at least `need`; the collective has
 * reached a threshold theta when that equals S with need = ceil(theta * P).  One launch, one block. */
int ec_threshold_segments(const uint32_t* contrib_count, size_t S, uint32_t need, uint32_t* ready_segments,
                          ec_stream_t stream);

/* ------------------------------------------------------------------------- */
const char* ec_strerror(int code);
/* The cudaError_t of the last failed CUDA call on this thread (0 if none). */
int ec_last_cuda_error(void);
/* Library version, major * 1000 + minor. */
int ec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EC_H_ */
