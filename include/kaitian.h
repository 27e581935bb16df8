/*
 * kaitian.h -- C ABI of the B200 library for KAITIAN's hierarchical, load-weighted
 * gradient synchronisation (the data-parallel hot path of a heterogeneous training
 * step; paper Sections III-A and III-C).
 *
 * K simulated ranks, split into G vendor groups, keep their per-parameter gradient
 * tensors in one GPU's memory.  One synchronisation step is
 *
 *   kt_schedule      step times -> integer batch shares            (Section III-C)
 *   kt_groups_init   rank->group map + shares -> weights            (Sections III-A, III-C)
 *   kt_bucket_pack   describe the gradient tensors, build buckets   (DDP bucketing, Section III)
 *   kt_hier_reduce   INTRA: P_g = sum_{r in g} a_r x_r  (fp32 transport, one per group)
 *   kt_stage_to_host relay of the partials through pinned host RAM  (Section III-A, steps 1-3)
 *   kt_hier_reduce   INTER: S = sum_g W_g P_g
 *   kt_unpack_scale  per-parameter gradients = cast(scale * S)
 * or, when no host relay is needed (Section III-B, homogeneous dispatch),
 *   kt_sync_direct   all of the above arithmetic in one pass, no transport
 * With every rank a process on a device of its own, the same calls work on one member's share
 * of each bucket after kt_shard_bind (group mates' tensors through peer-mapped addresses).
 *
 * Conventions
 *  - Every pointer argument says "host" or "device".  "host array of device pointers"
 *    means the array itself is read on the host during the call and may be freed after
 *    it returns; the pointers in it address device memory owned by the caller.
 *  - The library owns only the kt_ctx and its small device tables (pointer tables, tensor
 *    table).  Gradient tensors, transport buffers, pinned buffers and streams belong to
 *    the caller.  `stream` arguments are cudaStream_t values passed as void* (NULL = the
 *    legacy default stream).
 *  - All functions return KT_OK (0) or a negative kt_status.  Arguments are validated on
 *    the host before anything is launched; nothing traps on the device and nothing
 *    throws across the boundary.  kt_last_error() returns a message for the last failing
 *    call made by the calling thread.
 *  - Kernel launches and copies are asynchronous with respect to the given stream.
 *    kt_scores, kt_schedule, kt_route, kt_adapt_*, kt_sampler_steps, kt_plan_buckets,
 *    kt_shard_ranges, kt_work_unit, kt_host_barrier, kt_set_shares, kt_set_coefficients,
 *    kt_plan_query and kt_shard_query are pure host functions; those before kt_set_shares
 *    need no CUDA device at all.  kt_shard_step and kt_shard_bcast block the calling thread
 *    until every rank has finished.
 *  - A context is bound to the CUDA device that was current in kt_groups_init.  Calls on it
 *    make that device current for their own duration and leave the calling thread's current
 *    device as they found it.
 *  - A kt_ctx (and a kt_adapt, a kt_graph) is not safe for concurrent use from several host
 *    threads; different objects may be used from different threads.  kt_last_error() is per
 *    thread.
 *  - Arithmetic is IEEE fp32 with a fixed order (ascending rank inside a group, ascending
 *    group): the first term of a sum is one rounded product, every later term one fused
 *    multiply-add.  bf16 gradients are widened exactly; bf16 outputs are rounded to
 *    nearest-even.
 */
#ifndef KAITIAN_H
#define KAITIAN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kt_ctx kt_ctx;
typedef struct kt_adapt kt_adapt;
typedef struct kt_graph kt_graph;

typedef enum { KT_F32 = 0, KT_BF16 = 1 } kt_dtype;

typedef enum {
    KT_OK = 0,
    KT_ERR_INVALID = -1, /* bad argument value (null pointer, range, non-finite time ...) */
    KT_ERR_SHAPE = -2,   /* sizes inconsistent with the plan (T, R, bucket index ...) */
    KT_ERR_ALIGN = -3,   /* a transport / flat / combined buffer is not 16-byte aligned */
    KT_ERR_CUDA = -4,    /* a CUDA runtime call or launch failed; message has the CUDA text */
    KT_ERR_TIMEOUT = -5, /* kt_stage_wait: the copy had not finished at the deadline */
    KT_ERR_STATE = -6,   /* call order: e.g. kt_hier_reduce before kt_bucket_pack */
    KT_ERR_NOMEM = -7    /* host or device allocation of a table failed */
} kt_status;

typedef enum { KT_INTRA = 1, KT_INTER = 2, KT_BOTH = 3 } kt_phase;
typedef enum { KT_ROUTE_DIRECT = 0, KT_ROUTE_RELAY = 1 } kt_route_kind;
typedef enum { KT_D2H = 0, KT_H2D = 1 } kt_stage_dir;

#define KT_MAX_RANKS 64
#define KT_MAX_GROUPS 16

/* Section III-C (initial benchmarking + dynamic data allocation).
 * step_times[K] (host): measured per-rank step times, each finite and > 0.
 * shares_out[K] (host): integer batch shares, sum == global_batch, each >= 1.
 * score_i = t_min / t_i; quota_i = score_i / sum(score) * global_batch; quotas are floored
 * and the missing units go to the largest fractional parts (tie: lower rank).  A zero
 * share is raised to one at the expense of the largest share (tie: the slowest of them,
 * then the higher rank).  Requires 1 <= K <= KT_MAX_RANKS and global_batch >= K.
 * Errors: KT_ERR_INVALID. */
int kt_schedule(const double *step_times, int K, int global_batch, int32_t *shares_out);

/* Section III-C, "Initial Benchmarking": the fastest device scores 1.0, every other device
 * score_i = time_fastest / time_i.  step_times[K] (host): finite and > 0; scores_out[K] (host).
 * This is the first half of kt_schedule, exposed for callers that share or log the scores
 * (the paper publishes them to all ranks before training).  Errors: KT_ERR_INVALID. */
int kt_scores(const double *step_times, int K, double *scores_out);

/* Online adaptation of the scores (Section III-C, "Online Adaptation": monitor computation
 * times per batch during training and adjust the scores; the paper leaves the rule open).
 * Rule used here: a rank's measured step time T_r was spent on its current share b_r, so
 * tau_r = T_r / b_r (time per sample) is what reflects its speed; tau_r is smoothed with an
 * exponential moving average of factor alpha (first observation initialises it); every
 * `period` observations kt_schedule is run on the smoothed tau; the result replaces the
 * shares in use only if the step time it predicts, max_r tau_r * b_r, is below
 * (1 - hysteresis) times the prediction for the shares in use.
 * kt_adapt_create: shares[K] (host) are the shares in use at the start, summing to
 *        global_batch; alpha in (0, 1]; period >= 1; hysteresis in [0, 1).
 * kt_adapt_observe: step_times[K] (host), finite and > 0, measured with the shares in use;
 *        shares_out[K] (host, may be NULL) receives the shares to use from now on, *changed
 *        (may be NULL) whether they differ from before.  Pure host arithmetic in double.
 * kt_adapt_state: read-back of the smoothed per-sample times, shares, observation count
 *        (each may be NULL).
 * Errors: KT_ERR_INVALID, KT_ERR_NOMEM. */
int kt_adapt_create(const int32_t *shares, int K, int global_batch, double alpha, int period,
                    double hysteresis, kt_adapt **out);
int kt_adapt_observe(kt_adapt *state, const double *step_times, int32_t *shares_out, int *changed);
int kt_adapt_state(const kt_adapt *state, double *per_sample_out, int32_t *shares_out,
                   int64_t *count_out);
void kt_adapt_destroy(kt_adapt *state);

/* Load-adaptive sampler (Section III-C "Dynamic Data Allocation"; Section IV-A: a sampler
 * that takes the per-device scores and distributes dataset indices accordingly).  With
 * B = sum of shares and c_r = shares[0] + ... + shares[r-1]: step s of an epoch consumes
 * positions [s*B, (s+1)*B) of the epoch's index list, rank r the shares[r] consecutive
 * positions from s*B + c_r on; rank r's epoch list is its slices of all steps in order,
 *   out[r][s*shares[r] + j] = list[(s*B + c_r + j) mod dataset_size].
 * kt_sampler_steps: steps per epoch: floor(D / B) with drop_last, else ceil(D / B) (the list
 *        is continued from its own start); negative kt_status on bad arguments.
 * kt_sampler_indices: list (device, int64[dataset_size], or NULL for the identity = no
 *        shuffling) is the epoch's permutation, drawn by the caller; shares[K] (host);
 *        out: host array of K device pointers, out[r] holding steps * shares[r] int64.
 *        One kernel on `stream`.  Errors: KT_ERR_INVALID, KT_ERR_SHAPE, KT_ERR_ALIGN, KT_ERR_CUDA. */
int64_t kt_sampler_steps(int64_t dataset_size, int64_t global_batch, int drop_last);
int kt_sampler_indices(const int64_t *list, int64_t dataset_size, const int32_t *shares, int K,
                       int drop_last, int64_t *const *out, void *stream);

/* Sections III-A (groups of homogeneous devices) and III-C (shares).
 * group_of[K] (host): group index of every rank, each in [0, G), no group empty.
 * shares[K] (host): batch shares, each >= 1.
 * Computes a_r = b_r / B_g and W_g = B_g / B (double quotient, rounded once to float).
 * *out receives a new context bound to the current CUDA device; free with kt_destroy.
 * Errors: KT_ERR_INVALID, KT_ERR_NOMEM, KT_ERR_CUDA. */
int kt_groups_init(const int32_t *group_of, const int32_t *shares, int K, int G, kt_ctx **out);

/* New shares for the same groups (e.g. after re-running kt_schedule); the bucket plan is
 * kept.  Takes effect for launches made after the call returns. */
int kt_set_shares(kt_ctx *ctx, const int32_t *shares);

/* Replace the weights directly: a[K], W[G] (host).  Lets a caller use plain sums across
 * the hierarchy (a_r = b_r, W_g = 1) with a final scale of 1/B in kt_unpack_scale. */
int kt_set_coefficients(kt_ctx *ctx, const float *a, const float *W);

/* Element type of the transport buffers: KT_F32 (the default, and what the method asks
 * for) or KT_BF16.  The bf16 transport is an extension of this library, not of the paper:
 * it halves the bytes that cross the host link, which is where Section III-A and Section V
 * locate the cost, at the price of one extra rounding of every group partial (at most
 * 2^-8 relative).  With KT_BF16 the fused reduce still accumulates in fp32 and rounds each P_g to
 * nearest-even when it stores it; the combine widens exactly.  Every `transport`,
 * `host_pinned`, `send`, `recv` and non-combined `src` argument of the calls below then
 * addresses bf16 buffers of transport_numel elements (pass them through the float* parameter
 * by a pointer cast); `combined` stays fp32.  kt_sync_direct keeps its partials in fp32
 * registers and is therefore bit-identical to the fp32-transport route only.
 * Takes effect for calls made after it returns.  Errors: KT_ERR_INVALID. */
int kt_set_transport_dtype(kt_ctx *ctx, int dtype);

/* Read back the weights in use: a_out[K], W_out[G] (host, either may be NULL). */
int kt_get_coefficients(const kt_ctx *ctx, float *a_out, float *W_out);

/* Gradient bucketing of the data-parallel reducer (Section III: gradients are
 * all-reduced bucket by bucket; the paper leaves order and size open).
 * grads: host array of K*T device pointers, rank-major (grads[r*T + t] = tensor t of
 *        rank r), element type in_dtype, numel[t] elements each (host array, >= 0).
 *        Pointers need only element alignment; 16-byte aligned tensors take the
 *        vectorised path.  The pointers are remembered: kt_hier_reduce(KT_INTRA) reads
 *        the tensors in place, so they must stay valid until re-registered.
 * Plan: tensors are laid into the fp32 transport in reverse list order; a bucket holds at
 *        most bucket_cap_bytes / 4 elements (a larger tensor gets a bucket of its own,
 *        tensors are never split); every tensor starts at a multiple of 8 elements, every
 *        bucket at a multiple of 64; the gaps are zero padding.
 * flat_out: NULL, or host array of K device pointers to buffers of transport_numel
 *        elements of in_dtype, 16-byte aligned: the standalone pack kernel then copies
 *        every rank's tensors into its flat buffer at the plan's offsets (bit copy,
 *        padding zero) on `stream`.
 * Calling it again replaces plan and pointers.  Allocates the device tables (the only
 * call besides kt_unpack_scale that may allocate).
 * Errors: KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_NOMEM, KT_ERR_CUDA. */
int kt_bucket_pack(kt_ctx *ctx, const void *const *grads, const int64_t *numel, int T,
                   int in_dtype, int64_t bucket_cap_bytes, void *const *flat_out, void *stream);

/* The bucket plan alone, as a pure host function (same rules as kt_bucket_pack; no context,
 * no device): lets a caller size transport buffers before any tensor exists.  Outputs as in
 * kt_plan_query.  Errors: KT_ERR_INVALID. */
int kt_plan_buckets(const int64_t *numel, int T, int64_t bucket_cap_bytes, int32_t *n_buckets,
                    int64_t *bucket_start, int64_t *bucket_numel, int64_t *tensor_offset,
                    int32_t *bucket_of, int64_t *transport_numel);

/* Plan read-back (all outputs host, each may be NULL).  bucket_start / bucket_numel need
 * room for n_buckets entries (at most T), tensor_offset for T; offsets and sizes are in
 * transport elements.  Errors: KT_ERR_STATE before kt_bucket_pack. */
int kt_plan_query(const kt_ctx *ctx, int32_t *n_buckets, int64_t *bucket_start,
                  int64_t *bucket_numel, int64_t *tensor_offset, int32_t *bucket_of,
                  int64_t *transport_numel);

/* One rank per device (Section III-A: the devices of a group run the group's collective among
 * themselves, device to device; Section III-B, steps 2-3).  The calls above and below treat
 * all K ranks' tensors as resident in one device's memory.  When every rank is a process with
 * a device of its own, each device does a share of every collective: the range of a call (one
 * bucket, or the whole transport with bucket == -1) is cut into work units of
 * kt_work_unit(in_dtype) transport elements that never cross a tensor (a tensor owns the
 * transport from its offset to the next tensor's offset, padding included, and holds
 * ceil(extent / unit) units); with U units in the range and M members in the group, member m
 * (ranks of the group in ascending order) owns units floor(m*U/M) ... floor((m+1)*U/M) - 1,
 * one contiguous element range.
 *
 * kt_work_unit:    elements per work unit for gradients of in_dtype (negative status if unknown).
 * kt_shard_ranges: the members' element ranges as a pure host function (no context, no
 *        device): numel, T, bucket_cap_bytes as in kt_plan_buckets; lo_out[n_members],
 *        n_out[n_members] (host) receive start and length of every member's range; a member
 *        without a unit gets length 0.  Errors: KT_ERR_INVALID, KT_ERR_SHAPE.
 * kt_shard_bind:   declares that the context belongs to rank `rank` of the map given to
 *        kt_groups_init.  Call it before kt_bucket_pack.  From then on
 *          - kt_bucket_pack takes the tensors of the M members of the rank's group only:
 *            grads[m*T + t], members in ascending rank order, the rank's own tensors by their
 *            ordinary addresses and its group mates' tensors by addresses under which this
 *            device can read them (peer-mapped: kt_ipc_open, or peer access inside one
 *            process).  They are read with ordinary loads.
 *          - kt_hier_reduce(KT_INTRA) forms the group partial over this member's share of
 *            the range, from all M members' tensors, into transport[own group] (the other
 *            entries of `transport` are not looked at);
 *          - kt_stage_to_host(KT_D2H) copies that share of transport[own group] down;
 *            kt_stage_to_host(KT_H2D) copies the same element range of every OTHER group's
 *            partial up (host_pinned is memory that all processes share; between the two
 *            the caller needs a barrier across processes, after its own copy down has
 *            finished, because other processes write what the way up reads);
 *          - kt_hier_reduce(KT_INTER), kt_unpack_scale and kt_sync_direct work on the share
 *            only; with R = M and out_grads[m*T + t] addressing member m's output tensors
 *            (peer-mapped again) every member receives this member's share of the result,
 *            so that after all members have run, and a barrier, every rank holds the whole
 *            reduced gradient.  kt_sync_direct needs G == 1 (it reads all ranks).
 *          - the broadcast calls take this rank's part in a broadcast (see kt_shard_bcast);
 *          - kt_relay_through_host, kt_allreduce across groups and the standalone pack return
 *            KT_ERR_STATE.
 *        Per element the arithmetic and its order are unchanged: results are bit-identical to
 *        the unsharded calls.  Ranks synchronise on the host (barriers); no kernel waits for
 *        another device.  Errors: KT_ERR_INVALID.
 * kt_shard_query:  the element range of `member` (-1: this context's own) for `bucket` under
 *        the registered plan, and the number of members (each output may be NULL).
 *        Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID. */
int kt_work_unit(int in_dtype);
int kt_shard_ranges(const int64_t *numel, int T, int64_t bucket_cap_bytes, int64_t unit, int bucket,
                    int n_members, int64_t *lo_out, int64_t *n_out);
int kt_shard_bind(kt_ctx *ctx, int rank);
int kt_shard_query(const kt_ctx *ctx, int bucket, int member, int *n_members, int64_t *lo, int64_t *n);

/* Memory shared between the processes of one node, for one rank per device.
 * kt_ipc_export: dev_ptr (device, anywhere inside an allocation made with cudaMalloc, e.g. by a
 *        framework's allocator) -> a handle of KT_IPC_HANDLE_BYTES bytes (host) naming the
 *        allocation, and the pointer's byte offset inside it.  Both are plain bytes that can be
 *        sent to another process of the node.
 * kt_ipc_open:   in another process, with the device current that shall read or write the
 *        memory: handle + offset -> *dev_ptr_out, an address valid in this process.  A handle is
 *        mapped once per process and device and counted; the exporting process must keep the
 *        allocation alive while it is open elsewhere.
 * kt_ipc_close:  gives one reference back; the last one unmaps.
 * kt_host_register / kt_host_unregister: page-locks `bytes` bytes of host memory at `host`
 *        (for instance a POSIX shared-memory segment mapped by every process) so that
 *        kt_stage_to_host can copy to and from it asynchronously.
 * Errors: KT_ERR_INVALID, KT_ERR_STATE, KT_ERR_CUDA. */
#define KT_IPC_HANDLE_BYTES 64
int kt_ipc_export(const void *dev_ptr, void *handle_out, int64_t *offset_out);
int kt_ipc_open(const void *handle, int64_t offset, void **dev_ptr_out);
int kt_ipc_close(const void *handle);
int kt_host_register(void *host, int64_t bytes);
int kt_host_unregister(void *host);

/* A barrier between the processes of one node (the ranks of Section III-A's one-server
 * deployment meet between the copy down and the copy up of the relay, and before and after a
 * collective).  `shared` (host): KT_HOST_BARRIER_BYTES bytes, 64-byte aligned, in memory that
 * every participating process maps, zeroed once before the first use.  Every one of the n_ranks
 * processes calls kt_host_barrier; the call returns KT_OK once all have arrived.  Reusable at
 * once.  The wait is on the host and bounded: with timeout_ms >= 0 a process that has waited that
 * long returns KT_ERR_TIMEOUT (a rank died, hung or never joined), the device is not involved
 * and stays usable; after a timeout the block is in an undefined state and must be zeroed
 * again, by agreement of the survivors, before it is reused.  timeout_ms < 0 waits without
 * limit.  Pure host function.  Errors: KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_TIMEOUT. */
#define KT_HOST_BARRIER_BYTES 128
int kt_host_barrier(void *shared, int n_ranks, int timeout_ms);

/* One synchronisation step of a rank-bound context (kt_shard_bind), start to finish, in the
 * order of Section III-A / III-B step 3: barrier (all ranks' gradients are complete; this rank's
 * device is synchronised first) -> fused reduce over this member's share of every range and,
 * behind each, the copy of the share into host memory all ranks map (down_stream) -> then range
 * by range: wait for the own copy, barrier (every rank's share of the range is down), copy of
 * the same element range of the other groups' partials up (up_stream, while later ranges are
 * still going down), combine + scale + cast + unpack of the share into the R = M output sets
 * (this rank's and, peer-mapped, its group mates') -> wait for the own stream, barrier.  With
 * one group the middle is kt_sync_direct: nothing is stored in a transport, so the transport's
 * element type (kt_set_transport_dtype) has no effect on the result.
 *   barrier_block (host): the kt_host_barrier block shared by all K ranks of kt_groups_init.
 *   partials: host array of G device pointers, this rank's rows of transport_numel elements
 *        (row of its own group: the share it reduces; other rows: what it receives).
 *   host_shared: host array of G pointers into page-locked host memory that all ranks map,
 *        the same layout in every process.  Both may be NULL with one group.
 *   out_grads, R, out_dtype, scale: as in kt_unpack_scale, R = number of group members.
 *   per_bucket != 0: the ranges are the buckets (2 + number of buckets barriers per step; both
 *        directions of the host link work at the same time); 0: one range, the whole transport.
 *   down_stream, up_stream: two different copy streams (ignored with one group).
 *   timeout_ms: limit of every barrier and of the wait for the own copies (< 0: none).
 * The call blocks the calling thread until the step is complete on every rank (it returns
 * after the last barrier).  On return the outputs of this rank hold the reduced gradients and no
 * rank reads this rank's gradients any more.  Errors: those of the parts; KT_ERR_TIMEOUT when a
 * rank did not arrive (nothing is left running on this rank's device that waits for it). */
int kt_shard_step(kt_ctx *ctx, void *barrier_block, float *const *partials, float *const *host_shared,
                  void *const *out_grads, int R, int out_dtype, float scale, int per_bucket,
                  void *main_stream, void *down_stream, void *up_stream, int timeout_ms);

/* Model synchronisation with one rank per device (the Broadcast of Section III routed through
 * the hierarchy of Section III-A): rank `root`'s registered tensors reach the registered tensors
 * of every other rank, bit for bit.  On a rank-bound context the three broadcast calls take the
 * part that this rank has in it and are no-ops otherwise:
 *   kt_bcast_send   the root alone: one pass over its tensors (the whole range, not a share)
 *                   into its flat send buffer and, by peer stores, into its group mates' tensors;
 *   kt_bcast_relay  the root: copies the range of `send` into `host_pinned` (memory all ranks
 *                   map); a rank of another group: copies ITS SHARE of `host_pinned` into
 *                   recv[own group]; between the two the caller needs a barrier across ranks;
 *                   completion is what kt_stage_wait(KT_D2H / KT_H2D, bucket) waits for;
 *   kt_bcast_recv   a rank of another group: unpacks its share of recv[own group] into the
 *                   tensors of every member of its group (peer stores), so that after all
 *                   members have run every tensor is complete.
 * kt_shard_bcast is the whole sequence in one blocking call, like kt_shard_step: barrier ->
 * root sends and copies down, waits -> barrier -> the other groups' ranks copy their shares up
 * and unpack -> wait for the own stream, barrier.
 *   send (device, root only), recv (device, ranks outside the root's group): flat buffers of
 *        transport_numel elements of the registered dtype, 16-byte aligned;
 *   host_shared (host): the same size, page-locked, mapped by all ranks (NULL with one group).
 * Errors: those of the parts. */
int kt_shard_bcast(kt_ctx *ctx, int root, void *barrier_block, void *send, void *host_shared, void *recv,
                   int per_bucket, void *main_stream, void *d2h_stream, void *h2d_stream, int timeout_ms);

/* The two reductions of Section III-A.
 * transport: host array of G device pointers, fp32, transport_numel elements each,
 *        16-byte aligned.
 * phase KT_INTRA: the fused pack + widen + weighted intra-group reduce.  Reads every
 *        registered gradient element once and writes P_g = sum_{r in g} a_r x_r at the
 *        plan's offsets of transport[g], zero in the padding.
 * phase KT_INTER: combined[i] = sum_g W_g transport[g][i] over the bucket's range
 *        (combined: device fp32, transport_numel elements, 16-byte aligned).
 * phase KT_BOTH: KT_INTRA then KT_INTER on the same stream.
 * bucket: -1 for all buckets, else one bucket index; only that bucket's range of the
 *        buffers is read or written.
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_CUDA. */
int kt_hier_reduce(kt_ctx *ctx, int phase, int bucket, float *const *transport, float *combined,
                   void *stream);

/* Host relay of Section III-A (device -> host RAM -> [exchange] -> device).
 * dir KT_D2H: side_stream waits for the work queued so far on main_stream, then copies the
 *        bucket's range of every transport[g] (device) to host_pinned[g] (host, pinned,
 *        same element offsets).
 * dir KT_H2D: side_stream waits for main_stream and for the last KT_D2H of every range that
 *        overlaps this one (the same bucket, the whole transport, and with bucket == -1 each
 *        single bucket, whichever stream those went down on), then copies host_pinned[g]
 *        back into transport[g] (typically a second, "receive" set of device buffers).
 * Both record a completion event that kt_stage_wait consumes.  transport / host_pinned:
 * host arrays of G pointers.  bucket as in kt_hier_reduce.
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_CUDA. */
int kt_stage_to_host(kt_ctx *ctx, int dir, int bucket, float *const *transport,
                     float *const *host_pinned, void *main_stream, void *side_stream);

/* The relay of Section III-A as one pipelined call (device -> host RAM -> device): the
 * bucket's range is cut into chunks of chunk_bytes (a few MiB works best; very small chunks
 * use the host link badly); chunk k of every send[g] is copied
 * to host_pinned[g] on d2h_stream and, as soon as that copy is done, from host_pinned[g] to
 * recv[g] on h2d_stream, so the two directions of the host link work at the same time.  Both
 * copy streams first wait for the work queued so far on main_stream.  Completion of the way
 * down / up is what kt_stage_wait(KT_D2H / KT_H2D, bucket) waits for.
 * send, host_pinned, recv: host arrays of G pointers (device fp32, pinned host, device fp32),
 * same element offsets in all three.  chunk_bytes >= 256; the two copy streams must differ.
 * With bucket == -1, if the G buffers of each list are rows of one allocation of
 * G * transport_numel elements (back to back in memory, and the driver confirms that each
 * list's range is a single allocation: buffers that merely happen to be neighbours do not
 * count), a chunk of all groups moves in one copy.
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_CUDA. */
int kt_relay_through_host(kt_ctx *ctx, int bucket, float *const *send, float *const *host_pinned,
                          float *const *recv, int64_t chunk_bytes, void *main_stream,
                          void *d2h_stream, void *h2d_stream);

/* Makes main_stream wait for the last kt_stage_to_host(dir, bucket).  timeout_ms < 0:
 * returns at once (stream-side wait only).  timeout_ms >= 0: additionally polls the
 * event on the host until it completes or the deadline passes (KT_ERR_TIMEOUT; the copy
 * itself is left running).  KT_ERR_STATE if no such copy was queued. */
int kt_stage_wait(kt_ctx *ctx, int dir, int bucket, void *main_stream, int timeout_ms);

/* Copy-out of the reducer: per-parameter gradients from the reduced bucket.
 * src: host array of device pointers; from_combined != 0: src[0] is a combined buffer
 *        (S); from_combined == 0: src[0..G-1] are the group partials and the inter-group
 *        combine S = sum_g W_g P_g is fused into this kernel (no combined buffer).
 * out_grads: host array of R*T device pointers (copy-major: out_grads[c*T + t]),
 *        R = 1, or up to K to hand every rank its own copy; element type out_dtype;
 *        numel as registered.  16-byte aligned tensors take the vectorised path.
 * out[t][j] = cast(scale * S[tensor_offset[t] + j]); one rounded multiply; padding ignored.
 * In place: the outputs may be the registered gradient tensors themselves (the reduce that
 *        read them is an earlier launch on the stream); they must not overlap `src`.
 * Destination tables: the R*T output pointers live in a small device table.  A context keeps
 *        up to 8 such tables, one per set of output tensors it has seen (least recently used
 *        replaced), so a caller that alternates between sets -- double-buffered gradients --
 *        pays for each upload once.  A set seen for the first time allocates its table (device
 *        and pinned host memory, once) and uploads it with an asynchronous copy on `stream`;
 *        the host does not wait for the device.  A table that a recorded step uses is never
 *        replaced (until kt_bucket_pack re-plans).
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_NOMEM, KT_ERR_CUDA. */
int kt_unpack_scale(kt_ctx *ctx, const float *const *src, int from_combined,
                    void *const *out_grads, int R, int out_dtype, float scale, int bucket,
                    void *stream);

/* Section III-B, step 1: before a collective runs, look at the participating ranks and
 * decide whether it stays inside one group of like accelerators or spans several.
 * group_of[K] (host): group index of every rank, each in [0, G), as in kt_groups_init.
 * participants[n] (host): distinct rank indices in [0, K), n >= 1.
 * *route receives KT_ROUTE_DIRECT when all participants belong to one group (step 2: the
 * collective goes straight to the device-side reduction, kt_sync_direct) and KT_ROUTE_RELAY
 * when they span groups (step 3: kt_hier_reduce, the relay through host memory,
 * kt_unpack_scale).  groups_out (host, may be NULL, room for G entries) receives the
 * ascending list of groups that take part, *n_groups_out (may be NULL) their number.
 * Pure host function, no context and no device needed.
 * Errors: KT_ERR_INVALID (NULL, n < 1, rank or group out of range, rank repeated). */
int kt_route(const int32_t *group_of, int K, int G, const int32_t *participants, int n,
             int *route, int32_t *groups_out, int *n_groups_out);

/* The direct path: the whole synchronisation in one pass, without transport buffers.
 * Section III-B: a collective whose participants need no host relay (one vendor group, or
 * groups that share a device) is dispatched straight to the device-side reduction; only
 * collectives that span accelerator types take the staged route above.
 * Reads every registered gradient element once and writes
 *   out[t][j] = cast(scale * sum_g W_g * (sum_{r in g} a_r * f32(x_r^(t)[j])))
 * with the operation order of kt_hier_reduce(KT_INTRA) followed by kt_unpack_scale (group
 * partials are formed first, in fp32, then combined): results are bit-identical to that
 * route.  out_grads, R, out_dtype, scale, bucket as in kt_unpack_scale; the gradients are
 * the ones registered by kt_bucket_pack.  May allocate the destination table like
 * kt_unpack_scale.
 * In place: an output tensor may be one of the registered gradient tensors of the same index t
 * and the same element type (out_grads[c*T + t] == grads[r*T + t] for any c, r: the usual
 * all-reduce in place); the call detects exact pointer equality and reads the gradients
 * with ordinary loads then.  Outputs that overlap registered gradients in any other way
 * (shifted, another index, another type) are not allowed and not detected.
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_NOMEM, KT_ERR_CUDA. */
int kt_sync_direct(kt_ctx *ctx, void *const *out_grads, int R, int out_dtype, float scale,
                   int bucket, void *stream);

/* One AllReduce of the registered gradients in one call: Section III-B, steps 1-3, as the
 * meta process group performs them for every collective.  With one group the call is
 * kt_sync_direct.  With several groups it queues, on main_stream and the two copy streams,
 * kt_hier_reduce(KT_INTRA) over all buckets, kt_relay_through_host of the whole transport,
 * the wait for the way up, and kt_unpack_scale from the receive buffers.
 * transport, host_pinned, recv: as in kt_relay_through_host (ignored, may be NULL, with one
 * group); out_grads, R, out_dtype, scale: as in kt_unpack_scale; chunk_bytes >= 256.
 * Asynchronous like its parts; results are bit-identical to calling the parts.
 * Errors: those of the parts. */
int kt_allreduce(kt_ctx *ctx, float *const *transport, float *const *host_pinned, float *const *recv,
                 void *const *out_grads, int R, int out_dtype, float scale, int64_t chunk_bytes,
                 void *main_stream, void *d2h_stream, void *h2d_stream);

/* Hierarchical Broadcast (model synchronisation).  The paper routes Broadcast through the
 * same hierarchy as AllReduce (Section III, "broadcast for model synchronization"; Section
 * III-A: inside a group directly, between groups through host RAM in the three copy steps).
 * The tensors are the ones registered with kt_bucket_pack (here: parameters rather than
 * gradients; the same context type, usually a second context).  The root rank's tensors are
 * read, every other rank's registered tensors are WRITTEN; all copies are bit copies in the
 * registered dtype, laid out in the flat buffers at the plan's offsets (zero padding).
 *
 * kt_bcast_send: one pass over the root's tensors; writes the flat send buffer of the root's
 *        group (`send`: device, transport_numel elements of the registered dtype, 16-byte
 *        aligned) and the tensors of the root's group mates.
 * kt_bcast_relay: the bucket's range of `send` (device) goes to `host_pinned` (host, pinned,
 *        same layout) and from there into recv[g] (device) of every group g other than the
 *        root's, chunk by chunk on the two copy streams as in kt_relay_through_host;
 *        completion is what kt_stage_wait(KT_D2H / KT_H2D, bucket) waits for.
 *        recv: host array of G device pointers; the root group's entry is ignored.
 * kt_bcast_recv: one pass over the receive buffers; every group other than the root's reads
 *        recv[g] once and writes the tensors of all its members.  Passing the send buffer as
 *        recv[g] skips the relay (groups that can reach each other directly).
 * root: rank index in [0, K).  bucket as in kt_hier_reduce.
 * Errors: KT_ERR_STATE, KT_ERR_SHAPE, KT_ERR_INVALID, KT_ERR_ALIGN, KT_ERR_CUDA. */
int kt_bcast_send(kt_ctx *ctx, int root, int bucket, void *send, void *stream);
int kt_bcast_relay(kt_ctx *ctx, int root, int bucket, const void *send, void *host_pinned,
                   void *const *recv, int64_t chunk_bytes, void *main_stream, void *d2h_stream,
                   void *h2d_stream);
int kt_bcast_recv(kt_ctx *ctx, int root, int bucket, void *const *recv, void *stream);

/* Standalone cast kernel: n elements from `in` (device, in_dtype) to `out` (device,
 * out_dtype); bf16 -> fp32 exact, fp32 -> bf16 round-to-nearest-even, same type = copy.
 * Errors: KT_ERR_INVALID, KT_ERR_CUDA. */
int kt_cast(const void *in, int in_dtype, void *out, int out_dtype, int64_t n, void *stream);

/* Host <-> device movement of a tensor list (the accelerator <-> host RAM copies of
 * Section III-A applied to per-parameter tensors): n asynchronous copies dst[i] <- src[i] of
 * bytes[i] bytes on `stream`, one copy per tensor.
 * dst, src, bytes: host arrays.  dir KT_H2D: src host (pinned for true asynchrony), dst
 * device; KT_D2H: the reverse.  Errors: KT_ERR_INVALID, KT_ERR_CUDA. */
int kt_copy_tensors(void *const *dst, const void *const *src, const int64_t *bytes, int n, int dir,
                    void *stream);

/* The whole flat path in one call that allocates nothing.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * Who needs it: callers that are not allowed to allocate device memory at the point where
 * gradients must be synchronised -- code running inside a framework's no-allocation region,
 * plugins that must stay out of the host application's memory pool, processes whose device
 * memory is fully planned up front.  Every other entry point either allocates small device
 * tables itself (kt_bucket_pack, kt_unpack_scale) or needs caller-allocated transport
 * buffers; this one keeps its tables and the fp32 group partials in a fixed array that is
 * part of the library image.
 *
 * Computes, for one flat gradient buffer per rank,
 *   out[i] = cast(scale * sum_g W_g * sum_{r in g} a_r * f32(grads[r][i])),  i < n,
 * with the weights and the operation order of kt_groups_init / kt_hier_reduce /
 * kt_unpack_scale (results are bit-identical to that route).
 *   group_of[K], shares[K] (host): as in kt_groups_init.
 *   grads (host array of K device pointers): n elements of in_dtype each, element aligned.
 *   out (device): n elements of out_dtype.
 * Limit: G * round_up(n, 64) <= KT_STATIC_MAX_ELEMS fp32 elements of scratch (4 MiB, held
 * by every GPU that loads the library until the process exits); larger problems are
 * rejected with KT_ERR_SHAPE and a message naming the sizes.
 * Set-up: the first call on each device looks up the device address of the scratch array
 * (with that device current).  Make that first call outside any stream capture.
 * Sharing: all calls on a device use the same array, which keeps whatever the last call
 * left in it.  Nothing in it has to start at zero -- each call rewrites the tables and every
 * partial element it later reads -- but two calls that overlap on the GPU (different
 * streams, or different host threads without ordering) race on it: keep calls on one
 * stream, or order them with events.
 * Calls no cudaMalloc / cudaFree and no allocating library routine; host state is on the
 * stack, and nothing queued on the stream refers to it after the call returns (the tables
 * reach the scratch as the parameters of a small kernel, not through a copy from host memory).
 * Three kernels on `stream`.  Errors: KT_ERR_INVALID, KT_ERR_SHAPE, KT_ERR_ALIGN, KT_ERR_CUDA. */
#define KT_STATIC_MAX_ELEMS (1 << 20)
int kt_sync_flat_static(const int32_t *group_of, const int32_t *shares, int K, int G,
                        const void *const *grads, int in_dtype, int64_t n, void *out, int out_dtype,
                        float scale, void *stream);

/* One submission per step.  A synchronisation step is a fixed sequence of launches, copies
 * and event waits (the paper's step is one AllReduce call per bucket, Section III); between
 * kt_graph_begin and kt_graph_end every call of this library made by the calling thread on
 * `stream` (and on copy streams it pulls in: kt_stage_to_host, kt_relay_through_host) is
 * recorded instead of executed; kt_graph_launch then replays the whole sequence with one
 * submission, which removes the per-call host cost that dominates small tensor lists.
 * Rules while recording: the context must have run the same sequence once before (so that
 * its device tables are uploaded and its events exist; a call that would have to upload a
 * destination table returns KT_ERR_STATE and kt_graph_end then drops the recording with
 * KT_ERR_STATE); every copy stream must be waited
 * for with kt_stage_wait(..., timeout_ms < 0) before kt_graph_end; pointers, sizes, shares
 * and scale are frozen into the recording (record again after kt_set_shares; a recording is
 * void once kt_bucket_pack has re-planned the context and must not be launched again).
 * kt_graph_nodes: number of recorded operations.  The graph owns no buffers.
 * Errors: KT_ERR_STATE, KT_ERR_INVALID, KT_ERR_NOMEM, KT_ERR_CUDA. */
int kt_graph_begin(kt_ctx *ctx, void *stream);
int kt_graph_end(kt_ctx *ctx, void *stream, kt_graph **out);
int kt_graph_launch(kt_graph *graph, void *stream);
int64_t kt_graph_nodes(const kt_graph *graph);
void kt_graph_destroy(kt_graph *graph);

/* Number of kernels this context has launched so far (for launch accounting). */
int64_t kt_launch_count(const kt_ctx *ctx);

/* Message of the last failing call of this thread ("" if none).  ctx may be NULL. */
const char *kt_last_error(const kt_ctx *ctx);

/* Frees the context, its device tables and events.  NULL is allowed. */
void kt_destroy(kt_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* KAITIAN_H */
