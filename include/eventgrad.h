/*
 * eventgrad.h — C ABI of the B200 (sm_100a) library for EventGraD's per-iteration
 * event-triggered communication step.
 *
 * One context simulates a ring of P data-parallel replicas ("PEs" in the paper) that all
 * live in one GPU's memory.  One eg_step is one pass of the inner part of Algorithm B of
 * "EventGraD: Event-Triggered Communication in Parallel Machine Learning":
 *   for every replica i and every layer tensor I ("parameter" in the paper):
 *     d = || x - x_hat ||_2                         (trigger condition, Section 4)
 *     event  <=>  d >= delta  (or k == 0, forced)   (Section 4; Fig. 1 discussion)
 *     on an event: delta = horizon * mean of the last H slopes d / (k - k_hat)
 *                                                    (Eq. (thres); history: Section 7)
 *                  x_hat <- x   (dense message, the one-sided put into the neighbours'
 *                  windows of Section 6) or, with Top-K, the K_t entries of largest
 *                  |x - x_hat| packed as (index, value) and scattered into x_hat on
 *                  receipt (Top-K paragraph of Section 7)
 *   then  x_i <- w * (x_i + sum over ring neighbours j of x_hat_j) - lr * g_i,
 *         w = 1/(N_i + 1) = 1/3 on a ring            (Eq. (dist_sgd_event), Section 3)
 *
 * Conventions
 *  - All pointers named params / grads / *_dev are DEVICE pointers owned by the caller.
 *    Pointers named *_host (and all out-parameters of eg_stats, eg_layout,
 *    eg_last_decisions, eg_last_outbox, eg_export_state) are HOST pointers owned by the
 *    caller.  The context owns everything else and frees it in eg_destroy.
 *  - Parameter layout: fp32, [P][replica_stride]; tensor t of replica i starts at element
 *    i*replica_stride + tensor_offset[t].  The library chooses the offsets (each tensor
 *    starts on a 128-byte boundary; read them with eg_layout).  Padding elements between
 *    tensors are never written and their content is ignored.
 *  - params and grads must be 16-byte aligned device allocations of at least
 *    P*replica_stride floats.
 *  - eg_step only enqueues work on `stream` (a cudaStream_t passed as void*; NULL is the
 *    legacy default stream).  It never synchronises and never copies to the host.  The
 *    calls that read results back (eg_stats, eg_last_*, eg_export_state, eg_step_host)
 *    synchronise that stream.
 *  - One context belongs to one device (the one current at eg_create) and is used from one
 *    stream at a time: eg_step on another stream than the previous step's, while that stream
 *    still has unfinished work, returns EG_ERR_STATE (synchronise it first, or order the two
 *    streams and wait).  Ordering against the caller's other work on the stream is the
 *    caller's job.
 *  - Every function returns an eg_status; nothing throws, aborts or traps.  A device-side
 *    problem (an index outside its table, a bounded wait that ran out) sets an error word that
 *    the next synchronising call returns as EG_ERR_INTERNAL or EG_ERR_TIMEOUT.
 *  - Counters: an event of tensor t at replica i adds deg(i) to messages_sent (deg = number
 *    of distinct ring neighbours: min(2*hops, P-1), i.e. 2 on the paper's ring) and deg(i)*payload to
 *    bytes_sent; payload = 4*n_t for a dense message, 8*K_t for a Top-K message
 *    ("2K percent", Section 7).  The paper's "percentage of messages" (Table 1) is
 *    messages_sent / (P * T * 2 * steps).
 */
#ifndef EVENTGRAD_H
#define EVENTGRAD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eg_ctx eg_ctx; /* opaque */

typedef enum {
    EG_OK = 0,
    EG_ERR_INVALID = 1,  /* bad argument */
    EG_ERR_OOM = 2,      /* host or device allocation failed */
    EG_ERR_CUDA = 3,     /* a CUDA runtime call failed; see eg_last_cuda_error */
    EG_ERR_STATE = 4,    /* call not allowed in the context's current state */
    EG_ERR_TIMEOUT = 5,  /* a bounded device-side wait gave up (see eg_selftest_wait_timeout) */
    EG_ERR_INTERNAL = 6  /* device-side consistency check failed */
} eg_status;

enum { EG_TOPO_RING = 0 }; /* the topology the paper fixes (Section 3): nearest neighbours */
/* Ring in which every replica averages with the m nearest replicas on each side, 1 <= m <= 8
 * (Section 7: more neighbours per PE let information flow sooner); W_ij = 1/(N_i + 1) over the
 * distinct neighbours.  EG_TOPO_RING_HOPS(1) == EG_TOPO_RING. */
#define EG_TOPO_RING_HOPS(m) ((m) - 1)
enum { EG_THRESH_ADAPTIVE = 0, /* Eq. (thres) with a history of H slopes */
       EG_THRESH_FIXED = 1 };  /* one static threshold for all tensors (Section 4 calls it
                                  the simplest option); 0 gives regular D-PSGD, +inf none */

typedef struct {
    int mode;              /* EG_THRESH_ADAPTIVE or EG_THRESH_FIXED */
    double horizon;        /* h of Eq. (thres); the paper's experiments use 1 */
    int history_len;       /* H >= 1 slopes averaged; 1 is Eq. (thres) literally */
    double delta_init;     /* threshold in force until the second event of a tensor */
    double delta_fixed;    /* the threshold of EG_THRESH_FIXED */
    int force_first_event; /* 1: every tensor communicates at k = 0 (Section 4) */
} eg_threshold_params;

typedef struct {
    int enabled;           /* 0: dense messages */
    uint32_t k_num, k_den; /* K_t = max(1, ceil(n_t * k_num / k_den)) entries per message;
                              the first message of every tensor is dense */
} eg_topk_params;

/* Creates a context on the current device for P replicas of T tensors with layer_numel[t]
 * elements each (host array).  topk may be NULL (dense).  Allocates the mailboxes x_hat
 * (zero: X_0 = 0 of Assumption 2), the per-(replica, tensor) trigger state, scratch for the
 * norm partial sums, the Top-K outboxes and the counters.  *out is NULL on failure. */
eg_status eg_create(eg_ctx** out, int topology, int P, const int64_t* layer_numel, int T,
                    const eg_threshold_params* thr, const eg_topk_params* topk);

/* Layout chosen by the library for the parameters of one replica (the N parameters every PE
 * holds, Section 3): tensor_offset_host[T] (elements, within one replica) and
 * *replica_stride_host (elements).  Either pointer may be NULL. */
eg_status eg_layout(const eg_ctx* ctx, int64_t* tensor_offset_host, int64_t* replica_stride_host);

/* One iteration of Algorithm B (see the top of this file) on `stream`.  params (device,
 * [P][replica_stride] fp32) is updated in place; grads has the same layout and is only read.
 * Errors: EG_ERR_INVALID for NULL or misaligned pointers, EG_ERR_CUDA if a launch fails. */
eg_status eg_step(eg_ctx* ctx, float* params, const float* grads, float lr, void* stream);

/* Same iteration for callers whose data lives in HOST memory: copies params_host and
 * grads_host ([P][replica_stride] fp32, ideally pinned) to device staging buffers owned by
 * the context (allocated on first use), runs eg_step, copies the updated parameters back
 * and synchronises.  Tensors do not interact within an iteration, so for dense contexts on the
 * nearest-neighbour ring the work is pipelined in groups of tensors: while one group is being
 * computed the next is being copied in and the previous one copied out (pinned host buffers
 * are needed for the copies to overlap).  The result is the same as that of eg_step. */
eg_status eg_step_host(eg_ctx* ctx, float* params_host, const float* grads_host, float lr);

/* Carried-norm mode (off by default).  When on, the fused average/update kernel of step k
 * also accumulates || x_{k+1} - x_hat ||^2 of every tensor, so step k+1 skips its separate
 * norm pass (16 instead of 24 bytes of memory traffic per element).  Only valid while the
 * caller leaves params untouched between consecutive eg_step calls on the same buffer;
 * turning it on, eg_reset and eg_import_state make the next step recompute the norms. */
eg_status eg_set_carry_norm(eg_ctx* ctx, int enabled);

/* Two readings of the paper's text that differ from the defaults (both are what the text,
 * rather than the displayed formulas or the defaults' rationale, literally says):
 *  own_term       EG_OWN_CURRENT (default): a replica averages its CURRENT parameters with
 *                 the neighbours' last received ones.  EG_OWN_LAST_SENT: its own term is
 *                 x_hat_i as well, i.e. X_{k+1} = X_hat_k W - gamma G of Eq. (dist_sgd_event)
 *                 taken literally.
 *  trigger_metric EG_TRIGGER_NORM_OF_CHANGE (default): d = || x - x_hat || (the displayed
 *                 trigger condition).  EG_TRIGGER_CHANGE_OF_NORM: d = | ||x|| - ||x at the
 *                 last event|| | (the change-of-norm reading of the prose of Section 4); the
 *                 norm pass then reads x only.
 * Allowed before the first step of a context or right after eg_reset (EG_ERR_STATE later). */
enum { EG_OWN_CURRENT = 0, EG_OWN_LAST_SENT = 1 };
enum { EG_TRIGGER_NORM_OF_CHANGE = 0, EG_TRIGGER_CHANGE_OF_NORM = 1 };
eg_status eg_set_variant(eg_ctx* ctx, int own_term, int trigger_metric);

/* Intermittent delivery.  Section 7 remarks that the one-sided puts of the paper's
 * implementation arrive at unpredictable times; this models it with links that are up or down
 * per iteration.  After eg_enable_delivery_masks the context keeps two copies per replica: what
 * it has SENT (x_hat, the reference of its trigger test) and what its neighbours have RECEIVED
 * (the mailbox they average with).  eg_step_masked is eg_step with a device array
 * deliver_dev[P*T] (uint8): a non-zero entry [i*T + t] lets everything replica i has sent of
 * tensor t and that has not arrived yet -- this iteration's message included -- arrive now,
 * before the neighbours average; zero keeps it in flight (a later message replaces an earlier
 * one in flight, as a later put into the same window does).  deliver_dev == NULL (and plain
 * eg_step) delivers everything outstanding.  eg_enable_delivery_masks allocates the second
 * copy (P*replica_stride floats) and synchronises; everything sent until then counts as
 * arrived.  Not available together with EG_OWN_LAST_SENT (that reading has no received copy to
 * average with).  The carried norm, momentum, more neighbours and Top-K all work with it; the
 * carried norms are taken against what a replica has SENT.
 * eg_read_received copies the received copies to the host ([P][replica_stride] fp32; equal to
 * eg_read_mailboxes under synchronous delivery); eg_delivery_status returns the per-(replica,
 * tensor) "in flight" flags (host, P*T bytes) and the number of arrivals so far. */
eg_status eg_enable_delivery_masks(eg_ctx* ctx);
eg_status eg_step_masked(eg_ctx* ctx, float* params, const float* grads, float lr,
                         const uint8_t* deliver_dev, void* stream);
eg_status eg_read_received(eg_ctx* ctx, float* received_host);
eg_status eg_delivery_status(eg_ctx* ctx, uint8_t* pending_host, uint64_t* arrivals_host);

/* Bound on the thresholds (Assumption 1 of Section 5, with the geometric sequence
 * g(k) = alpha * beta^k of Corollary 2): the threshold a tensor is tested against in iteration
 * k becomes min(delta, sqrt(g(k))); the adaptive delta itself is left as computed.
 * alpha <= 0 removes the bound (default).  g lives on the device and is carried as the geometric
 * sequence it is -- g(0) = alpha, g(k+1) = beta * g(k), one fp64 multiplication per iteration,
 * made by the kernels of the step -- so a step recorded into a CUDA graph keeps the right bound
 * on every replay.  The call synchronises the context's stream and starts the sequence at the
 * term of the iteration the context has reached; eg_reset restarts it at alpha. */
eg_status eg_set_threshold_cap(eg_ctx* ctx, double alpha, double beta);

/* Heavy-ball momentum.  The Introduction says that event-triggered communication extends to
 * other training algorithms and gives none; this is the plain momentum method with a velocity
 * per replica that is never communicated:
 *     v_i <- mu * v_i + g_i,     x_i <- w * (x_i + sum of the neighbours' x_hat_j) - lr * v_i,
 * i.e. Eq. (dist_sgd_event) with the gradient replaced by the velocity.  v is fp32, laid out
 * like params, owned by the context (allocated and zeroed by the first enabling call, zeroed
 * again by eg_reset); mu * v + g is one fp64 fused multiply-add rounded to fp32, and the update
 * uses that rounded value.  mu = 0 reproduces the plain update bit for bit.  0 <= mu < 1
 * (EG_ERR_INVALID otherwise).  Works with every other option (readings, more neighbours,
 * intermittent delivery, Top-K, either kernel choice); the default readings on the
 * nearest-neighbour ring have the fastest kernel.  enabled = 0 returns to the plain update and
 * keeps the buffer.  The velocities are part of eg_export_state once the
 * buffer exists; eg_read_velocity / eg_write_velocity copy them to / from a host buffer of
 * P*replica_stride floats (both synchronise; EG_ERR_STATE before the first enabling call). */
eg_status eg_set_momentum(eg_ctx* ctx, int enabled, double mu);

/* Quantised messages: a second compression on top of the events.  Section 7 says that
 * quantization can be applied on top of event-triggered communication and gives no scheme; the
 * one built here quantises the CHANGE since the last message.  On an event of a tensor that has
 * been sent before, with d[e] = x[e] - x_hat[e] (one fp32 subtraction) and L = 2^(bits-1) - 1:
 *   scale    2^E, E the smallest integer with L * 2^E >= max_e |d[e]|   (E = 0 if all d are 0)
 *   codes    q[e] = d[e] / 2^E rounded to the nearest integer, ties to even (so |q[e]| <= L)
 *   message  E and the n codes: 4 + ceil(n * bits / 8) bytes per neighbour
 *   receipt  x_hat[e] <- fp32( fp64(x_hat[e]) + q[e] * 2^E ), at the sender too, so that x_hat
 *            stays what the receivers hold.
 * What was not sent, x - x_hat, remains part of the difference: it enters the next trigger test
 * and the next message (nothing is dropped for good).  The first message of a tensor is sent in
 * full precision (x_hat <- x, 4 n bytes), as with Top-K messages; so is a message whose change
 * holds an infinity or a NaN.  bits: 2..16; 0 or 32 switches quantisation off.  Only before the
 * first step or after eg_reset (EG_ERR_STATE otherwise).  Works with every other option: the
 * messages are delivered into x_hat by kernels of their own before the averaging kernel runs,
 * the way Top-K messages are.
 * In a context with Top-K messages both compressions apply ("quantization and sparsification on
 * top of event-triggered communication", Section 7): the K_t entries are selected as without
 * quantisation, E comes from the largest change of the tensor (which is among them), the message
 * holds E, the K_t indices and the K_t codes (4 + 4 K_t + ceil(K_t * bits / 8) bytes), and x_hat is
 * updated at the selected entries only; eg_last_outbox then returns, as values, what the
 * receivers hold at those entries after the message.
 * eg_last_quantised copies, for the last step, which (replica, tensor) pairs sent a quantised
 * message (1; 2: the change was not finite and the message went out in full; 0: none) and the
 * exponents E of those messages to host arrays of P*T entries; EG_ERR_STATE when quantisation
 * was never switched on.  Synchronises. */
eg_status eg_set_quantisation(eg_ctx* ctx, int bits);
eg_status eg_last_quantised(eg_ctx* ctx, uint8_t* quantised_host, int32_t* exponents_host);
eg_status eg_read_velocity(eg_ctx* ctx, float* velocity_host);
eg_status eg_write_velocity(eg_ctx* ctx, const float* velocity_host);

/* Which implementation of the fused snapshot / average / SGD kernel eg_step launches.  All
 * compute bit-identical parameters, mailboxes, flags and counters.
 *  EG_FUSED_AUTO (default)  for small problems (dense messages on the nearest-neighbour ring,
 *                      default readings, P <= 16, few enough tiles of 1024 elements for all
 *                      their thread blocks to be resident at once) the whole iteration -- decisions, snapshot, average, update,
 *                      next norms -- runs as ONE kernel launch, because such an iteration is
 *                      bound by launch latency; everything else takes EG_FUSED_PIPELINED.
 *  EG_FUSED_PIPELINED  streams the operands through shared memory with bulk asynchronous
 *                      copies (a decision kernel runs before it).
 *  EG_FUSED_REGISTER   keeps the ring walk in registers with plain vector loads. */
enum { EG_FUSED_PIPELINED = 0, EG_FUSED_REGISTER = 1, EG_FUSED_AUTO = 2 };
eg_status eg_set_fused_kernel(eg_ctx* ctx, int kind);

/* Per-kernel timing for measurements (off by default).  When on, eg_step brackets each
 * kernel group with a pair of CUDA events recorded on the step's own stream (and launches the
 * kernels one strictly after the other, so that every duration is the kernel's own: a step is
 * then a few percent slower than without timing); eg_kernel_times
 * synchronises, adds up the elapsed milliseconds per group since the last call into
 * ms_host[EG_KERNEL_GROUPS], the number of timed sections into
 * sections_host[EG_KERNEL_GROUPS], and forgets them.  At most 32768 sections are kept
 * between two reads; further ones are not timed. */
enum { EG_KERNEL_NORM = 0, EG_KERNEL_DECIDE = 1, EG_KERNEL_TOPK = 2, EG_KERNEL_FUSED = 3,
       EG_KERNEL_GROUPS = 4 };
eg_status eg_set_timing(eg_ctx* ctx, int enabled);
eg_status eg_kernel_times(eg_ctx* ctx, double* ms_host, uint64_t* sections_host);

/* Totals since creation / eg_reset (Table 1 and Table 2 report ratios of these).
 * Synchronises.  Pointers may be NULL. */
eg_status eg_stats(eg_ctx* ctx, uint64_t* messages_sent_host, uint64_t* bytes_sent_host);
eg_status eg_event_count(eg_ctx* ctx, uint64_t* events_host);

/* Decisions of the most recent step (trigger condition of Section 4), host arrays of P*T
 * entries indexed [i*T + t]: flags (1 = event), norms (d), thresholds (the delta that d was
 * compared with).
 * Any pointer may be NULL.  Synchronises. */
eg_status eg_last_decisions(eg_ctx* ctx, uint8_t* flags_host, double* norms_host,
                            double* thresholds_host);

/* Threshold in force after the most recent step and number of events so far, per
 * (replica, tensor); host arrays of P*T entries.  Synchronises. */
eg_status eg_thresholds(eg_ctx* ctx, double* delta_host, uint64_t* events_host);

/* The Top-K message replica i sent for tensor t in the most recent step: *count_host entries
 * (0 if it sent none or sent a dense message), ascending indices in idx_host and the
 * parameter values in val_host (capacity: eg_topk_count(t) entries each). */
eg_status eg_last_outbox(eg_ctx* ctx, int i, int t, int32_t* idx_host, float* val_host,
                         int32_t* count_host);
eg_status eg_topk_count(const eg_ctx* ctx, int t, int64_t* k_t_host);

/* How the Top-K entries are found (Top-K paragraph of Section 7; the result is always the exact
 * K_t largest |x - x_hat|, ties to the lower index).  For a large tensor the library first
 * guesses, from a sample of the tensor, a magnitude bin at or below that of the K_t-th largest
 * entry, collects everything at or above it in one pass and finishes the selection exactly on
 * what it collected; when the guess turns out wrong (too few collected, or far too many) that
 * tensor is selected again without guessing, at the cost of two more passes over it.
 * eg_topk_repeat_count returns how many sparse messages took that second route since the
 * context was created or reset (synchronises).  EG_TOPK_GUESS_MARGIN in the environment at
 * eg_create sets the safety margin of the guess in standard deviations of the sampled count
 * (default 5; a negative value makes every guess fail, which exercises the second route). */
eg_status eg_topk_repeat_count(eg_ctx* ctx, uint64_t* repeats_host);

/* Copies the mailboxes x_hat ([P][replica_stride] fp32) into a host buffer. Synchronises. */
eg_status eg_read_mailboxes(eg_ctx* ctx, float* xhat_host);

/* After training: the model averaged over all replicas (the final averaging step of
 * Algorithms A and B): avg_dev[e] = (1/P) sum_i params[i][e] for every
 * element of the replica layout (device buffer of replica_stride floats), fp64 sum in
 * ascending i, rounded once.  consensus_host, if not NULL, receives
 * sum_i || x_i - mean ||^2 (the consensus distance bounded in the appendix) and makes the
 * call synchronise. */
eg_status eg_average_model(eg_ctx* ctx, const float* params, float* avg_dev,
                           double* consensus_host, void* stream);

/* Checkpoint: eg_export_state with host_buf == NULL stores the needed size in *bytes;
 * otherwise writes the state and the size: iteration counter, counters, trigger state (Eq.
 * (thres): thresholds, last-event iterations, slope histories), mailboxes, and, where the
 * context has them, the delivery state (received copies, what is in flight, arrival count) and
 * the velocities.  eg_import_state restores it into a context created with the same arguments
 * and configured alike -- ring size, tensors, neighbourhood, threshold parameters, Top-K
 * fraction, readings (eg_set_variant), threshold bound, delivery masks enabled or not,
 * momentum buffer and coefficient, bits of a quantised message -- and returns EG_ERR_INVALID
 * otherwise. */
eg_status eg_export_state(eg_ctx* ctx, void* host_buf, size_t* bytes);
eg_status eg_import_state(eg_ctx* ctx, const void* host_buf, size_t bytes);

/* Change norms without any allocation.  (The paper has no counterpart: this is a service
 * entry point of the library, not a step of the method.)
 *
 * Some callers may not allocate device memory at the moment they need the norms: code that
 * runs while a stream is being captured, code inside a framework whose memory pool forbids
 * raw cudaMalloc / cudaFree (both also synchronise the whole device), or a control loop with
 * a hard latency budget.  For them this call computes
 *     norms_dev[i*T + t] = || x[i][t] - x_hat[i][t] ||_2        (fp64, device array of P*T)
 * exactly as the norm pass of eg_step does (same tiles, same summation order, hence the same
 * bits), without a context and without allocating: the tensor table is passed by value to
 * the kernels and the per-tile partial sums go to a fixed array of
 * EG_STATIC_MAX_PARTIALS doubles (4 MiB) that is part of the library's device image -- every
 * GPU that loads the library holds that array until the process exits.
 *
 * x_dev, xhat_dev: device, fp32, [P][replica_stride], 16-byte aligned; replica_stride and
 * every tensor_offset_host[t] multiples of 4 elements (no padding between tensors needed).
 * tensor_offset_host, layer_numel_host: host arrays of T entries.  Enqueues two kernels on
 * `stream` and returns; it never synchronises.
 *
 * Limits, checked before anything is launched (EG_ERR_INVALID): T <= EG_STATIC_MAX_TENSORS,
 * P <= 65535, every tensor inside its replica (offset + n_t <= replica_stride), and
 * P * sum_t ceil(n_t / 4096) <= EG_STATIC_MAX_PARTIALS.
 *
 * The first call on each device looks up the device address of the scratch array (a runtime
 * query, no allocation); make that first call outside any stream capture.  All calls on one
 * device share the scratch array: each call overwrites the part it uses (nothing has to be
 * cleared beforehand), so two calls whose kernels may overlap on the GPU (different streams)
 * race with each other -- keep them on one stream or order them with events. */
#define EG_STATIC_MAX_TENSORS 192
#define EG_STATIC_MAX_PARTIALS 524288
eg_status eg_change_norms_static(const float* x_dev, const float* xhat_dev, int P,
                                 int64_t replica_stride, const int64_t* tensor_offset_host,
                                 const int64_t* layer_numel_host, int T, double* norms_dev,
                                 void* stream);

/* Self-test of the failure path of the pipelined kernels.  Their waits on shared-memory
 * barriers are bounded: a wait that runs out sets a bit in the context's error word and the
 * kernel returns instead of hanging.  This call launches one warp that waits (for about a
 * millisecond) on a barrier that nothing completes.  It returns EG_OK when the wait gave up as
 * designed; from then on the calls that synchronise (eg_stats, eg_last_*, ...) return
 * EG_ERR_TIMEOUT until eg_reset clears the error word.  The context stays usable. */
eg_status eg_selftest_wait_timeout(eg_ctx* ctx, void* stream);

/* Back to iteration 0 of Algorithm B: empty mailboxes (X_0 = 0, Assumption 2), initial
 * thresholds, zero counters, zero velocities, the threshold bound back at its first term. */
eg_status eg_reset(eg_ctx* ctx);
void eg_destroy(eg_ctx* ctx);

/* Test hook for the allocation-failure paths: the nth device allocation the library makes from
 * now on (in any context of this process) fails as if the device were out of memory, without
 * touching the device; 0 switches the hook off.  eg_create then frees what it had allocated,
 * stores NULL in *out and returns EG_ERR_OOM. */
void eg_debug_fail_allocation(int nth);

/* Tracing: with EG_NVTX set (to anything but 0) in the environment when a context is created,
 * eg_step wraps the launches of every kernel group in a named NVTX range ("eventgrad:norm",
 * ":decide", ":topk", ":fused"); without a profiler attached the ranges cost nothing. */

/* Device-side checks.  Kernels never trap: a problem found on the device sets a bit of the
 * context's error word, the affected access is skipped, and the next call that synchronises
 * returns eg_status_of_error_word(word): EG_ERR_TIMEOUT when a bounded wait ran out (bit 8),
 * EG_ERR_INTERNAL when a Top-K entry pointed outside its message (bit 2) or -- in the
 * bounds-checked build of the library, compiled with -DEG_DEBUG (eg_debug_build() == 1) -- when
 * an index left its table (bit 4: tile records, per-replica modes, pipeline stages, partial sums,
 * entry slots are all checked before use there); EG_OK for 0.  eg_reset clears the word. */
eg_status eg_status_of_error_word(unsigned int word);
int eg_debug_build(void);

const char* eg_strerror(eg_status s);
/* cudaError_t of the most recent failed CUDA call of this context (0 if none). */
int eg_last_cuda_error(const eg_ctx* ctx);
/* Kernels launched by the most recent eg_step of this context. */
int eg_last_launch_count(const eg_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* EVENTGRAD_H */
