/*
 * rudra_ps.h -- C interface of the B200 parameter-server update path of the Rudra framework
 * (Gupta, Zhang, Wang, "Model Accuracy and Runtime Tradeoff in Distributed Deep Learning: A
 * Systematic Study", arXiv 1509.04210).
 *
 * The server of Section 2 does two things: sumGradients (receive and accumulate the learners'
 * gradients) and applyUpdate (multiply the accumulated gradient by the learning rate and update
 * the weights, Eq. 1c).  Under the n-softsync protocol of Section 3.1 (Eq. 5) it updates after
 * collecting c = floor(lambda / n) gradients, averaging them; every update raises a scalar
 * weight timestamp by one, a gradient carries the timestamp of the weights it was computed
 * from, and its staleness sigma is the server's timestamp minus the gradient's (Section 3.1).
 * The learning rate is divided by the staleness (Section 3.2; Eq. 6: alpha = alpha0 / n).
 * pullWeights hands a learner the weights and their timestamp (Section 2, Section 3.2).
 *
 * Conventions
 *   - Plain C, no exceptions cross this boundary, the library never aborts the process.
 *   - "dev" pointers are CUDA device addresses on the device that was current at create time;
 *     "host" pointers are ordinary (preferably page-locked) host addresses.
 *   - Every device vector is flat and contiguous and must start on a 32-byte boundary (the
 *     kernels move 256 bits per access).  For full speed start vectors on a 1 KB boundary: a
 *     warp moves 1 KB per instruction, and on a B200 a window of updates at 61 M weights runs
 *     3 % slower with 512-byte-aligned vectors and 7 % slower with 32-byte-aligned ones.
 *   - Return values: >= 0 success, < 0 one of the RUDRA_E_* codes; rudra_last_error() gives
 *     the reason as text.
 *   - All device work is enqueued on the handle's stream and is asynchronous to the host;
 *     only rudra_ps_sync and rudra_ps_destroy wait for the device.  The kernels contain no
 *     waits, flags or inter-block communication.
 *   - A handle is not thread-safe (the server of Section 3.2 handles messages one at a time);
 *     distinct handles are independent.
 *   - A pull destination must not overlap a gradient buffer that is still queued; two pulls may
 *     name the same destination, in which case the later one wins.
 *   - There is no CPU implementation behind these calls.
 */
#ifndef RUDRA_PS_H
#define RUDRA_PS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rudra_ps rudra_ps;
typedef struct rudra_sched rudra_sched;

/* error codes */
#define RUDRA_E_INVAL      (-1) /* null / misaligned pointer, bad argument, bad handle          */
#define RUDRA_E_BAD_TS     (-2) /* pulled_ts is ahead of the server timestamp                    */
#define RUDRA_E_QUEUE_FULL (-3) /* more than RUDRA_QUEUE_CAP gradients waiting                   */
#define RUDRA_E_CUDA       (-4) /* a CUDA call failed; text in rudra_last_error()                */
#define RUDRA_E_STATE      (-5) /* call not legal in the current state (e.g. queue not empty)    */
#define RUDRA_E_NOMEM      (-6) /* host memory ran out inside the call; destroy the handle       */

#define RUDRA_MAX_GROUP  128    /* largest c = floor(lambda / n) one update can combine          */
#define RUDRA_MAX_DSTS   128    /* most destinations of one pull_many / step_pull_many           */
#define RUDRA_QUEUE_CAP  4096   /* most gradients that may wait in the queue                     */
#define RUDRA_HIST_BINS  4096   /* staleness histogram: the last bin counts this much and more   */

/* rudra_ps_set_option keys and values */
#define RUDRA_OPT_GRAD_DTYPE 1
#define   RUDRA_GRAD_F32  0     /* gradients are float (the paper's precision, Section 4.2)      */
#define   RUDRA_GRAD_BF16 1     /* gradients are bfloat16; weights and state stay float          */
#define RUDRA_OPT_LR_POLICY 2
#define   RUDRA_LR_PAPER_N      0 /* alpha = alpha0 / n for every gradient (Eq. 6)               */
#define   RUDRA_LR_PER_GRADIENT 1 /* alpha_l = alpha0 / max(sigma_l, 1) (Section 5.1, footnote)  */
#define   RUDRA_LR_GROUP_MEAN   2 /* alpha = alpha0 / max(<sigma>, 1), <sigma> of Eq. 2          */
#define RUDRA_OPT_OPTIMIZER 3
#define   RUDRA_OPTIM_MOMENTUM_SGD 0 /* momentum-accelerated SGD with weight decay (Section 4.2) */
#define   RUDRA_OPTIM_ADAGRAD      1 /* AdaGrad at the server (Section 5.5)                      */
#define RUDRA_OPT_PUSH_MODE 4
#define   RUDRA_PUSH_BORROW 0   /* a pushed device buffer is read by the update that consumes it */
#define   RUDRA_PUSH_COPY   1   /* the server copies it at push time (Section 3.2: the message   */
                                /* carries the gradient); costs one more read and write of it    */
#define RUDRA_OPT_TREE_FANIN 5  /* learners per leaf when rudra_ps_run_events plays the server    */
                                /* tree of Section 3.3; 0 (default): learners talk to the server */

/*
 * rudra_ps_create -- a parameter server for a flat model of nparams weights, lambda learners and
 * splitting parameter n (Section 3.1: 1 <= n <= lambda, c = floor(lambda / n) gradients per
 * update).  alpha0 is the base learning rate of Eq. 6, momentum and weight_decay those of
 * Section 4.2.  Allocates the weights and one state vector (fp32, zeroed) on the current device;
 * timestamp = 0.  Returns NULL on invalid arguments (nparams == 0, lambda == 0, n == 0,
 * n > lambda, c > RUDRA_MAX_GROUP, negative or non-finite alpha0 / momentum / weight_decay,
 * momentum >= 1) or CUDA failure.
 */
rudra_ps* rudra_ps_create(uint64_t nparams, uint32_t lambda, uint32_t n,
                          float alpha0, float momentum, float weight_decay);

/* Frees everything the handle owns after waiting for its stream.  NULL is a no-op. */
void rudra_ps_destroy(rudra_ps* ps);

/* All later device work of this handle goes to cuda_stream (a cudaStream_t / CUstream value,
 * e.g. torch.cuda.Stream().cuda_stream); NULL selects the legacy default stream.  The call does
 * not wait for or order anything: work already enqueued on the previous stream (updates, copies
 * of queued COPY-mode gradients) must have finished, or the caller must make the new stream wait
 * for it, before the next call that touches the device. */
int rudra_ps_set_stream(rudra_ps* ps, void* cuda_stream);

/* Sets one RUDRA_OPT_* key.  Only legal while no gradient is queued (else RUDRA_E_STATE).
 * Changing the optimizer zeroes the state vector. */
int rudra_ps_set_option(rudra_ps* ps, int key, int64_t value);

/* Base learning rate for later updates (the step schedule of Section 4.2 divides it by 10). */
int rudra_ps_set_alpha0(rudra_ps* ps, float alpha0);

/* Copies nparams floats from src into the weights, zeroes the state, resets the timestamp to 0
 * and empties the queue.  src_dev: device memory; src_host: host memory (copied on the stream). */
int rudra_ps_set_weights(rudra_ps* ps, const float* src_dev);
int rudra_ps_set_weights_host(rudra_ps* ps, const float* src_host);

/*
 * rudra_ps_push -- pushGradient as the server sees it (Section 2; Section 3.2: the message is the
 * gradient plus the timestamp of the weights it was computed from).  grad_dev: nparams elements
 * of the configured gradient type in device memory.  The buffer is BORROWED: it is read by the
 * update that consumes it and must stay valid and unchanged until that update has run on the
 * stream (re-use ordered on the same stream is safe).  pulled_ts must not exceed the server's
 * timestamp (RUDRA_E_BAD_TS).  Returns the number of gradients now queued.  No device work.
 */
int64_t rudra_ps_push(rudra_ps* ps, const void* grad_dev, uint64_t pulled_ts);

/* With RUDRA_OPT_PUSH_MODE = RUDRA_PUSH_COPY, rudra_ps_push (and the PUSH events of
 * rudra_ps_run_events, and rudra_ps_push_group) copy the vector into a buffer the handle owns,
 * on the handle's stream, before returning: the caller may overwrite or free grad_dev with any work
 * ordered after the call on that stream.  For learners that cannot keep a buffer alive until the
 * group closes.  Buffers are allocated on first use and re-used. */

/* Same, for a gradient in host memory: it is copied into a staging buffer the handle owns
 * (allocated on first use, re-used afterwards) on an upload stream of the handle's own, so that
 * uploads, updates and rudra_ps_pull_host downloads overlap; the consuming update waits for the
 * copy.  grad_host may be re-used after rudra_ps_sync.  Page-locked memory makes the copy
 * asynchronous. */
int64_t rudra_ps_push_host(rudra_ps* ps, const void* grad_host, uint64_t pulled_ts);

/*
 * rudra_ps_step -- one weight update if at least c gradients are queued (Eq. 5): takes the c
 * oldest, fixes sigma_l = timestamp - pulled_ts_l (Section 3.1), records the vector clock and
 * <sigma> (Eq. 2), forms the per-gradient step sizes s_l = alpha_l / c (Eq. 5, Eq. 6), enqueues
 * ONE fused kernel that computes, per weight k,
 *     acc = sum_l s_l * g_l[k];  u = acc + (sum_l s_l) * weight_decay * theta[k];
 *     v[k] = momentum * v[k] + u;  theta[k] -= v[k]
 * and raises the timestamp by one.  Returns 1 if an update was enqueued, 0 if fewer than c
 * gradients wait (nothing changes), < 0 on error.
 */
int rudra_ps_step(rudra_ps* ps);

/*
 * The server tree of Section 3.3 (Rudra-adv), two levels.  A leaf node sits with the learners it is
 * responsible for, averages the gradients they send and relays the average to its parent; the
 * root -- this handle -- applies the update, and all weights keep one timestamp.
 *
 * rudra_leaf_average is the leaf's work: avg_dev[i] = mean over l of grads_dev[l][i] for k vectors
 * of grad_dtype (RUDRA_GRAD_F32 / RUDRA_GRAD_BF16), nparams elements each; the result is a float
 * vector like every message of the paper (Section 4.2).  It needs no handle and may run on the
 * leaf's own GPU, with avg_dev in the root's memory (peer access enabled by the caller): k vectors
 * are read locally and one crosses the link.  Per weight: k reads and one 4-byte write.
 *
 * rudra_ps_push_group hands the root one message that stands for k gradients, with the timestamps
 * of all k (pulled_ts[0..k-1]): the root's vector clock, staleness and Eq. 2 are then those of a
 * server that received the k gradients itself.  nvec == 1: vecs_dev[0] is the leaf's average (float;
 * the handle's gradient type must be RUDRA_GRAD_F32).  nvec == k: vecs_dev[0..k-1] are the k raw
 * gradients of the handle's gradient type, for a leaf that shares the root's GPU -- the update
 * kernel averages them on the way and no intermediate vector is written.  The message takes the
 * share k / c of Eq. 5's average at the rate of Eq. 6; under RUDRA_LR_PER_GRADIENT the rate is
 * alpha0 / max(mean staleness of the message's gradients, 1).  A message must fit the open group
 * (queued % c + k <= c, else RUDRA_E_STATE).  Buffers are borrowed or copied as in rudra_ps_push.
 * Returns the number of gradients now queued.
 *
 * rudra_ps_last_messages reports, for the most recent update, how many gradients each of its
 * messages stood for and the step size its vector was multiplied by; returns the message count.
 * (rudra_ps_last_clock's scale_out is that step size divided by the fan-in, per gradient.)
 */
int rudra_leaf_average(const void* const* grads_dev, uint32_t k, int grad_dtype, uint64_t nparams, float* avg_dev,
                       void* cuda_stream);
int64_t rudra_ps_push_group(rudra_ps* ps, const void* const* vecs_dev, uint32_t nvec, const uint64_t* pulled_ts,
                            uint32_t k);
int rudra_ps_last_messages(const rudra_ps* ps, uint32_t* fanin_out, float* step_out);

/* Like rudra_ps_step, and the same kernel also writes the new weights into k learner buffers
 * (dsts_dev: host array of k device pointers, each nparams floats, 0 <= k <= RUDRA_MAX_DSTS):
 * the update followed by k pulls at the cost of one read of the weights.  Section 3.1's hardsync
 * broadcast and Section 3.3's weight down-cast are this call with k = lambda. */
int rudra_ps_step_pull_many(rudra_ps* ps, float* const* dsts_dev, uint32_t k);

/*
 * rudra_ps_pull -- pullWeights (Section 2, Section 3.2): enqueues a copy of the weights, as of
 * every update issued so far, into dst (caller-owned, nparams floats) and returns their
 * timestamp.  rudra_ps_pull_many serves k learners with one read of the weights.
 * rudra_ps_pull_host copies to host memory: a device snapshot on the handle's stream, then the
 * transfer on a download stream of the handle's own, so later updates do not wait for the link;
 * dst_host is complete after rudra_ps_sync.
 */
int64_t rudra_ps_pull(rudra_ps* ps, float* dst_dev);
int64_t rudra_ps_pull_host(rudra_ps* ps, float* dst_host);
int64_t rudra_ps_pull_many(rudra_ps* ps, float* const* dsts_dev, uint32_t k);

/* The timestamp inquiry of Section 3.2: a learner whose copy already has this timestamp skips
 * the pull.  Host only. */
int64_t rudra_ps_timestamp(const rudra_ps* ps);

/* Vector clock of the most recent update (Section 3.1): the c gradient timestamps, their
 * staleness, the step sizes s_l used, and <sigma> of Eq. 2.  Any output may be NULL.  Returns c,
 * or 0 before the first update. */
int rudra_ps_last_clock(const rudra_ps* ps, uint64_t* pulled_ts_out, uint32_t* sigma_out,
                        float* scale_out, double* avg_sigma_out);

/* The server's record of its updates: Section 3.2 has the server log every update's vector clock
 * so that the average staleness can be followed over training (Fig. 3 plots both).
 * rudra_ps_clock_log copies
 * out, for the updates that advanced the timestamp from first_ts, first_ts + 1, ... (at most
 * count of them, only the most recent 4096 are kept), the c gradient timestamps of each
 * (pulled_ts_out, count * c entries, may be NULL) and its <sigma> by Eq. 2 (avg_sigma_out, count
 * entries, may be NULL); returns how many were written, RUDRA_E_STATE if first_ts has left the
 * log.  rudra_ps_staleness_histogram writes how many gradients had staleness 0, 1, ..., nbins - 1
 * since create (set_weights and import_state do not reset it) and returns the number of bins
 * needed to hold every value seen, at most RUDRA_HIST_BINS: the bin RUDRA_HIST_BINS - 1 also counts
 * every larger staleness. */
int64_t rudra_ps_clock_log(const rudra_ps* ps, uint64_t first_ts, uint64_t count, uint64_t* pulled_ts_out,
                           double* avg_sigma_out);
int64_t rudra_ps_staleness_histogram(const rudra_ps* ps, uint64_t* counts_out, uint32_t nbins);

/* Checkpoint hooks: device-to-device copies of the weights and the state vector (either may be
 * NULL) out of / into the handle; import also sets the timestamp and empties the queue. */
int rudra_ps_export_state(rudra_ps* ps, float* theta_dst_dev, float* state_dst_dev);
int rudra_ps_import_state(rudra_ps* ps, const float* theta_src_dev, const float* state_src_dev, uint64_t ts);

/* Waits for the handle's stream and its upload / download streams; reports asynchronous CUDA
 * errors as RUDRA_E_CUDA. */
int rudra_ps_sync(rudra_ps* ps);

/* Counters since create: out[0] pushes, out[1] updates, out[2] pulls served (learners),
 * out[3] kernels launched, out[4] bytes copied host->device, out[5] bytes copied device->host,
 * out[6] copies of the weights written for pulls, out[7] of those, shared versions (zero-copy). */
int rudra_ps_counters(const rudra_ps* ps, uint64_t out[8]);

/*
 * Zero-copy pulls.  Section 3.3 gives each learner a computation buffer and a communication
 * buffer for pullWeights, so that switching to newly received weights costs an exchange of two
 * pointers and no copy.  With learners and server sharing one GPU's memory the same idea removes the copy: the handle
 * keeps a pool of nversions immutable weight vectors, a pull hands the learner a pointer to the
 * one holding the current timestamp, and learners that pull the same timestamp share it -- a
 * version is written once (4 bytes per weight, by the update kernel when the pull sits in a
 * rudra_ps_run_events batch) however many learners read it.
 *
 * rudra_ps_enable_views allocates the pool (nparams floats each; legal only while no learner holds
 * a view).  rudra_ps_pull_view gives learner `learner` (0 <= learner < lambda) the current
 * version and takes back the one it held; returns the timestamp and stores the device pointer in
 * *view_out.  The pointer stays valid, and the vector behind it unchanged, until the same
 * learner's next pull; the learner must have finished reading the old vector (ordered before the
 * handle's stream) when it makes that call.  If every version is still held by some learner the
 * call fails with RUDRA_E_STATE and nothing changes: lambda + 1 versions always suffice.
 * While views are enabled, the PULL and BROADCAST events of rudra_ps_run_events are served this
 * way (slots_dev is ignored; BROADCAST hands the current version to all lambda learners) and
 * rudra_ps_view_of reads back a learner's current view and its timestamp.
 */
int rudra_ps_enable_views(rudra_ps* ps, uint32_t nversions);
int64_t rudra_ps_pull_view(rudra_ps* ps, uint32_t learner, const float** view_out);
int64_t rudra_ps_view_of(const rudra_ps* ps, uint32_t learner, const float** view_out);

/* Reason of the calling thread's most recent failure; static storage, never freed. */
const char* rudra_last_error(void);

/*
 * rudra_ps_update_host_noalloc -- (The paper has no counterpart to this call; it exists for
 * callers of this library that cannot allocate device memory.)
 *
 * Who needs it: a process that gave the whole GPU to its own memory pool at start-up, so that a
 * later cudaMalloc fails or fragments the pool; or a loop that cannot tolerate the device-wide
 * synchronisation an allocation causes.  rudra_ps_push_host stages host gradients in device
 * buffers that it allocates on demand; this call does the same update with no allocation at all
 * (no cudaMalloc, no cudaFree, no allocating library routine): the staging area is a fixed array
 * of RUDRA_NOALLOC_MAX_FLOATS floats inside the library image, resident on every GPU that loads
 * the library until the process exits.
 *
 * What it does: copies the c fp32 gradients grads_host[0..c-1] (host memory, nparams floats each)
 * to the staging array on cuda_stream and enqueues the fused kernel of rudra_ps_step on
 * caller-owned vectors:  acc = sum_l scales[l] * g_l[k];  u = acc + (sum_l scales[l]) *
 * weight_decay * theta[k];  state[k] = momentum * state[k] + u;  theta[k] -= state[k].
 * theta_dev / state_dev: device memory, nparams floats, 32-byte aligned, updated in place
 * (state_dev may be NULL when momentum == 0).  scales: c step sizes in host memory (what
 * rudra_ps_last_clock reports as scale_out).  The timestamp bookkeeping stays with the caller.
 *
 * Limits and hazards: c * round_up(nparams, 64) must not exceed RUDRA_NOALLOC_MAX_FLOATS, else
 * RUDRA_E_INVAL with a message naming the limit.  Every call on a device shares the one array:
 * calls whose device work may overlap (different streams or threads) race on it; calls ordered on
 * one stream do not.  The array keeps the last call's gradients; nothing in it needs clearing
 * because each call overwrites all it reads.  The first call on each device looks up the array's
 * device address (cudaGetSymbolAddress, with that device current); make that first call before
 * any stream capture begins.  That first call is also where the CUDA runtime may load the
 * library's device image onto the device, which is when the 16 MiB become resident: a process
 * that is about to hand the rest of the GPU to its own pool should make one call (any small
 * update) on each device before it does so.
 * Host buffers: the gradients are copied with cudaMemcpyAsync.  From pageable memory the copy has
 * left grads_host[l] when the call returns; from page-locked memory it is asynchronous, and
 * grads_host[l] must stay unchanged until cuda_stream has passed the copies (an event recorded on
 * cuda_stream after the call, or a synchronise).  scales is read before the call returns.
 * Returns 0, or RUDRA_E_INVAL / RUDRA_E_CUDA with the reason in rudra_noalloc_last_error().
 */
#define RUDRA_NOALLOC_MAX_FLOATS (4u * 1024u * 1024u)
int rudra_ps_update_host_noalloc(float* theta_dev, float* state_dev, uint64_t nparams,
                                 const float* const* grads_host, const float* scales, uint32_t c,
                                 float momentum, float weight_decay, void* cuda_stream);
const char* rudra_noalloc_last_error(void);

/* ------------------------------------------------------------------------------------------
 * Learner event model.  The paper's server handles incoming messages strictly one by one
 * (Section 3.2), which makes the arrival order the whole control; this host-only scheduler
 * produces that order for lambda simulated learners running the loop of Section 2
 * (pull, compute, push), with the timestamp inquiry of Section 3.2.
 * ------------------------------------------------------------------------------------------ */
#define RUDRA_EV_PUSH      1 /* learner's gradient arrives; pulled_ts = timestamp it carries      */
#define RUDRA_EV_STEP      2 /* the c-th gradient of a group arrived: update; ts = new timestamp  */
#define RUDRA_EV_PULL      3 /* learner receives the weights with timestamp ts                    */
#define RUDRA_EV_PULL_SKIP 4 /* inquiry found the learner's copy current: no copy                 */
#define RUDRA_EV_BROADCAST 5 /* all lambda learners receive the weights with timestamp ts         */
#define RUDRA_EV_RELAY     6 /* server tree: leaf `learner` relays the average of its k gradients  */

#define RUDRA_SCHED_HARDSYNC        0 /* Section 3.1 hardsync: n = 1, barrier, broadcast          */
#define RUDRA_SCHED_SOFTSYNC_ROUNDS 1 /* every learner pushes once per round, seeded order        */
#define RUDRA_SCHED_SOFTSYNC_TIMED  2 /* learners with seeded lognormal compute times             */

typedef struct rudra_event {
  int32_t  kind;       /* RUDRA_EV_*                                                            */
  uint32_t learner;    /* learner the event belongs to (STEP: whose push closed the group;     */
                       /* RELAY: the leaf)                                                      */
  uint64_t pulled_ts;  /* PUSH: timestamp of the weights the gradient was computed from         */
  uint64_t ts;         /* PUSH: server timestamp at arrival; others: timestamp after the event  */
  uint64_t seq;        /* PUSH: index of this learner's mini-batch, from 0; RELAY: of the leaf's relay */
  uint64_t tick;       /* simulated arrival time (timed mode) or global push count (rounds)     */
} rudra_event;

/* mode: RUDRA_SCHED_*; hardsync requires n == 1.  lognormal_sigma: spread of ln(compute time)
 * in timed mode.  downcast != 0: after every update the new weights are broadcast to all
 * learners' receive buffers (Section 3.3), so per-learner pulls become inquiry skips.
 * Returns NULL on invalid arguments. */
rudra_sched* rudra_sched_create(uint32_t lambda, uint32_t n, int mode, uint64_t seed,
                                double lognormal_sigma, int downcast);
/* The same learners behind the two-level server tree of Section 3.3: learner l sends to leaf
 * l / fanin; a leaf that holds fanin gradients relays their average to the root at once (a RELAY
 * event right after the PUSH that filled it); the root updates when the averages it received stand
 * for c gradients.  fanin must divide lambda and c = lambda / n; fanin = 0 is rudra_sched_create. */
rudra_sched* rudra_sched_create_tree(uint32_t lambda, uint32_t n, int mode, uint64_t seed,
                                     double lognormal_sigma, int downcast, uint32_t fanin);
void rudra_sched_destroy(rudra_sched* s);
/* Writes the next count events to out; returns count, or RUDRA_E_INVAL. */
int64_t rudra_sched_next(rudra_sched* s, rudra_event* out, uint64_t count);
/* For a caller that drives real learners: learner `learner` reports that the weights it now
 * computes on carry timestamp ts (its pull was late, lost, or served from a cache), overriding
 * what its last PULL / PULL_SKIP / BROADCAST event assumed.  Its next PUSH event then carries
 * pulled_ts = ts.  Call it after reading that learner's pull event and before asking for further
 * events.  RUDRA_E_BAD_TS if ts is ahead of the simulated server, RUDRA_E_INVAL for a bad learner. */
int rudra_sched_on_pull(rudra_sched* s, uint32_t learner, uint64_t ts);

/*
 * rudra_ps_run_events -- handle a backlog of messages.  Section 3.2's server takes messages one at
 * a time and Section 5.2 / 5.5 name the cost: with many learners and small mini-batches updates
 * and pulls arrive faster than the server finishes them.  This call takes the waiting messages in
 * arrival order (events[0..count-1], as rudra_sched_next produces them) and does exactly what
 * rudra_ps_push / rudra_ps_step / rudra_ps_pull / rudra_ps_pull_many would do one by one -- same
 * timestamps, same staleness, bit-identical weights, state and pulled copies -- but packs
 * consecutive updates and the pulls between them into one launch: the weights and the state stay
 * in registers across up to max_window updates (0 = as many as the launch tables hold: at most
 * 32 updates, RUDRA_MAX_GROUP gradients and RUDRA_MAX_DSTS pull destinations per launch), every
 * gradient is read once and every pull is a store.  Per weight a window of W updates with P pulls
 * moves W*c*G + 16 + 4*P bytes instead of W*(c*G + 16) + 8*P.
 *
 * With RUDRA_OPT_TREE_FANIN = k the batch may come from rudra_sched_create_tree: PUSH events then
 * deliver to the learner's leaf and each RELAY event hands the root that leaf's k gradients as one
 * message (the leaves share this GPU: rudra_ps_push_group with nvec == k).
 *
 * grads_dev[l] is learner l's gradient buffer (read by the update that consumes the push, as in
 * rudra_ps_push), slots_dev[l] its weight buffer (written by its pulls and by broadcasts); both
 * are host arrays of lambda device pointers; slots_dev may be NULL if no event pulls.  The events'
 * ts fields are checked against the server's timestamp.  The whole batch is validated before
 * anything is queued or launched: RUDRA_E_INVAL, RUDRA_E_BAD_TS, RUDRA_E_STATE and
 * RUDRA_E_QUEUE_FULL mean that nothing has changed.  RUDRA_E_CUDA (a launch the driver refused) or
 * RUDRA_E_NOMEM can come after part of the batch was handled: timestamp, queue and counters then
 * stand where the failure left them, the weights may hold some of the batch's updates, and the
 * handle is only good for rudra_ps_destroy.  Returns the number of updates performed.
 */
int64_t rudra_ps_run_events(rudra_ps* ps, const rudra_event* events, uint64_t count,
                            const void* const* grads_dev, float* const* slots_dev, uint32_t max_window);

#ifdef __cplusplus
}
#endif
#endif /* RUDRA_PS_H */
