/*
 * lossy.h — C ABI of the packet-loss-tolerant data-parallel step for one B200.
 *
 * The library simulates, inside one GPU's HBM, the iteration of the paper's
 * "Model Formulation" section for W workers that each own one shard of a flat
 * parameter bucket:
 *
 *   (2) gradient communication  -> lossy_aggregate   (unbiased estimate, Section 3 step (2))
 *   (3) local update            -> lossy_step        (Section 3 step (3); SGD or Adam)
 *   (4) parameter broadcast     -> lossy_broadcast   (Section 3 step (4), stale retention)
 *   drift between replicas      -> drift_norms       ("Quantifying Model Drift")
 *   all four in one pass        -> lossy_fused_step
 *
 * Conventions shared by every entry point
 *   - Every data pointer is DEVICE memory owned by the caller unless the comment
 *     says "host". Pointer tables (`grads`, `replicas`) are HOST arrays of W
 *     device pointers; they are copied into the kernel arguments at the call.
 *   - All data pointers must be 16-byte aligned. `packet_elems` must be a
 *     multiple of 8 so that every packet starts on a 16-byte boundary in both
 *     supported element types.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream). Calls are asynchronous on that stream and never synchronise.
 *   - `step` is 1-based: it is the hash's step counter and Adam's t.
 *   - Return value: LOSSY_OK or an error code; nothing throws, nothing traps on
 *     the device. A bad argument is rejected before any launch.
 *   - A context owns scratch that its calls share (partial sums, a block counter):
 *     issue the calls of one context on one stream, or order them with events,
 *     and from one host thread at a time. Different contexts are independent and
 *     may be driven from different host threads (the little process-wide state the
 *     launches share is locked inside the library).
 *   - After LOSSY_ECUDA the context stays usable only if the CUDA error was not
 *     sticky (a failed launch configuration is not; a device fault is): check the
 *     runtime's own error state before going on.
 *   - The bucket is cut into K = ceil(n / packet_elems) packets of
 *     `packet_elems` contiguous elements (the last may be short). Shard j, owned
 *     by worker j, is the contiguous packet range [j*pps, min(K,(j+1)*pps)) with
 *     pps = ceil(K / W)  (Section 3: theta = (theta^(1) ... theta^(N))).
 *   - Packets evolve independently of one another, so a bucket may be split into packet
 *     ranges run by different contexts (or GPUs): see shard_packet0 / bucket_packets.
 *   - Packet k of the bucket has the global packet id packet_base + k; only the
 *     drop-mask hash sees the global id, so a model can be streamed bucket by
 *     bucket with independent masks.
 */
#ifndef LOSSY_H_
#define LOSSY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lossy_ctx lossy_ctx; /* opaque; host object + small device scratch */

enum { LOSSY_OK = 0, LOSSY_EINVAL = 1, LOSSY_ENOMEM = 2, LOSSY_ECUDA = 3, LOSSY_EDEVICE = 4,
       LOSSY_ELIMIT = 5 /* a size is beyond what drift_norms_static supports */,
       LOSSY_EDEVCHECK = 6 /* debug build only: a kernel's index check failed (lossy_device_status) */ };
enum { LOSSY_F32 = 0, LOSSY_BF16 = 1 };  /* element types of gradients / replicas */
enum { LOSSY_SGD = 0, LOSSY_ADAM = 1 };
enum {
  /* The owner's own gradient piece (src == dst) is always delivered. Default (flag
   * clear) follows the estimator as printed: the sum runs over all N workers and
   * every indicator is Bernoulli(1-p). */
  LOSSY_SELF_LOSSLESS = 1u,
  /* A packet that received nothing leaves theta, m, v untouched. Default: the
   * estimate is exactly 0 and is fed to the unmodified optimizer. */
  LOSSY_ZERO_SKIP = 2u,
  /* Every entry point uses the register-path kernel. Default: complete packets go through the
   * bulk-copy (TMA) pipelines (one for the fused step, one per single-phase call) when they hold
   * at least 1024 elements; the fused step also when they are a multiple of 128 that divides
   * the tile and the measured policy favours it (few workers, or low loss; that build also
   * fetches the dropped packets of a tile). Same parameters, replicas and masks either way; drift
   * sums agree to rounding (another summation order). */
  LOSSY_REGISTER_PATH = 4u,
  /* Owner-elided replicas. Section 3 step (4) sends a shard's new values "to all OTHER workers": the
   * owner of a shard needs no replica of it (what it owns is the master copy, and its drift term is
   * exactly 0). With this flag replica i holds the bucket WITHOUT the packets worker i owns: the
   * elements in front of worker i's shard keep their index, the elements behind it sit
   * |shard i| elements lower, and the array has lossy_replica_elems(ctx, i) elements (n minus the
   * shard). Every entry point that takes `replicas` reads and writes this layout; masks, counts,
   * parameters, moments, every element a worker does not own and the drift norms are the same as
   * without the flag. It saves 1/W of the replica memory (a full 7B-parameter model with W = 8 then
   * fits one 180 GB GPU). A replica that would hold nothing (W = 1) may be NULL.
   * drift_pairwise then sums, on every element, over the pairs of workers that both hold a copy;
   * lossy_closed_loop_grads needs full replicas and rejects such a context. */
  LOSSY_REPLICA_SKIP_OWNER = 8u,
  /* Packets shorter than a tile of the fused step: use the packed bulk-copy build (one bulk copy per worker and
   * tile, dropped sub-packets fetched too) where the launch policy allows it, instead of the gather pipeline
   * (per-lane asynchronous copies of the delivered sub-packets only). Same results; for comparison and tests. */
  LOSSY_PACKED_BULK = 16u,
  /* Packets shorter than a tile: use the gather pipeline wherever one of its builds fits, also where the launch
   * policy would pick the register kernel (many workers at high loss). Same results; for comparison and tests. */
  LOSSY_GATHER_PATH = 32u
};

#define LOSSY_MAX_WORKERS 64u

typedef struct {
  uint32_t W;            /* workers = shards = replicas, 1..64 (the paper's N)           */
  uint32_t packet_elems; /* P > 0, multiple of 8                                        */
  uint64_t n;            /* elements in the bucket; 0 makes every call a no-op          */
  uint64_t packet_base;  /* global id of this bucket's packet 0                         */
  double   p_grad;       /* drop probability of a gradient packet, in [0,1)             */
  double   p_param;      /* drop probability of a broadcast packet, in [0,1)            */
  uint64_t seed;         /* hash key; same seed => same masks, on host and device       */
  uint32_t grad_dtype;   /* LOSSY_F32 or LOSSY_BF16                                     */
  uint32_t replica_dtype;/* LOSSY_F32 or LOSSY_BF16 (bf16 = round-to-nearest-even cast) */
  uint32_t optimizer;    /* LOSSY_SGD or LOSSY_ADAM                                     */
  uint32_t flags;        /* OR of the LOSSY_* flags above */
  float lr, beta1, beta2, eps; /* eta_t and Adam's constants (beta/eps unused for SGD)  */
  /* Packet-range sharding (several GPUs simulate one bucket, each a contiguous range of its
   * packets for all W workers): this context's packet 0 is packet shard_packet0 of a bucket of
   * bucket_packets packets; owners and hash ids follow the whole bucket, `n` and every array
   * are the range's. Both 0 = the context covers the whole bucket. A range may be ragged (n not
   * a multiple of packet_elems) only if it ends the bucket. */
  uint64_t shard_packet0;
  uint64_t bucket_packets;
} lossy_config;

/*
 * lossy_init — validate `cfg`, derive the integer drop thresholds
 * T = floor(p * 2^32) (a packet is dropped iff its 32-bit hash value is < T, so
 * p = 0 never drops) and allocate the per-block partial sums the drift reduction
 * needs on the CURRENT device. `*out` receives the context; free it with
 * lossy_destroy. Section 3 fixes W (= N), p; Algorithm 1 separates p_grad and
 * p_param; Theorem "Bounded Model Drift" requires p < 1.
 * Errors: LOSSY_EINVAL (W = 0 or > 64, P = 0 or not a multiple of 8, p outside
 * [0,1), unknown enum, NULL pointer), LOSSY_ENOMEM, LOSSY_ECUDA.
 */
int lossy_init(const lossy_config* cfg, lossy_ctx** out);

/* lossy_destroy — free the context and its device scratch. NULL is allowed. */
void lossy_destroy(lossy_ctx* ctx);

/*
 * lossy_set_lr — change eta_t for the following steps (Section 3 step (3) lets the
 * learning rate depend on t). Returns LOSSY_EINVAL for a NULL context.
 */
int lossy_set_lr(lossy_ctx* ctx, float lr);

/*
 * lossy_set_bursty — replace the independent Bernoulli drops by bursty loss, the
 * correlated regime the paper's Limitations section leaves open (its analysis
 * assumes i.i.d. drops): every link (src -> dst) of every packet is a two-state
 * Gilbert-Elliott chain driven by the SAME hash value u as the independent draw,
 *     bad_t = bad_{t-1} ? (u < floor((1 - p_leave_bad) 2^32)) : (u < floor(p_enter_bad 2^32)),
 * and a transmission is lost iff its link is bad at step t (p_grad / p_param are
 * then unused). Stationary loss rate p_enter/(p_enter + p_leave), mean burst length
 * 1/p_leave; p_enter = p, p_leave = 1 - p has the statistics of independent loss.
 *   state   device, caller-owned, 4*K uint64 = [2 buffers][row 0 gradient links,
 *           row 1 broadcast links][K], bit i = the link of worker i is bad; zero it
 *           before step 1 (all links good). Step t reads buffer (t-1)&1 and writes
 *           buffer t&1, so steps must be issued in order 1, 2, 3, ... and the array
 *           belongs in a checkpoint. NULL switches back to independent loss.
 * In Algorithm 1 mode the gradient half uses one chain per packet (bit 0).
 * lossy_mask / lossy_mask_grid keep evaluating the independent draw.
 * Errors: LOSSY_EINVAL (probabilities outside 0 <= p_enter < 1, 0 < p_leave <= 1;
 * misaligned state).
 */
int lossy_set_bursty(lossy_ctx* ctx, double p_enter_bad, double p_leave_bad, uint64_t* state);

/*
 * lossy_set_reliable — hybrid reliable/unreliable transport, the first of the
 * paper's Future Directions: traffic classed as important (there: gradients of
 * large norm) goes over a reliable channel, the rest stays best-effort.
 * Transmissions whose bit is set here are never lost.
 *   reliable  device, caller-owned, 2*K uint64: row 0 gradient links (bit i of entry
 *             k = worker i's piece of packet k), row 1 broadcast links (bit i = the
 *             broadcast of packet k to replica i). Read at every later call; the
 *             caller may rewrite it between steps. NULL = everything best-effort.
 * In Algorithm 1 mode bit 0 of row 0 makes the packet's single transmission reliable.
 * The estimator is then no longer the unbiased one of the paper (reliable pieces are
 * over-represented); the paper gives no correction and none is applied.
 */
int lossy_set_reliable(lossy_ctx* ctx, const uint64_t* reliable);

/*
 * lossy_packet_sqnorms — what an importance rule starts from: the squared L2 norm
 * of every gradient piece, out[i*K + k] = sum over packet k of float(g_i[e])^2
 * (fp32, fixed summation order).
 *   grads  host array of W device pointers, each [n] of cfg.grad_dtype
 *   out    [W*K] fp32 device, written
 */
int lossy_packet_sqnorms(lossy_ctx* ctx, const void* const* grads, float* out, void* stream);

/*
 * lossy_aggregate — Section 3 step (2) and "Unbiased Gradient Aggregation":
 * for every packet k with owner j,
 *     s_i   = 1 iff hash(seed, step, src=i, dst=j, packet_base+k) >= T_grad
 *     c_k   = sum_i s_i
 *     ghat[e] = (sum over i ascending with s_i = 1 of float(g_i[e])) / float(c_k),  e in packet k
 *     ghat[e] = 0 when c_k = 0 (the regularised fallback).
 * The sum is accumulated in fp32 in ascending worker order; the division is an
 * IEEE fp32 division. Dropped packets are never read.
 *   grads      host array of W device pointers, each [n] of cfg.grad_dtype (read only)
 *   ghat       [n] fp32, written
 *   count      [K] uint8, written (c_k), or NULL
 *   recv_bits  [K] uint64, written (bit i = s_i), or NULL
 */
int lossy_aggregate(lossy_ctx* ctx, uint64_t step, const void* const* grads,
                    float* ghat, uint8_t* count, uint64_t* recv_bits, void* stream);

/*
 * lossy_step — Section 3 step (3): the owner's update of its shard with ghat,
 * in fp32, every operation rounded separately (no fused multiply-add):
 *   SGD : theta = theta - (lr * ghat)
 *   Adam: m = b1*m + (1-b1)*ghat;  v = b2*v + ((1-b2)*ghat)*ghat
 *         theta = theta - (lr * (m*ibc1)) / (sqrt(v*ibc2) + eps)
 *         ibc1 = float(1/(1-b1^step)), ibc2 = float(1/(1-b2^step)) from double on the host.
 *   count      [K] uint8 from lossy_aggregate; needed (non-NULL) only with
 *              LOSSY_ZERO_SKIP, where packets with count 0 are left untouched. (The update
 *              as the paper prints it needs only ghat; this one argument carries the
 *              "nothing arrived" fact from the aggregate to the update when the two are
 *              separate calls, which the fused call knows by itself.)
 *   master     [n] fp32, updated in place;  m, v: [n] fp32 (Adam only, else NULL)
 */
int lossy_step(lossy_ctx* ctx, uint64_t step, const float* ghat, const uint8_t* count,
               float* master, float* m, float* v, void* stream);

/*
 * lossy_broadcast — Section 3 step (4): x = cast(master) is offered to every
 * replica; replica i takes packet k iff i is its owner or
 *     hash(seed, step, src=owner, dst=i, packet_base+k) >= T_param,
 * otherwise the replica's packet is left exactly as it was (stale).
 *   master     [n] fp32 (read only)
 *   replicas   host array of W device pointers, each [n] of cfg.replica_dtype (with
 *              LOSSY_REPLICA_SKIP_OWNER: [lossy_replica_elems(ctx, i)], see the flag)
 *   stale_bits [K] uint64, written (bit i = replica i kept its old packet), or NULL
 * `step` must be >= 1 here and in lossy_aggregate too (LOSSY_EINVAL otherwise).
 */
int lossy_broadcast(lossy_ctx* ctx, uint64_t step, const float* master,
                    void* const* replicas, uint64_t* stale_bits, void* stream);

/*
 * drift_norms — "Quantifying Model Drift": for every replica i
 *     d_i = sqrt( sum_e ( float(replica_i[e]) - float(cast(master[e])) )^2 )
 * i.e. the distance of worker i's copy from the owners' current values.
 *   norms  [W] fp32, written, or NULL
 *   sumsq  [W] fp64, the squared sums are ADDED to it (sum several buckets by
 *          zeroing it once and calling per bucket), or NULL
 * The reduction order is fixed, so the result is reproducible run to run.
 */
int drift_norms(lossy_ctx* ctx, const float* master, const void* const* replicas,
                float* norms, double* sumsq, void* stream);

/*
 * drift_pairwise — the theorem's own quantity ("Quantifying Model Drift":
 * D = theta^(i,j) - theta^(k,j) between two workers' copies): for every pair
 *     d2[i*W + k] += sum_e ( float(replica_i[e]) - float(replica_k[e]) )^2 .
 * A diagnostic: it re-reads each replica once per block of four partner
 * replicas and is not part of the timed step.
 *   d2   [W*W] fp64 device, ADDED to (zero it first; symmetric, zero diagonal)
 * The sum over thread blocks uses fp64 atomics, so its order is not fixed: two
 * runs agree to about 1e-15 relative, not bit for bit.
 */
int drift_pairwise(lossy_ctx* ctx, const void* const* replicas, double* d2, void* stream);

/*
 * drift_norms_static — the same norms as drift_norms for callers that must not
 * allocate device memory. The paper has no counterpart: this entry point exists
 * only for the way the library is embedded.
 *
 * Some callers cannot call cudaMalloc: a training loop that lives inside a
 * framework's frozen memory pool, a process that has already committed all of
 * HBM to its own buffers, a service that bans allocation calls after start-up
 * because they synchronise the device. lossy_init allocates (the per-block
 * partial sums of the drift reduction), so such a caller cannot have a context.
 * This function therefore takes the configuration itself and keeps the partial
 * sums in a fixed 512 KB array that is part of the library image (held by every
 * GPU that loads the library, until the process exits). It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 *   cfg       host pointer; W, n, packet_elems and replica_dtype are used (the
 *             chunks of the reduction follow the packet grid), and of the flags
 *             LOSSY_REPLICA_SKIP_OWNER with shard_packet0 / bucket_packets (the
 *             replica layout depends on the shard map); the rest is ignored
 *   master    [n] fp32 device;  replicas: host array of W device pointers, each [n]
 *   norms     [W] fp32 device, written, or NULL;  sumsq: [W] fp64 device, ADDED to,
 *             or NULL (at least one of the two)
 *
 * Limits: W <= 64 and ceil(n / packet_elems) * ceil(packet_elems / 256) <=
 * LOSSY_STATIC_MAX_CHUNKS; anything larger returns LOSSY_ELIMIT and launches
 * nothing. The grid is capped at the 1024 rows of the static array.
 * First call on a device: looks up the device address of the static array
 * (cudaGetSymbolAddress, with that device current) and caches it; make that
 * first call at start-up, before any stream capture begins and before the
 * process commits or freezes the rest of its device memory: CUDA loads a
 * library's device code on first use, and that first use is what reserves the
 * kernels' and the array's memory (LOSSY_ENOMEM if there is no room for it).
 * The cached address does not survive a cudaDeviceReset of that device.
 * Sharing: every call in the process uses the same array and finds the last
 * call's contents in it; each call overwrites every row it later reads, so
 * nothing needs clearing, but two calls that overlap on the GPU (different
 * streams, or different host threads without ordering) race on it: serialise
 * them on one stream or with events.
 * Results agree with drift_norms up to the rounding of the fixed summation order.
 */
#define LOSSY_STATIC_MAX_CHUNKS 0x7FFFFFFFull
int drift_norms_static(const lossy_config* cfg, const float* master, const void* const* replicas,
                       float* norms, double* sumsq, void* stream);

/*
 * lossy_fused_step — steps (2), (3), (4) and the drift norms in ONE pass over
 * the bucket; ghat is not materialised unless asked for. The state it leaves
 * (master, m, v, replicas), ghat, the counts and the bit sets are bit-identical
 * to the sequence lossy_aggregate -> lossy_step -> lossy_broadcast ->
 * drift_norms; the norms agree up to the rounding of a different (but fixed)
 * summation order.
 * Optional outputs (NULL to skip): ghat [n], count [K], recv_bits [K],
 * stale_bits [K], norms [W], sumsq [W] (added to, as in drift_norms).
 */
int lossy_fused_step(lossy_ctx* ctx, uint64_t step, const void* const* grads,
                     float* master, float* m, float* v, void* const* replicas,
                     float* ghat, uint8_t* count, uint64_t* recv_bits,
                     uint64_t* stale_bits, float* norms, double* sumsq, void* stream);

/*
 * lossy_aggregate_alg1 / lossy_fused_step_alg1 — the gradient half of the paper's
 * Algorithm 1 ("Drop simulation on worker n") in place of Section 3's per-link loss:
 * the gradient reduce is reliable (plain mean over all W workers, ascending order,
 * fp32, divided by W), then ONE draw per packet,
 *     keep = hash(seed, step, src=owner, dst=owner, packet_base+k) >= T_grad,
 * decides: keep => ghat = mean and ghat_prev <- mean; drop => ghat = ghat_prev and
 * ghat_prev is left as it was (the two branches of Algorithm 1's gradient loop).
 * The algorithm's renormalisation step is read as the division of the reduced
 * sum by the worker count. Shard-granular loss, as the algorithm prints it,
 * is packet_elems = shard length. The parameter half (stale-retaining broadcast with
 * p_param) and everything else are those of lossy_aggregate / lossy_fused_step.
 *   ghat_prev  [n] fp32 device, caller-owned state, zero before the first step;
 *              read on a drop, written on a keep
 *   count[k]   W for a kept packet, 0 for a dropped one; recv_bits all ones / zero
 * Gradients of a dropped packet are not read. LOSSY_SELF_LOSSLESS contexts are
 * rejected (LOSSY_EINVAL); with LOSSY_ZERO_SKIP a dropped packet skips the optimizer.
 */
int lossy_aggregate_alg1(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev,
                         float* ghat, uint8_t* count, uint64_t* recv_bits, void* stream);
int lossy_fused_step_alg1(lossy_ctx* ctx, uint64_t step, const void* const* grads, float* ghat_prev,
                          float* master, float* m, float* v, void* const* replicas,
                          float* ghat, uint8_t* count, uint64_t* recv_bits,
                          uint64_t* stale_bits, float* norms, double* sumsq, void* stream);

/*
 * lossy_fused_step_host — the same step for a caller whose gradients live in
 * HOST memory, with the W norms delivered to host memory.
 * Pinned (page-locked, device-mapped) buffers are read by the kernel directly over
 * PCIe: there is no staging copy, and the packets the network dropped are never
 * transferred at all. If any buffer is pageable, every worker's gradient is first
 * copied into dev_grads[i] on `stream`. The call returns after the stream has been
 * synchronised (through lossy_device_status), so `host_norms` is valid on return.
 *   host_grads  host array of W HOST pointers, each [n] of cfg.grad_dtype, 16-byte aligned
 *   dev_grads   host array of W DEVICE staging pointers, each [n], caller-owned; only
 *               used (and only then required to be non-NULL) for pageable host memory
 *   dev_norms   [W] fp32 device; host_norms [W] fp32 host
 */
int lossy_fused_step_host(lossy_ctx* ctx, uint64_t step, const void* const* host_grads,
                          void* const* dev_grads, float* master, float* m, float* v,
                          void* const* replicas, float* dev_norms, float* host_norms,
                          void* stream);

/*
 * lossy_closed_loop_grads — a stand-in for Section 3 step (1), "local gradient
 * computation", that restores the feedback the paper describes there: worker i
 * computes its gradient at ITS OWN, possibly stale, replica. The objective is a
 * diagonal quadratic, L(theta) = 1/2 sum_e a[e] (theta[e] - x*[e])^2, so
 *     g_i[e] = cast( a[e] * (float(replica_i[e]) - x*[e]) + float(noise_i[e]) ),
 * subtraction, multiplication and addition each rounded to fp32 on their own,
 * cast = identity or RNE to bf16 (cfg.grad_dtype). Call it before
 * lossy_fused_step to run the method in closed loop on synthetic data.
 *   curv, target  [n] fp32 device (a and x*)
 *   noise         host array of W device pointers, each [n] of cfg.grad_dtype
 *                 (the mini-batch noise of worker i, drawn by the caller)
 *   replicas      host array of W device pointers, each [n] of cfg.replica_dtype
 *   grads_out     host array of W device pointers, each [n] of cfg.grad_dtype, written
 */
int lossy_closed_loop_grads(lossy_ctx* ctx, const float* curv, const float* target,
                            const void* const* noise, const void* const* replicas,
                            void* const* grads_out, void* stream);

/*
 * lossy_device_status — synchronise `stream` and report whether any kernel of
 * this context gave up a bounded wait (the bulk-copy pipeline bounds every wait
 * on its barriers instead of spinning forever). LOSSY_OK, or LOSSY_EDEVICE if
 * the results of an earlier call on this context must be discarded. The paper
 * has no counterpart; this is the library's failure report.
 * The status word is sticky: once set it stays set, and every later
 * lossy_device_status on the context returns LOSSY_EDEVICE, until
 * lossy_reset_status clears it.
 */
int lossy_device_status(lossy_ctx* ctx, void* stream);

/*
 * Debug build. The same sources compiled with -DLOSSY_DEVCHECK give a second
 * library (liblossy_b200_check.so) with the same entry points, in which every
 * kernel of the step path (register kernel, fused and single-phase bulk-copy
 * pipelines, gather pipeline) checks, before it touches memory for a chunk or
 * tile, that the packet index is one of the context's packets, that the element
 * range lies inside the slab, and that every replica's range (through the
 * owner-elided index map where that layout is on) lies inside that replica's
 * array. A range that fails is recorded (first failure wins: kernel, array kind,
 * offset, length) and is not touched: the register kernel skips the chunk, a
 * pipeline stops through its bounded-wait exit. Nothing traps or asserts. The
 * next lossy_device_status returns LOSSY_EDEVCHECK with the record in
 * lossy_last_error; lossy_reset_status clears it. The checks stand in for a
 * memory-checking tool where none can be run; the normal build contains none of
 * them (they compile to nothing) and never returns LOSSY_EDEVCHECK.
 *
 * lossy_has_device_checks — 1 in the debug build, 0 in the normal one.
 *
 * lossy_selftest_shrink_checks — a test hook of the debug build: from the next
 * call on, the checks hold every range against n - elems elements instead of n
 * (elems = 0 restores n), so that ranges near the end fail their check although
 * the arrays behind them are whole: the failure report runs without an access
 * out of bounds. LOSSY_EINVAL in the normal build. The paper has no counterpart.
 */
int lossy_has_device_checks(void);
int lossy_selftest_shrink_checks(lossy_ctx* ctx, uint64_t elems);

/*
 * lossy_reset_status — clear the context's device status word and its
 * finished-block counter on `stream` (asynchronous), so that the context can be
 * used again after a reported LOSSY_EDEVICE. The state arrays of the step that
 * reported it (master, m, v, replicas) are the caller's to restore, e.g. from a
 * checkpoint: a kernel that gave up may have updated some tiles and not others.
 * The paper has no counterpart.
 */
int lossy_reset_status(lossy_ctx* ctx, void* stream);

/*
 * lossy_selftest_wait_expiry — exercise the failure report without a failure.
 * Launches one small thread block that waits, with the pipelines' own bounded
 * wait and a poll limit of `max_polls` (1 .. 2^20), on a barrier that nothing
 * will ever complete; no copy is in flight. The wait runs out, the block leaves
 * through the pipelines' exit path and sets this context's status word, so the
 * next lossy_device_status returns LOSSY_EDEVICE. Nothing faults, traps or hangs,
 * and the device context stays usable. A test hook; the paper has no counterpart.
 */
int lossy_selftest_wait_expiry(lossy_ctx* ctx, uint32_t max_polls, void* stream);

/*
 * lossy_mask — host evaluation of one delivery indicator of Section 3:
 * returns 1 if the transmission (src -> dst) of global packet `packet` at `step`
 * is delivered, 0 if dropped, using T_param when `is_param` is non-zero and
 * T_grad otherwise. The device kernels evaluate the same integer function.
 * Returns -1 for a NULL context.
 */
int lossy_mask(const lossy_ctx* ctx, uint64_t step, uint32_t src, uint32_t dst,
               uint64_t packet, int is_param);

/*
 * lossy_hash_u32 — the 32-bit uniform value behind lossy_mask (context-free).
 */
uint32_t lossy_hash_u32(uint64_t seed, uint64_t step, uint32_t src, uint32_t dst,
                        uint64_t packet);

/*
 * lossy_mask_grid — evaluate delivery indicators on the DEVICE for a dense grid
 * (a test hook that proves host and device agree): for q in [0, count),
 * out[q] = delivered(step, src[q], dst[q], packet[q]) as uint8.
 *   src, dst  [count] uint32 device; packet [count] uint64 device; out [count] uint8 device
 */
int lossy_mask_grid(lossy_ctx* ctx, uint64_t step, const uint32_t* src, const uint32_t* dst,
                    const uint64_t* packet, uint64_t count, int is_param, uint8_t* out,
                    void* stream);

/* lossy_last_error — text of the last error on this context (host string, never NULL). */
const char* lossy_last_error(const lossy_ctx* ctx);

/* lossy_num_packets — K = ceil(n / packet_elems) for this context (0 for NULL). */
uint64_t lossy_num_packets(const lossy_ctx* ctx);

/* lossy_replica_elems — elements replica `worker`'s array holds: n, or with LOSSY_REPLICA_SKIP_OWNER n minus
 * the elements of that worker's own shard inside this context's packet range (0 for NULL or worker >= W). */
uint64_t lossy_replica_elems(const lossy_ctx* ctx, uint32_t worker);

/* lossy_kernel_launches — kernels this context has launched so far (0 for NULL). */
uint64_t lossy_kernel_launches(const lossy_ctx* ctx);

/* lossy_describe_plan — which kernel build lossy_fused_step would launch for the complete packets of
 * this context, as text for logs and benchmarks: "bulk-copy wide|twin group=4|8 stale=late|early|staged
 * [packed] [split] stages=N", or "register kernel" when no bulk-copy build fits (a ragged last packet goes
 * to the register kernel in either case). with_drift != 0 asks for the call that also returns drift norms.
 * Host only: launches nothing and allocates nothing. Writes at most size bytes including the terminator
 * (truncating); buf is a host buffer owned by the caller. LOSSY_EINVAL for a NULL argument or size 0.
 * The paper has no counterpart: the build choice is this library's measured launch policy. */
int lossy_describe_plan(lossy_ctx* ctx, int with_drift, char* buf, size_t size);

#ifdef __cplusplus
}
#endif
#endif /* LOSSY_H_ */
