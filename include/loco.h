/*
 * loco.h -- C ABI of the B200 (sm_100a) LoCo hot-path library.
 *
 * LoCo (Low-bit Communication Adaptor, arXiv 2407.04480) sends gradients between
 * data-parallel workers as low-bit integer codes and feeds the compression error
 * back into the next iteration.  This library implements the two elementwise passes
 * every worker runs per gradient bucket and iteration:
 *
 *   send    (Algorithm 1, steps 1-2; Eq. 1-7): compensate the fresh gradient with the
 *           stored error, quantise, form the new moving-average error, store it in the
 *           8-bit state, pack the codes into the communication buffer;
 *   receive (Algorithm 1, step 3; Eq. 8): unpack N workers' buffers, dequantise,
 *           average in fp32, write the fp32/bf16 gradient for the optimizer.
 *
 * Conventions for every call
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  All device
 *     buffers are owned by the caller and must be 16-byte aligned and must not
 *     overlap.  The library never frees or reallocates them.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Kernel launches are asynchronous on it; nothing synchronises unless stated.
 *   - Every function that returns int returns LOCO_OK (0) or a negative loco_status_t.
 *     Nothing aborts, traps or throws.  On error no kernel has been launched.
 *   - Element counts are 64-bit; a flat buffer may exceed 2^32 elements.
 *
 * Layout of the communication buffer ("wire layout", little-endian)
 *   The bucket's n elements are cut into P = num_partitions consecutive parts of
 *   Lp = loco_partition_capacity() elements (the N parts of Sec. 3.3; the last parts
 *   may be short or empty).  Part j occupies bytes [j*stride, (j+1)*stride),
 *   stride = loco_partition_bytes():
 *       [ codes: Lp*p/8 bytes ][ scales: (Lp/B) fp32, BLOCK_ABSMAX only ][ pad to 128 B ]
 *   Element o of a part is the p-bit two's-complement field at bit (o mod 8/p)*p of
 *   byte o*p/8 (4-bit: even element in the low nibble).  Elements past n carry code 0,
 *   blocks entirely past n carry scale 0.  Pad bytes are never written.
 *   Lp = ceil(n/P) rounded up to a multiple of max(256, B).
 *
 * Layout of the error state
 *   STATE_INT8  : n int8 codes e (1 byte per element, as Table 1's text counts);
 *                 BLOCK_ABSMAX adds ceil(n/B) fp32 scales at byte offset roundup(n, 256).
 *   STATE_FP32 / STATE_FP32_Q8COMP : n fp32 values of the uncompressed error.
 *   STATE_NONE  : nothing.
 */
#ifndef LOCO_B200_H
#define LOCO_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOCO_OK = 0,
    LOCO_ERR_ARG = -1,          /* null pointer, value out of range, bad configuration       */
    LOCO_ERR_ALIGN = -2,        /* a device pointer is not 16-byte aligned                   */
    LOCO_ERR_SIZE = -3,         /* a buffer is smaller than the layout requires               */
    LOCO_ERR_CUDA = -4,         /* the CUDA runtime reported an error (no device, launch...)  */
    LOCO_ERR_UNSUPPORTED = -5   /* valid request that this build does not implement           */
} loco_status_t;

typedef enum { LOCO_F32 = 0, LOCO_BF16 = 1 } loco_dtype_t;

typedef enum {
    LOCO_SCALE_FIXED = 0,        /* Eq. 1: one global s (and s_e); only codes travel            */
    LOCO_SCALE_BLOCK_ABSMAX = 1  /* extension, not in the paper: fp32 scale amax/qmax per B      */
} loco_scale_mode_t;

typedef enum { LOCO_ROUND_NEAREST = 0, LOCO_ROUND_STOCHASTIC = 1 } loco_rounding_t;

typedef enum {
    LOCO_STATE_INT8 = 0,         /* the paper's 8-bit error e_k (Eq. 7); Eq. 5 uses dec(e_k)     */
    LOCO_STATE_FP32 = 1,         /* uncompressed error, the ablation without error compression   */
    LOCO_STATE_NONE = 2,         /* no error feedback: plain quantisation                        */
    LOCO_STATE_FP32_Q8COMP = 3   /* keep e~ in fp32, compensate with dec(comp(e~; s_e, 8); s_e),
                                    the form Lemma 1 is stated for; FIXED scale only            */
} loco_state_fmt_t;

/* Bits of the status word returned by loco_last_status(). */
#define LOCO_FLAG_NONFINITE 1u   /* some compensated gradient was NaN or +-Inf */

/* Algorithm 1's inputs (s, s_e, T_c, beta), Eq. 1's p, and the storage choices. */
typedef struct {
    int32_t bits;            /* p of Eq. 1 for the gradient codes: 2, 4 or 8 (the paper uses 4); 1 = the
                                sign code of "1-bit LoCo" (named in the paper's GPT-2 experiment, not
                                defined there): q = -1 if h < 0 else +1, one wire bit per element
                                (1 = negative), d = q / s, or q x (mean |h| of the block) with block
                                scales, that mean summed pairwise in fp32 over the block's positions */
    int32_t scale_mode;      /* loco_scale_mode_t                                                 */
    int32_t block_size;      /* B, BLOCK_ABSMAX only: power of two in [32, 4096].  A block of up to 512
                                elements lives in one warp of the streaming routine; a wider one is
                                spread over 2, 4 or 8 neighbouring warps that exchange their maxima
                                (with stochastic rounding: walked block by block instead, slower)  */
    float   s;               /* Eq. 1 / Eq. 3 scale, FIXED only (> 0, finite)                     */
    float   s_e;             /* Eq. 2 / Eq. 7 scale of the 8-bit error, FIXED only                */
    float   beta;            /* Eq. 5, in [0, 1]: weight of the NEW compression error             */
    int32_t reset_period;    /* T_c of Eq. 7: state := 0 after iteration k when k % T_c == 0;
                                0 = never                                                        */
    int32_t state_fmt;       /* loco_state_fmt_t                                                  */
    int32_t grad_dtype;      /* loco_dtype_t of the gradient handed to the send pass              */
    int32_t out_dtype;       /* loco_dtype_t of the averaged gradient the receive pass writes     */
    int32_t num_partitions;  /* P >= 1: parts of the all-to-all layout (Sec. 3.3)                 */
    int32_t collect_stats;   /* non-zero: count, during send, the gradient codes and the 8-bit error codes
                                whose nearest integer fell outside their range (second case of the
                                rounding lemma; the clamp of Eq. 7); costs a few instructions/element */
    float   clip;            /* > 0: clip every element of the local gradient to [-clip, clip] before
                                step 1 (the element-wise clipping of the Sky-MoE runs in the paper's
                                experiments; the paper states no threshold); 0 = off.  +-Inf becomes
                                +-clip, NaN stays NaN                                             */
    int32_t rounding;        /* loco_rounding_t: 0 = nearest integer as Eq. 1 states (the paper), 1 =
                                stochastic rounding, an extension: q = clamp(floor(h x s + u)) with
                                u = (b + 1/2) / 256, one fp32 add, where for element i of the bucket at
                                iteration k the byte b is byte (i mod 4), least significant first, of
                                output word ((i mod 16) / 4) of Philox4x32-10 with the 4-word counter
                                (floor(i/16) low 32 bits, floor(i/16) high 32 bits, k low, k high) and
                                the 2-word key (seed_lo, seed_hi): 16 elements share one Philox block,
                                256 equally likely values of u at the centres of their cells.  Not
                                available with bits = 1                                           */
    uint32_t seed_lo, seed_hi; /* key of that stream (ignored with rounding 0)                      */
} loco_config_t;

/* Per-bucket, per-worker handle: a host object holding the configuration, the bucket
 * length, the caller's state pointer and a 16-byte device status word. */
typedef struct loco_state loco_state_t;

/* ---- sizes (pure host arithmetic; 0 on a bad configuration or n == 0) ------------------ */
uint64_t loco_state_bytes(const loco_config_t *cfg, uint64_t n);        /* error state            */
uint64_t loco_packed_bytes(const loco_config_t *cfg, uint64_t n);       /* whole comm buffer      */
uint64_t loco_partition_bytes(const loco_config_t *cfg, uint64_t n);    /* stride of one part     */
uint64_t loco_partition_capacity(const loco_config_t *cfg, uint64_t n); /* Lp, padded elements    */
uint64_t loco_partition_elems(const loco_config_t *cfg, uint64_t n, int32_t j); /* valid elements */

/* LOCO_OK if the configuration is one this library accepts, else the error it would give. */
int loco_config_check(const loco_config_t *cfg);

/*
 * Create the handle for one bucket of n elements whose error state lives in the caller's
 * device buffer d_state (>= loco_state_bytes(); may be NULL for STATE_NONE) and zero-fill
 * that buffer asynchronously on `stream`: the error starts at zero (Eq. 5's initialisation).
 * Allocates the host handle and 16 bytes of device memory; the only allocating call.
 * Errors: ARG (null out/cfg, bad cfg), ALIGN, SIZE (d_state_bytes too small), CUDA.
 */
int loco_state_init(loco_state_t **out, const loco_config_t *cfg, uint64_t n,
                    void *d_state, uint64_t d_state_bytes, void *stream);

/* Zero the error state (the explicit reset of Algorithm 1) and the status word; asynchronous. */
int loco_state_reset(loco_state_t *st, void *stream);

/* Free the handle and its status word.  The caller's buffers are untouched. */
int loco_state_destroy(loco_state_t *st);

/*
 * Send pass for iteration `step_k` (the paper's 0-based k) -- Algorithm 1 steps 1-2:
 *     h = g + dec(e_k; s_e);  q = comp(h; s, p);  d = dec(q; s);
 *     e~_{k+1} = (1-beta) e~_k + beta (h - d);   e_{k+1} = 0 if k % T_c == 0 else comp(e~_{k+1}; s_e, 8)
 * in one fused pass: reads d_grad (n elements of grad_dtype) and the state, writes the
 * state in place and every code (and scale) byte of d_comm (>= loco_packed_bytes()).
 * d_grad is not modified.  One launch, no allocation, no synchronisation.
 * Errors: ARG (null, step_k < 0), ALIGN, CUDA.
 */
int loco_compensate_quantize_pack(loco_state_t *st, const void *d_grad, void *d_comm,
                                  int64_t step_k, void *stream);

/*
 * The same send pass with the all-to-all of Sec. 3.3 folded into its stores: part j of the
 * communication buffer (codes, then scales, loco_partition_bytes() in all) is written to
 * d_part_dst[j] instead of d_comm + j * loco_partition_bytes().
 *   d_part_dst  HOST array of num_partitions DEVICE pointers, 16-byte aligned each, every one
 *               with loco_partition_bytes() writable bytes.  A pointer may lie in this GPU's
 *               memory or in a peer GPU's memory that the caller has made accessible from this
 *               device (peer access enabled, or a mapped inter-process / symmetric-memory
 *               handle): worker r passes, as d_part_dst[j], slot r of worker j's receive area,
 *               and after every worker's pass has completed, worker j holds part j of all
 *               workers in its own memory and reduces it with loco_unpack_dequant_reduce
 *               (first_partition = j, partition_count = 1) from local pointers only.
 *               The table is copied into the launch; the array may be reused on return.
 * The kernel only stores to these addresses (plain global stores, no loads, no waits, no flags):
 * making "every worker's pass has completed" known to the readers is the caller's business (an
 * event, a barrier of its communication library, or stream order on one GPU).
 * num_partitions <= 64 here (UNSUPPORTED beyond).  One launch, no allocation, no synchronisation.
 * Errors: ARG (null table or entry, step_k < 0), ALIGN, UNSUPPORTED, CUDA.
 */
int loco_compensate_quantize_pack_scatter(loco_state_t *st, const void *d_grad,
                                          void *const *d_part_dst, int64_t step_k, void *stream);

/*
 * Receive pass -- Eq. 8: for `partition_count` consecutive parts starting at
 * `first_partition`, average the dequantised codes of `num_workers` workers (summed in
 * worker order in fp32, divided by N) and write out_dtype values to d_out.
 *   d_packed   HOST array of num_workers DEVICE pointers; d_packed[w] points at part
 *              `first_partition` inside worker w's communication buffer (the next parts
 *              follow at +loco_partition_bytes() each), 16-byte aligned.
 *   n          length of the whole bucket (fixes Lp and the valid length of each part).
 *   d_out      receives the valid elements of those parts contiguously, i.e. bucket
 *              elements [first*Lp, min((first+count)*Lp, n)).
 * 1 <= num_workers <= 64.  One launch, no allocation, no synchronisation.
 * Errors: ARG, ALIGN, UNSUPPORTED (num_workers > 64), CUDA.
 */
int loco_unpack_dequant_reduce(const loco_config_t *cfg, const void *const *d_packed,
                               int32_t num_workers, uint64_t n, int32_t first_partition,
                               int32_t partition_count, void *d_out, void *stream);

/*
 * Receive pass fused with the optimizer's update -- Algorithm 1 step 3 ("use g~_k to update theta_k") with the paper's
 * Adam-family equations and Adam's pre-conditioner:
 *     g      = Eq. 8 (as loco_unpack_dequant_reduce, kept in fp32)
 *     m      = (1 - beta1) m + beta1 g          beta1, beta2 weight the NEW term, as the paper writes them
 *     v      = (1 - beta2) v + beta2 g^2
 *     theta  = theta - lr / sqrt(v + delta) * m      no bias correction, delta inside the root (the printed form)
 * d_m, d_v, d_theta: fp32 DEVICE arrays holding the same elements d_out would (the valid elements of the parts,
 * contiguously), 16-byte aligned, updated in place.  d_grad_out may be NULL; otherwise it also receives g in out_dtype.
 * The averaged gradient then never travels through HBM: 24 B/element of optimizer state plus the packed codes.
 * One launch, no allocation, no synchronisation.  Errors: as loco_unpack_dequant_reduce, plus ARG for a null adam /
 * moment pointer or beta outside [0, 1], non-finite lr, negative delta.
 */
typedef struct {
    float lr;       /* eta */
    float beta1;    /* weight of the new gradient in the first moment  */
    float beta2;    /* weight of the new squared gradient in the second moment */
    float delta;    /* >= 0, added to v inside the square root */
} loco_adam_t;
int loco_unpack_dequant_reduce_adam(const loco_config_t *cfg, const void *const *d_packed, int32_t num_workers,
                                    uint64_t n, int32_t first_partition, int32_t partition_count,
                                    const loco_adam_t *adam, float *d_m, float *d_v, float *d_theta,
                                    void *d_grad_out, void *stream);

/* ---- several buckets per call -----------------------------------------------------------------
 * (No counterpart in the paper: a convenience of the library.)  Algorithm 1 is applied bucket by bucket, and a
 * bucket of the usual size is a kernel of 15-30 microseconds, a third of which is start-up and tail when the
 * kernels of a stream run strictly one after the other.  These two calls do what `count` single-bucket calls on
 * `stream` would do -- same arithmetic, same results, ordered like any other work on `stream` -- in ONE kernel
 * launch: the buckets are the third dimension of the grid and their table (pointers and sizes) travels in the
 * kernel's parameters, so nothing is allocated, nothing is synchronised and a captured launch carries its own copy
 * of the table.  The hardware hands the blocks of bucket 0, then bucket 1, ... to the SMs as places become free: no
 * bucket boundary drains the machine and the launch costs are paid once per call.
 *   - The buckets of one call must be independent of each other (distinct states and buffers), as they run
 *     concurrently.  All of them belong to the current device.
 *   - A launch holds up to 448 buckets on the send side (consecutive buckets of one configuration share a launch;
 *     a change of configuration starts a new one) and min(280, 2304 / num_workers) on the receive side; longer lists
 *     take several launches.
 *   - Every argument is checked before anything is launched: on an argument error nothing has been enqueued.
 * count = 0 does nothing.  Errors: as for the single-bucket calls, ARG for null arrays or entries.
 */

/* loco_compensate_quantize_pack for buckets i < count: states[i], d_grads[i], d_comms[i] (HOST arrays of count
 * entries each), all at iteration step_k. */
int loco_compensate_quantize_pack_multi(loco_state_t *const *states, const void *const *d_grads,
                                        void *const *d_comms, int32_t count, int64_t step_k, void *stream);

/* loco_unpack_dequant_reduce over all parts (first_partition 0, partition_count num_partitions) for buckets
 * i < count: d_packed[i] is bucket i's HOST array of num_workers DEVICE pointers, n[i] its length, d_outs[i] its
 * output (HOST arrays of count entries). */
int loco_unpack_dequant_reduce_multi(const loco_config_t *cfg, const void *const *const *d_packed,
                                     int32_t num_workers, const uint64_t *n, void *const *d_outs, int32_t count,
                                     void *stream);

/* ---- host-buffer variants ------------------------------------------------------------------
 * The same two passes for callers whose gradient and communication buffers live in HOST memory
 * (pinned memory makes the copies asynchronous).  Each call enqueues, on `stream`: the
 * host-to-device copy of its inputs into the caller's device workspace d_work, the kernel, and
 * the device-to-host copy of its result.  Nothing is allocated; the call returns without
 * synchronising, so the host buffers must stay untouched until the stream has drained.  The
 * error state stays on the device (it never leaves the worker, Sec. 3.1 of the paper).
 * Pad bytes of h_comm (see the wire layout) receive unspecified values.
 * Errors as for the device variants, plus SIZE when d_work_bytes is too small.
 */
uint64_t loco_send_host_workspace_bytes(const loco_config_t *cfg, uint64_t n);
uint64_t loco_reduce_host_workspace_bytes(const loco_config_t *cfg, uint64_t n, int32_t num_workers,
                                          int32_t partition_count);

/* Algorithm 1 steps 1-2 with h_grad (n elements) read from and h_comm (loco_packed_bytes())
 * written to host memory. */
int loco_compensate_quantize_pack_host(loco_state_t *st, const void *h_grad, void *h_comm,
                                       void *d_work, uint64_t d_work_bytes, int64_t step_k,
                                       void *stream);

/* Eq. 8 with h_packed[w] (HOST pointers to part `first_partition` of worker w's buffer,
 * partition_count * loco_partition_bytes() readable bytes each) and h_out in host memory. */
int loco_unpack_dequant_reduce_host(const loco_config_t *cfg, const void *const *h_packed,
                                    int32_t num_workers, uint64_t n, int32_t first_partition,
                                    int32_t partition_count, void *h_out, void *d_work,
                                    uint64_t d_work_bytes, void *stream);

/*
 * Receive pass for host buffers that needs no device memory from the caller and allocates none.
 * (No counterpart in the paper: this is a convenience of the library, not a step of the method.)
 *
 * Who needs it: code that has host buffers to reduce but no way to obtain device memory at the
 * point of the call -- a communication hook running while the training framework's caching
 * allocator already owns all of the GPU's free memory (a raw cudaMalloc then fails although the
 * framework "has" memory), a plug-in loaded into a process whose memory budget is fixed at
 * start-up, or a latency-critical loop in which cudaMalloc/cudaFree are banned because they
 * synchronise the whole device.  loco_unpack_dequant_reduce_host asks such a caller for a
 * workspace it cannot provide; this variant brings its own.
 *
 * Same arguments, result and errors as loco_unpack_dequant_reduce_host without d_work: the staging
 * area is a fixed array of LOCO_NOALLOC_SCRATCH_BYTES that is part of the library image, so every
 * GPU on which the library is used holds that much memory from the moment the library's device
 * code is loaded there until the process exits.  The call performs only asynchronous copies and one
 * kernel launch on `stream`; it calls no cudaMalloc, cudaFree or any other allocating routine.
 *   - Limit: loco_reduce_host_workspace_bytes(cfg, n, num_workers, partition_count) must not
 *     exceed LOCO_NOALLOC_SCRATCH_BYTES; a larger request returns LOCO_ERR_SIZE and enqueues
 *     nothing (e.g. 8 workers, 4-bit codes, bf16 output: up to about 690,000 elements per call).
 *     Reduce a longer part in several calls, one partition range at a time.
 *   - The first call on each device looks up the array's device address (a host-side query, done
 *     once per device with that device current).  Make that first call outside any stream
 *     capture; later calls only enqueue work.
 *   - All calls on one device share the one array and it keeps whatever the previous call left
 *     in it.  Nothing in it has to start at zero: every byte the kernel reads is first overwritten
 *     by this call's own host-to-device copies.  For the same reason two calls whose work overlaps
 *     on the GPU (different streams, or a second process thread) race on the array and corrupt
 *     each other's result: keep all calls on one device in one stream, or order them with events.
 *   - h_packed / h_out must stay untouched until `stream` has drained, as for the _host variant.
 */
#define LOCO_NOALLOC_SCRATCH_BYTES (4u * 1024u * 1024u)
int loco_unpack_dequant_reduce_host_noalloc(const loco_config_t *cfg, const void *const *h_packed,
                                            int32_t num_workers, uint64_t n, int32_t first_partition,
                                            int32_t partition_count, void *h_out, void *stream);

/*
 * Read the status words accumulated by the send passes of this handle since init/reset.
 * SYNCHRONISES `stream` (the one the passes ran on).  n_saturated counts gradient codes
 * whose nearest integer fell outside the p-bit range (second case of the rounding lemma);
 * n_saturated_state counts 8-bit error codes that Eq. 7's compressor clamped to [-128, 127]
 * (global s_e only: a block-scaled state cannot saturate; with STATE_FP32_Q8COMP the 8-bit
 * image is formed, and counted, when the error is next used).  Both stay 0 unless
 * collect_stats; the sign code has no range and counts nothing.  Any output pointer may be NULL.
 */
int loco_last_status(loco_state_t *st, uint32_t *flags, uint64_t *n_saturated, void *stream);
int loco_status_counters(loco_state_t *st, uint32_t *flags, uint64_t *n_saturated,
                         uint64_t *n_saturated_state, void *stream);

/*
 * Diagnostic for the block-scaled extension (no counterpart in the paper).  The send kernel forms a block's scale
 * amax/qmax and its inverse qmax/amax with short multiply-add sequences instead of the general division routine;
 * this call runs both sequences against the IEEE division for every positive finite fp32 amax and qmax in
 * {1, 7, 127} on the current device (about a second, synchronous, allocates and frees 16 bytes) and writes the number
 * of differing results: mismatches[0] for amax/qmax, mismatches[1] for qmax/amax.  Both must be 0.
 * Errors: ARG (null), CUDA.
 */
int loco_selfcheck_block_division(uint64_t *mismatches /* host, 2 elements */);

/* Human-readable name of a loco_status_t. */
const char *loco_status_string(int status);

/* Number of kernels this library has launched in the calling process (for accounting). */
uint64_t loco_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LOCO_B200_H */
