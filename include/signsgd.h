/*
 * signsgd.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path of
 * signSGD / Signum with majority vote (Algorithm 1 of "signSGD with Majority Vote is
 * Communication Efficient and Fault Tolerant").
 *
 * One iteration of Algorithm 1, for M workers whose gradients sit in one GPU's memory:
 *
 *   on worker m:   v_m <- (1 - beta) g_m + beta v_m          ("update momentum")
 *                  push sign(v_m)                             (1 bit per coordinate)
 *   on server:     V <- sum_m sign(v_m);  push sign(V)        ("majority vote")
 *   on every worker: x <- x - eta (sign(V) + lambda x)        ("update parameters")
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 * Sign code.   sign(z) is carried in one bit: bit = 1 means +1, and bit = 1 iff z >= 0 as a
 *              value (+0.0 and -0.0 give 1, NaN gives 0, +Inf gives 1, -Inf gives 0). The
 *              vote uses the same rule on the integer tally V, so a tie at even M votes +1.
 * Packing.     d coordinates occupy W = ceil(d/32) uint32 words (the 32x compression of the
 *              abstract). Coordinate 32 j + i is bit i of word j, bit 0 least significant.
 *              Bits at coordinates >= d are written as 0 in every output.
 * Arithmetic.  fp32, round to nearest even, every multiply and add rounded separately (no
 *              fused multiply-add), denormals kept. (1 - beta) is formed once in fp32 on the
 *              host. bf16 gradients are widened exactly to fp32. With weight_decay == 0 the
 *              update is x <- x - (+-lr); otherwise x <- x - lr * (s + weight_decay * x) with
 *              s = +-1, evaluated in that order.
 * Adversaries. flip_mask bit m set makes worker m an inverting adversary (Definition 1 (iii),
 *              Section 4.2): its sign bits are complemented before the vote. Bits >= M must be 0.
 * Memory.      Every data buffer is caller-owned DEVICE memory unless a parameter is documented
 *              as host memory. Arrays of pointers (grads, momenta, packed) are HOST arrays of M
 *              device pointers; they are read during the call and may be freed after it returns.
 *              The library allocates no device memory and never frees or keeps a caller pointer.
 *              No buffer that a call writes (momenta, param, packed or vote words, staging) may
 *              overlap any other buffer of the call; momentum and param are updated in place.
 *              Read-only inputs may alias one another (two workers with the same gradient).
 * Alignment.   Word buffers: 4 bytes. Gradients: their element size. fp32 state: 4 bytes. When
 *              every gradient, momentum and parameter pointer of a call is 16-byte aligned
 *              (8-byte for bf16 gradients) the 128-bit vectorised kernels run; otherwise a
 *              scalar-load kernel with identical results runs. Misalignment below the element
 *              size is SS_ERR_MISALIGNED.
 * Streams.     cuda_stream is a cudaStream_t (NULL = the legacy default stream). Calls enqueue
 *              work on it and return without synchronising. The device that is current when
 *              the call is made is used.
 * Limits.      1 <= M <= SS_MAX_WORKERS. 0 <= d <= SS_MAX_COORDS; d == 0 is a no-op that returns
 *              SS_OK, a d beyond the limit is SS_ERR_INVALID_ARG.
 * Errors.      Every function returns an int status: SS_OK (0) or a negative SS_ERR_* code;
 *              nothing is thrown across the boundary. Every argument of a call is checked before
 *              its first copy or kernel is enqueued: on an argument error nothing is enqueued.
 *              SS_ERR_CUDA reports a failed launch or runtime call; ss_last_cuda_error() gives
 *              its cudaError_t value for the calling thread.
 */
#ifndef SIGNSGD_H_
#define SIGNSGD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SS_MAX_WORKERS 64
#define SS_MAX_COORDS ((int64_t)1 << 40) /* keeps every byte count formed from d inside 64 bits */

typedef enum { SS_F32 = 0, SS_BF16 = 1 } ss_dtype;

enum {
    SS_OK = 0,
    SS_ERR_INVALID_ARG = -1,  /* NULL pointer, M or d out of range, flip_mask bit >= M, bad dtype */
    SS_ERR_MISALIGNED = -2,   /* pointer not aligned to its element size */
    SS_ERR_UNSUPPORTED = -3,  /* valid request that this build cannot serve */
    SS_ERR_CUDA = -4          /* CUDA runtime or launch failure */
};

/* ceil(d/32): words needed for d sign bits (abstract: 32x less than fp32). -1 if d < 0. */
int64_t ss_packed_words(int64_t d);

/* Static, human-readable name of a status code. Never NULL. */
const char* ss_status_string(int status);

/* cudaError_t of the last SS_ERR_CUDA returned on the calling thread (0 if none). */
int ss_last_cuda_error(void);

/*
 * Sign compression of one worker's gradient (Algorithm 1, "push sign(.)" with beta = 0;
 * Section 4: bit-packing a sign tensor to one bit per element).
 *   grad       in   d elements of dtype dt
 *   out_words  out  ceil(d/32) words
 */
int ss_sign_pack(const void* grad, ss_dtype dt, int64_t d, uint32_t* out_words, void* cuda_stream);

/*
 * Server side of Algorithm 1: V = sum_m sign(v_m), result sign(V), on packed words.
 *   packed      in   HOST array of M device pointers, each to ceil(d/32) words
 *   vote_words  out  ceil(d/32) words; must not overlap any input
 * Bits of the inputs at coordinates >= d are ignored.
 */
int ss_majority_vote(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                     uint32_t* vote_words, void* cuda_stream);

/*
 * The tally of Algorithm 1's server line itself, V = sum_m sign(v_m), one int8 per coordinate
 * (-M <= V <= M, same parity as M). A diagnostic, not a step of the iteration: it gives the
 * margin of every vote (V = 2 Z - M with Z the count of +1 votes that the proof of Theorem 2
 * bounds), e.g. to compare measured vote failures with that theorem's bound.
 *   packed     in   HOST array of M device pointers, each to ceil(d/32) words
 *   tally_out  out  d int8 (any alignment)
 * sign of the tally under the header's sign rule (V >= 0 -> +1) is what ss_majority_vote packs.
 */
int ss_vote_tally(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                  int8_t* tally_out, void* cuda_stream);

/*
 * Worker side of Algorithm 1 with momentum: v <- (1 - beta) g + beta v in place, then sign(v)
 * packed. beta = 0 gives the packed sign of g (and v = g).
 *   grad       in      d elements of dtype dt
 *   momentum   in/out  d fp32
 *   out_words  out     ceil(d/32) words
 */
int ss_signum_update(const void* grad, ss_dtype dt, float* momentum, float beta, int64_t d,
                     uint32_t* out_words, void* cuda_stream);

/*
 * ss_signum_update that also performs the first push of Algorithm 1 ("push sign(v_m) to
 * server"): each packed word is stored to every one of n_dests buffers by the kernel that
 * produces it. With one worker per GPU the destinations are the slot reserved for this worker
 * in every worker's receive buffer -- its own and its peers', mapped into this process with
 * peer access enabled -- so that the all-gather of packed words needs no separate collective.
 * Only plain stores go to a peer; nothing is read from one, whatever the alignment of grad and
 * momentum (off the 16-byte grid a scalar-load kernel runs and stores to every destination
 * itself). The caller orders the exchange:
 * every worker's call must have completed (stream synchronisation plus a barrier across the
 * workers) before any worker's ss_vote_apply reads its receive buffer, and the next step's push
 * must not start before those reads have finished.
 *   grad, momentum, beta, d   as ss_signum_update
 *   dests    out  HOST array of n_dests device pointers, each to ceil(d/32) words, disjoint
 *   n_dests  1 .. SS_MAX_WORKERS
 * Every destination receives exactly what ss_signum_update would write.
 */
int ss_signum_update_push(const void* grad, ss_dtype dt, float* momentum, float beta, int64_t d,
                          uint32_t* const* dests, int n_dests, void* cuda_stream);

/*
 * Algorithm 1, "update parameters": x <- x - lr (sign(V) + weight_decay x) from the packed vote.
 *   param       in/out  d fp32
 *   vote_words  in      ceil(d/32) words
 */
int ss_apply_vote(float* param, const uint32_t* vote_words, int64_t d, float lr,
                  float weight_decay, void* cuda_stream);

/*
 * ss_majority_vote and ss_apply_vote in one pass: what every worker does once the M packed
 * sign vectors are in its memory (its own, and the others' after the exchange of Algorithm 1's
 * two push steps). The tally never leaves the registers; the packed vote is written only if asked.
 *   packed          in      HOST array of M device pointers, each to ceil(d/32) words
 *   param           in/out  d fp32
 *   vote_words_out  out     ceil(d/32) words, or NULL
 * Results are identical to ss_majority_vote followed by ss_apply_vote.
 */
int ss_vote_apply(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask, float* param,
                  float lr, float weight_decay, uint32_t* vote_words_out, void* cuda_stream);

/*
 * Flag-ordered exchange for one worker per GPU (Algorithm 1's "push sign(v_m) to server" and
 * "push sign(V) to each worker", with every worker acting as its own server). Each worker owns a
 * flag array of SS_MAX_WORKERS uint32 words in its memory, mapped into its peers. A step with
 * epoch e (1, 2, 3, ... ; serial-number comparison, so wrap-around is harmless):
 *   1. ss_signum_update_push stores this worker's packed signs into its slot of every worker's
 *      receive buffer;
 *   2. ss_flags_signal, on the same stream, writes e into word `index` (= this worker's rank) of
 *      every worker's flag array: it runs once the push kernel has completed, so a peer that sees
 *      the flag sees the words;
 *   3. ss_flags_wait polls this worker's OWN flag array until words 0 .. M-1 have all reached e,
 *      for at most timeout_ns, and writes 0 or (1 + lowest missing worker) to *status_dev;
 *   4. ss_vote_apply_guarded votes and updates unless *status_dev is non-zero, in which case the
 *      whole launch does nothing: parameters are updated for all coordinates or for none.
 * Two receive buffers used alternately (by the parity of e) make a second synchronisation
 * unnecessary: a worker reaches its push of step e+2 only after its wait of step e+1, i.e. after
 * every peer has finished its update of step e, which is what read the buffer now overwritten.
 * Only plain stores go to a peer; nothing is read from one; the only wait is the bounded one of
 * step 3, on local memory. The host decides what a time-out means: read *status_dev after
 * synchronising the stream (a worker left, or is late), before trusting the step.
 */
#define SS_FLAGS_MAX_TIMEOUT_NS 2000000000ull /* 2 s: the longest wait ss_flags_wait accepts */

/*   flags    in   HOST array of n_flags device pointers, each to a flag array (4-byte aligned)
 *   index    in   word to write in each array, 0 .. SS_MAX_WORKERS-1 (the signalling worker's rank)
 *   epoch    in   value to write */
int ss_flags_signal(uint32_t* const* flags, int n_flags, int index, uint32_t epoch, void* cuda_stream);

/*   flags_local  in   this worker's own flag array (device memory of the current device)
 *   M            in   workers to wait for: words 0 .. M-1
 *   timeout_ns   in   at most SS_FLAGS_MAX_TIMEOUT_NS, else SS_ERR_INVALID_ARG
 *   status_dev   out  one uint32 in device memory: 0, or 1 + the lowest worker that did not arrive
 * One block of SS_MAX_WORKERS threads; it always terminates (time limit, plus an iteration limit
 * as a backstop) and leaves the context usable. */
int ss_flags_wait(const uint32_t* flags_local, int M, uint32_t epoch, uint64_t timeout_ns,
                  uint32_t* status_dev, void* cuda_stream);

/* ss_flags_signal followed by ss_flags_wait in one launch (steps 2 and 3 above back to back). */
int ss_flags_signal_wait(uint32_t* const* flags, int n_flags, int index, const uint32_t* flags_local, int M,
                         uint32_t epoch, uint64_t timeout_ns, uint32_t* status_dev, void* cuda_stream);

/* ss_vote_apply that does nothing at all when the word at skip_if_nonzero_dev (device memory,
 * written by an earlier call on the same stream, e.g. ss_flags_wait) is not zero. */
int ss_vote_apply_guarded(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                          float* param, float lr, float weight_decay, uint32_t* vote_words_out,
                          const uint32_t* skip_if_nonzero_dev, void* cuda_stream);

/*
 * One whole iteration of Algorithm 1 in a single pass over memory: momentum, sign, vote and
 * parameter update per coordinate, the packed signs never leaving the chip.
 *   grads           in      HOST array of M device pointers, d elements of dt each
 *   momenta         in/out  HOST array of M device pointers to d fp32 each, or NULL for
 *                           signSGD (no momentum state; beta is ignored)
 *   param           in/out  d fp32
 *   vote_words_out  out     ceil(d/32) words, or NULL if the packed vote is not wanted
 * Results are identical, bit for bit, to ss_signum_update (or ss_sign_pack) per worker followed
 * by ss_majority_vote and ss_apply_vote.
 */
int ss_fused_step(const void* const* grads, ss_dtype dt, float* const* momenta, int M, int64_t d,
                  float beta, uint64_t flip_mask, float* param, float lr, float weight_decay,
                  uint32_t* vote_words_out, void* cuda_stream);

/*
 * Tensor fusion (Section 4 reports that merging small tensors into one buffer before
 * compression saved compression and communication cost). A model's parameter tensors are laid
 * out back to back in one flat vector of d coordinates, so that one
 * call packs, votes and updates all of them; the gradient and momentum buffers use the same
 * layout. Each tensor keeps its own learning rate and weight decay (Algorithm 1's eta and
 * lambda) through a table of segments sorted by first coordinate: entry k covers coordinates
 * [begin_k, begin_{k+1}), the last entry runs to d, entry 0 begins at 0. Tensors may start at
 * any coordinate (no padding to word boundaries is needed); an entry whose range is empty is
 * allowed and ignored.
 */
typedef struct ss_segment {
    int64_t begin;       /* first coordinate of the tensor in the flat vector */
    float lr;            /* eta for this tensor */
    float weight_decay;  /* lambda for this tensor */
} ss_segment;

/*
 * Validates a segment table and enqueues its copy to device memory.
 *   host_segments  in   HOST array of n_segments entries (may be freed after the call returns
 *                       only if it is pageable memory; pinned memory must outlive the copy)
 *   segments_dev   out  caller-owned DEVICE array of n_segments entries, 8-byte aligned
 * SS_ERR_INVALID_ARG if n_segments < 1, begin[0] != 0, the begins decrease, or a begin exceeds d.
 */
int ss_segments_upload(const ss_segment* host_segments, int n_segments, int64_t d,
                       ss_segment* segments_dev, void* cuda_stream);

/*
 * ss_fused_step over a fused flat vector with per-tensor eta and lambda: coordinate c is
 * updated as x <- x - lr_k (sign(V) + weight_decay_k x) with k the segment that holds c. The
 * momentum, the signs and the vote do not depend on the table. The result equals one
 * ss_fused_step per tensor on that tensor's slices.
 *   segments_dev  in  DEVICE table written by ss_segments_upload (not validated again here)
 * Other arguments as ss_fused_step.
 */
int ss_fused_step_segments(const void* const* grads, ss_dtype dt, float* const* momenta, int M,
                           int64_t d, float beta, uint64_t flip_mask, float* param,
                           const ss_segment* segments_dev, int n_segments,
                           uint32_t* vote_words_out, void* cuda_stream);

/* ss_vote_apply with per-tensor eta and lambda from a device segment table. */
int ss_vote_apply_segments(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                           float* param, const ss_segment* segments_dev, int n_segments,
                           uint32_t* vote_words_out, void* cuda_stream);

/* ss_vote_apply_guarded over a fused vector of tensors: ss_vote_apply_segments that does nothing
 * at all when the word at skip_if_nonzero_dev is not zero. */
int ss_vote_apply_guarded_segments(const uint32_t* const* packed, int M, int64_t d, uint64_t flip_mask,
                                   float* param, const ss_segment* segments_dev, int n_segments,
                                   uint32_t* vote_words_out, const uint32_t* skip_if_nonzero_dev,
                                   void* cuda_stream);

/* ss_apply_vote with per-tensor eta and lambda from a device segment table. */
int ss_apply_vote_segments(float* param, const uint32_t* vote_words, int64_t d,
                           const ss_segment* segments_dev, int n_segments, void* cuda_stream);

/*
 * ss_fused_step for gradients that start in HOST memory (the end-to-end form: what a step costs
 * when the M gradients arrive over PCIe and the packed vote goes back, as the d-bit messages of
 * Algorithm 1's push steps do).
 *   host_grads      in      HOST array of M HOST pointers (pinned memory recommended), d elements each
 *   staging         scratch HOST array of M device pointers, d elements of dt each; overwritten
 *   momenta, param, M, d, beta, flip_mask, lr, weight_decay: as ss_fused_step (device memory)
 *   vote_words_dev  out     ceil(d/32) words of device memory (required)
 *   host_vote_out   out     ceil(d/32) words of HOST memory, or NULL to skip the copy back
 * Enqueues M host-to-device copies, the fused kernel and one device-to-host copy on cuda_stream
 * and returns; host_grads and host_vote_out must stay valid until the stream has drained.
 */
int ss_fused_step_host(const void* const* host_grads, ss_dtype dt, void* const* staging,
                       float* const* momenta, int M, int64_t d, float beta, uint64_t flip_mask,
                       float* param, float lr, float weight_decay, uint32_t* vote_words_dev,
                       uint32_t* host_vote_out, void* cuda_stream);

/*
 * ss_fused_step_host without any device memory from the caller or from an allocator.
 * (The paper has no counterpart to this entry point; it exists for deployment.)
 *
 * Who needs it: a host program that cannot call cudaMalloc at the point where it wants a step.
 * Typical cases are a process that has handed the whole device to a framework's caching
 * allocator, so that a raw allocation fails or eats into that pool; a plug-in or a control loop
 * whose rules forbid allocating after start-up, because cudaMalloc takes a device-wide lock and
 * can stall every stream; and a sandboxed component that is given streams and buffers but not
 * the right to create allocations. Such a caller cannot provide ss_fused_step_host's `staging`
 * buffers, so here the staging area is a fixed array of SS_STATIC_STAGING_BYTES that is part of
 * the library's device image: every GPU on which the library's CUDA module is loaded holds that
 * much memory until the process exits.
 *
 *   host_grads      in      HOST array of M HOST pointers (pinned memory recommended), d elements each
 *   momenta, param, vote_words_dev: caller-owned DEVICE memory as in ss_fused_step_host
 *   host_vote_out   out     ceil(d/32) words of HOST memory, or NULL
 *
 * Limit: M * round_up(d * element size, 256) <= SS_STATIC_STAGING_BYTES. A larger request returns
 * SS_ERR_UNSUPPORTED and enqueues nothing; split the coordinates into ranges and call once per range.
 * First call on a device: it looks up the device address of the staging array (once per device,
 * with that device current) and keeps it. With lazy module loading, the CUDA default, that
 * look-up is also what loads this part of the library onto the device, so it is then that the
 * SS_STATIC_STAGING_BYTES are reserved; if the device has no room left for them the call returns
 * SS_ERR_CUDA. Make that first call during start-up, before the device's memory is handed away
 * and outside any stream capture. Every later call on that device performs no cudaMalloc,
 * cudaFree or other allocating call and leaves the amount of free device memory unchanged.
 * Sharing: all calls on a device use the same staging array, and it keeps whatever the last call
 * left there. Every byte a call reads is first overwritten by that call's own copies, so nothing
 * needs clearing; but two calls whose work overlaps on the GPU (different streams, no dependency)
 * race on the array. Issue them on one stream or order them with events.
 * Results are identical to ss_fused_step_host. Errors as for ss_fused_step_host.
 */
#define SS_STATIC_STAGING_BYTES (64u << 20)
int ss_fused_step_host_static(const void* const* host_grads, ss_dtype dt, float* const* momenta,
                              int M, int64_t d, float beta, uint64_t flip_mask, float* param,
                              float lr, float weight_decay, uint32_t* vote_words_dev,
                              uint32_t* host_vote_out, void* cuda_stream);

/*
 * The comparison codec of Appendix B: 1-bit max-norm QSGD, the ternary quantiser against which
 * the paper sets the bits per iteration of majority vote. Coordinate g_i becomes sign(g_i) with
 * probability |g_i| / ||g||_inf and 0 otherwise; the code takes two bits per coordinate (Appendix
 * B: 2d bits always store d numbers in {0, +-1}), 16 coordinates per uint32 word: coordinate
 * 16 j + i sits at bits 2i, 2i+1 of word j as 0 (zero), 1 (+1) or 3 (-1); bits at coordinates
 * >= d are 0. A comparison system, not a step of Algorithm 1.
 *
 * The draws come from the Philox4x32-10 counter-based generator evaluated inside the kernel:
 * the block with counter (q, 0, 0) [q split into two 32-bit words] and key `seed` gives the four
 * 32-bit words r of coordinates 4q .. 4q+3. With u = (r >> 9) * 2^-23, a coordinate is kept iff
 * RN(u * ||g||_inf) < |g_i| in fp32: the maximum is always kept, zeros and NaNs never; nothing is
 * kept when ||g||_inf is 0 or Inf. The same (gradient, max-norm, seed) always gives the same code.
 */

/* ceil(d/16): words of a ternary code. -1 if d < 0. */
int64_t ss_ternary_words(int64_t d);

/*
 * ||g||_inf = max |g_i| over the elements that are not NaN (0 for d == 0), as fp32.
 *   grad        in   d elements of dtype dt
 *   absmax_dev  out  one fp32 in DEVICE memory (zeroed, then raised by the kernel)
 */
int ss_absmax(const void* grad, ss_dtype dt, int64_t d, float* absmax_dev, void* cuda_stream);

/*
 * Ternary code of one worker's gradient.
 *   grad        in   d elements of dtype dt
 *   absmax_dev  in   DEVICE pointer to ||g||_inf as written by ss_absmax on the same stream
 *   seed        in   key of the generator; use a fresh one per worker and per step
 *   out_codes   out  ceil(d/16) words
 */
int ss_ternary_pack(const void* grad, ss_dtype dt, int64_t d, const float* absmax_dev, uint64_t seed,
                    uint32_t* out_codes, void* cuda_stream);

/*
 * Decoder: out_i = scale * q_i with q_i in {0, +-1} read from the code (QSGD's estimate of the
 * gradient uses scale = ||g||_inf; its expectation over the draws is g).
 *   codes      in   ceil(d/16) words
 *   scale_dev  in   DEVICE pointer to one fp32
 *   out        out  d fp32
 */
int ss_ternary_unpack(const uint32_t* codes, int64_t d, const float* scale_dev, float* out,
                      void* cuda_stream);

/*
 * Launch-shape override for benchmarking sweeps: not part of the method, and the one piece of
 * process-wide state in the library (three integers, written and read atomically; a launch uses the
 * values it finds when it is made, so change them only between calls whose shape matters).
 *   key: "threads" (block size: a multiple of 32 in [64, 256], the bound the kernels are compiled
 *        for; 0 = default, 256) or
 *        "blocks_per_sm" (0 = one block per tile, the default; n > 0 = a persistent grid of
 *        n blocks per SM that strides over the tiles; at most 4096) or
 *        "plain_loads_from_mib" (ss_fused_step without momentum: the gradient bytes of a call, in
 *        MiB, from which the gradients are fetched with plain loads instead of evict-first ones;
 *        0 = default, 1536; 1 = practically always; at most 2^20 = never). Results do not depend
 *        on any of the three.
 * Returns SS_ERR_INVALID_ARG for an unknown key or a value out of range.
 */
int ss_set_launch_option(const char* key, int value);

#ifdef __cplusplus
}
#endif

#endif /* SIGNSGD_H_ */
