/*
 * pop.h - C ABI of the POP (partition-guided online pruning) hot path for one
 * SwiGLU FFN / MoE expert block on an NVIDIA B200 (sm_100a).
 *
 * The paper states the method in two stages (Sec. 3.3, Sec. 3.4):
 *   prefill : score every intermediate channel from the whole prompt (Eq. 3) and split the
 *             channels into Retained / Candidate / Pruned regions around the pruning
 *             threshold;
 *   decode  : per step, run the block's first projections over Retained + Candidate only,
 *             score the Candidate channels from this step's activations, switch on the k
 *             best of them, and finish the block over Retained + selected channels.
 * The paper defines no API; the two main calls below follow that statement of the problem.
 *
 * Conventions
 *   d  hidden size, N intermediate size (the N prunable channels), L prompt tokens with the
 *   batch folded in, B decode batch.  Wg, Wu are [N, d] row-major (row i = channel i); Wd is
 *   [d, N] row-major (column i = channel i).  f(x) = silu(Wg x) * (Wu x).
 *   All data pointers are DEVICE pointers unless a parameter is named h_* (host).
 *   Every function returns an int status (POP_OK == 0, errors negative).  Nothing throws,
 *   aborts or synchronises the device unless stated; device work is enqueued on the
 *   cudaStream_t passed as `cuda_stream` (NULL = the legacy default stream).
 *   A partition is used by one stream at a time.
 */
#ifndef POP_H_
#define POP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define POP_OK                 0
#define POP_ERR_INVALID_ARG   -1   /* null pointer, size out of range, ratios invalid, k > n_cand ... */
#define POP_ERR_UNSUPPORTED   -2   /* dtype / shape / batch outside what the kernels handle          */
#define POP_ERR_ALLOC         -3   /* device or host allocation failed                                */
#define POP_ERR_CUDA          -4   /* a CUDA runtime call failed; see pop_last_cuda_error()           */
#define POP_ERR_TIMEOUT       -5   /* a bounded device-side wait expired (reported by pop_partition_check) */

#define POP_MAX_BATCH          8   /* largest decode batch B a partition's scratch is sized for       */
#define POP_NOALLOC_MAX_N  32768   /* largest N pop_prefill_scores_noalloc accepts                    */

typedef enum { POP_F32 = 0, POP_BF16 = 1 } pop_dtype_t;

/* Fractions of the N channels put into each region; each >= 0, candidate + pruned <= 1. */
typedef struct { double retained, candidate, pruned; } pop_ratios_t;

/* Opaque, library-owned: repacked weights, region indices, prefill scores, decode scratch. */
typedef struct pop_partition pop_partition_t;

/* Opaque, library-owned: what a prefill needs from one weight set alone (see pop_weights_prepare). */
typedef struct pop_weights pop_weights_t;

/*
 * Process-wide settings (host only; the paper has no counterpart: they choose among the library's kernels).
 *   decode_kernel   which decode kernel family serves partitions created from now on.  POP_DECODE_AUTO: the
 *                   streaming kernel for bf16 partitions with d in {2048, 4096, 5120} and at most 3072
 *                   candidates, the fused persistent kernel or, where that does not fit, the multi-kernel
 *                   path for everything else; POP_DECODE_FUSED / POP_DECODE_SIMPLE force those two.
 *   launch_mode     how every later step of the streaming kernel is launched.  Its CTAs wait on one
 *                   another's results.  POP_LAUNCH_PDL (default): plain launch with programmatic stream
 *                   serialization, which hides the launch latency between the steps of a decode loop but
 *                   relies on the device being free enough for all CTAs to be resident at once: use it
 *                   when the decode stream has the device to itself.  POP_LAUNCH_COOPERATIVE: the driver
 *                   places all CTAs at once or fails the launch (about 2.4 us per step slower): use it
 *                   when other streams keep SMs busy.  POP_LAUNCH_PLAIN: plain launch.
 *   wait_budget_us  how long any single device-side wait of a decode step may last before the step gives
 *                   up (default 50000).  A step that gives up leaves y undefined and is reported by
 *                   pop_partition_check as POP_ERR_TIMEOUT; it never hangs.
 *   slab_cache_bytes  device memory of destroyed partitions that the library keeps for the next partition
 *                   of the same size (default 1 GiB; 0 = keep nothing, and releases what is held).
 * The temporaries of a prefill come from a stream-ordered memory pool of the library's own (one per device)
 * that keeps what it has allocated while the device is idle: a few MB, tens of MB after
 * pop_prefill_partition_with_output.
 * pop_release_cached_memory() gives all of that memory (cached slabs and the pool's unused memory) back to
 * the driver at once (it calls cudaFree, which synchronises the device).
 */
typedef enum { POP_DECODE_AUTO = 0, POP_DECODE_FUSED = 1, POP_DECODE_SIMPLE = 2 } pop_decode_kernel_t;
typedef enum { POP_LAUNCH_PDL = 0, POP_LAUNCH_COOPERATIVE = 1, POP_LAUNCH_PLAIN = 2 } pop_launch_mode_t;
typedef struct {
    pop_decode_kernel_t decode_kernel;
    pop_launch_mode_t launch_mode;
    unsigned int wait_budget_us;
    unsigned long long slab_cache_bytes;
} pop_config_t;
int pop_get_config(pop_config_t* out);
int pop_set_config(const pop_config_t* in);
int pop_release_cached_memory(void);

/* ---- library information (host only) ------------------------------------------------------- */
const char* pop_version(void);
const char* pop_status_string(int status);
/* Text of the last CUDA runtime error seen by this thread inside the library ("" if none). */
const char* pop_last_cuda_error(void);

/* Number of CUDA kernels this library has launched in this process so far (kernels recorded into
 * a CUDA graph during stream capture count once, at capture). */
unsigned long long pop_kernel_launch_count(void);

/*
 * Region sizes for N channels (Sec. 3.3: thresholds at the (r - delta) and (r + delta) quantiles;
 * taken by rank so that the sizes are exact):
 *   n_pruned = floor(pruned * N + 1e-9), n_cand = floor(candidate * N + 1e-9),
 *   n_ret = N - n_cand - n_pruned, k_default = floor(n_cand / 2).
 * Host only. Any output pointer may be NULL.  POP_ERR_INVALID_ARG on bad ratios or N <= 0.
 */
int pop_region_sizes(int N, pop_ratios_t ratios, int* n_ret, int* n_cand, int* n_pruned, int* k_default);

/*
 * Prefilling stage (Sec. 3.3 "Prefilling Stage"; score = Eq. 3 of Sec. 3.4).
 *   X [L, d], Wg [N, d], Wu [N, d], Wd [d, N]: row-major device arrays of `dtype`, read-only,
 *   owned by the caller; they may be freed once the stream has passed this call (the
 *   partition keeps its own repacked copy of the live rows).
 * Computes, on `cuda_stream`:
 *   H[t, i] = silu(Wg[i].X[t]) * (Wu[i].X[t]);  s_i = sqrt(sum_t H[t,i]^2);
 *   I_i = s_i * ||Wd[:, i]||_2   (Eq. 3 with W = the down projection, whose input channel i
 *   is intermediate channel i);
 *   ranks channels by (I_i descending, i ascending): the first n_ret are Retained, the next
 *   n_cand Candidate, the rest Pruned (sizes as pop_region_sizes);
 *   repacks Wg/Wu rows and Wd columns of Retained then Candidate channels contiguously.
 * The ranking is the one exact (fp64) scores give: see pop_partition_scores.  For bf16 the dense
 * contraction runs on the tensor cores (tcgen05, operands through TMA) when d >= 64.
 * *out receives a new partition (destroy it with pop_partition_destroy).  Allocates device memory
 * (about (n_ret + n_cand) * 3 * d elements, plus stream-ordered temporaries).
 * Requirements: d * sizeof(element) a multiple of 16; pointers 16-byte aligned; L >= 1.
 * Errors: POP_ERR_INVALID_ARG, POP_ERR_UNSUPPORTED, POP_ERR_ALLOC, POP_ERR_CUDA.
 */
int pop_prefill_partition(const void* X, int L, int d,
                          const void* Wg, const void* Wu, const void* Wd, int N,
                          pop_dtype_t dtype, pop_ratios_t ratios,
                          void* cuda_stream, pop_partition_t** out);

/*
 * The input-independent part of the prefilling stage, once per weight set instead of once per prompt
 * (Eq. 3 factors into an activation norm and the weight norm ||Wd[:, i]||_2, which does not depend on
 * the prompt): the column norms of Wd and, for the tensor-core scoring pass, the row norms of Wg and Wu
 * (they enter its error bounds) and the TMA descriptors of Wg and Wu.
 *   Wg, Wu [N, d], Wd [d, N] as for pop_prefill_partition.  The object does NOT copy the weights: the
 *   caller keeps them alive, at the same addresses and unchanged, until pop_weights_destroy.
 * Enqueues its kernels on `cuda_stream`; later prefills that use the object must be ordered after them
 * (same stream, or an event).  Allocates a few N-element device arrays.
 * pop_prefill_partition_prepared(X, L, w, ...) is pop_prefill_partition(X, L, d, Wg, Wu, Wd, N, dtype, ...)
 * with those statistics taken from `w`: same results, bit for bit.  The current device must be the one
 * `w` was prepared on (POP_ERR_INVALID_ARG otherwise).  pop_weights_destroy: the caller has synchronised
 * the work that used the object.
 */
int pop_weights_prepare(const void* Wg, const void* Wu, const void* Wd, int N, int d, pop_dtype_t dtype,
                        void* cuda_stream, pop_weights_t** out);
int pop_prefill_partition_prepared(const void* X, int L, const pop_weights_t* w, pop_ratios_t ratios,
                                   void* cuda_stream, pop_partition_t** out);

/*
 * Partial probing (Sec. 3.4 names "partial probing prompt activations" as the source of the prefill statistics
 * without defining the subset; here: every token_stride-th prompt token, rows 0, token_stride, 2 token_stride, ...
 * of X).  pop_prefill_partition_probe(X, L, s, w, ...) gives exactly the partition that
 * pop_prefill_partition_prepared gives for those ceil(L / s) rows alone (s = 1: the whole prompt), at a cost that
 * falls with s: the rows are gathered on the device into a temporary and scored from there.  X [L, d] device,
 * row-major, 16-byte aligned; token_stride >= 1 (POP_ERR_INVALID_ARG otherwise).  Everything else as
 * pop_prefill_partition_prepared.
 */
int pop_prefill_partition_probe(const void* X, int L, int token_stride, const pop_weights_t* w, pop_ratios_t ratios,
                                void* cuda_stream, pop_partition_t** out);
int pop_weights_destroy(pop_weights_t* w);

/*
 * The prefilling stage together with the prompt's own block output "under the resulting pruning structure"
 * (Sec. 3.4).  The paper does not say which channels that structure keeps for the prompt; the reading taken
 * here is the mask a static variant would reuse at every step (Sec. 4.6, Variant (1)): Retained plus the
 * k_candidate Candidates with the largest PREFILL score (ties by lower channel id), i.e. the n_ret + k_candidate
 * best channels by I_i.
 *   Y [L, d]: device array of the weights' dtype, caller-owned:
 *   Y[t] = sum over those channels i of Wd[:, i] * silu(Wg[i].X[t]) * (Wu[i].X[t]).
 * Everything else as pop_prefill_partition_prepared.  The intermediate activations of the scoring pass (fp32
 * accumulation on the tensor cores) are kept as bf16 pairs (16 significant bits) and contracted with Wd by a second tensor-core pass (fp32
 * accumulation, one rounding to bf16 at the end); the mask itself is decided on exact scores like the regions.
 * bf16 with d >= 64 and N a multiple of 8 only (POP_ERR_UNSUPPORTED otherwise); 0 <= k_candidate <= n_cand.
 */
int pop_prefill_partition_with_output(const void* X, int L, const pop_weights_t* w, pop_ratios_t ratios,
                                      int k_candidate, void* Y, void* cuda_stream, pop_partition_t** out);

/*
 * Build a partition from caller-chosen regions instead of prefill scores (the regions of
 * Sec. 3.3 given explicitly).  h_ret [n_ret] and h_cand [n_cand] are HOST arrays of channel
 * ids, each strictly ascending, disjoint, in [0, N); channels in neither are Pruned.
 * The prefill scores of such a partition are all zero.  Same requirements and errors as above.
 */
int pop_partition_from_indices(const void* Wg, const void* Wu, const void* Wd, int N, int d,
                               pop_dtype_t dtype,
                               const int32_t* h_ret, int n_ret, const int32_t* h_cand, int n_cand,
                               void* cuda_stream, pop_partition_t** out);

/* Sizes of the three regions (host values, available as soon as the partition exists). */
int pop_partition_sizes(const pop_partition_t* p, int* n_ret, int* n_cand, int* n_pruned);

/*
 * Region index arrays: DEVICE int32 arrays owned by the partition, each ascending by channel
 * id, of the sizes above (Sec. 3.3: R, C, P are disjoint and cover all channels).  Valid on the
 * stream the partition was built on (or after synchronising it).  Any output may be NULL.
 */
int pop_partition_indices(const pop_partition_t* p, const int32_t** d_ret,
                          const int32_t** d_cand, const int32_t** d_pruned);

/*
 * Prefill importance scores I_i (Eq. 3), DEVICE double [N], owned by the partition, and a bound of
 * the error of each, DEVICE double [N]: |scores[i] - I_i of exact arithmetic| <= bounds[i].
 * fp32 partitions are scored in fp64 throughout (all bounds 0, scores within rounding of fp64).
 * bf16 partitions are scored on the tensor cores (fp32 accumulation); every channel whose bound
 * reaches one of the two rank boundaries (Retained | Candidate, Candidate | Pruned) is scored again
 * in fp64 and carries that score with bound 0, so the regions are the ones exact scores give, while
 * the scores of channels far from both boundaries are good to about 1e-4 relative.
 * A partition built by pop_partition_from_indices has all scores and bounds 0.
 */
int pop_partition_scores(const pop_partition_t* p, const double** d_scores);
int pop_partition_score_bounds(const pop_partition_t* p, const double** d_bounds);

/*
 * Diagnostic view of the last decode step's candidate scoring (Sec. 3.3 decoding stage) on a
 * partition served by the streaming kernel: DEVICE array of n_cand pairs of fp32 values
 * (score as streamed through the tensor cores, bound of |that score - exact score|), owned by
 * the partition.  The selection treats a candidate as decided only when the bounds separate it
 * from the k-th score, and re-scores the others exactly; tests use this view to check the bounds
 * against exact arithmetic.  POP_ERR_UNSUPPORTED when the partition is served by another kernel.
 */
int pop_partition_streamed_scores(const pop_partition_t* p, const float** d_score_bound_pairs);

/* Shape of a partition: any output may be NULL. */
int pop_partition_shape(const pop_partition_t* p, int* d, int* N, pop_dtype_t* dtype);

/*
 * Synchronises the partition's device (cudaDeviceSynchronize) and reports whether any decode
 * step on it gave up a bounded wait since the last check: POP_OK or POP_ERR_TIMEOUT.  After a
 * timeout the outputs of that step are undefined; the partition stays usable.
 */
int pop_partition_check(pop_partition_t* p);

/*
 * Releases everything the partition owns.  The caller must have synchronised the work that used
 * it.  Its device memory may stay with the library for the next partition of the same size on
 * the same device (at most pop_config_t.slab_cache_bytes in all; pop_release_cached_memory() returns
 * it): building a partition per prompt and layer then costs no cudaMalloc / cudaFree.
 */
int pop_partition_destroy(pop_partition_t* p);

/*
 * One decoding step (Sec. 3.3 "Decoding Stage"; Sec. 3.4: forward over R u C, scores of the
 * candidates from H_t, selection, final computation over R u selected only).
 *   x [B, d] -> y [B, d], device arrays of the partition's dtype, caller-owned; 1 <= B <= POP_MAX_BATCH.
 *   h[b, i] = silu(Wg[i].x[b]) * (Wu[i].x[b]) for i in R u C;
 *   score_i = ||Wd[:, i]||_2 * sqrt(sum_b h[b, i]^2) for i in C (one mask shared by the batch);
 *   M = the k_candidate candidates with the largest (score descending, channel id ascending),
 *       as exact (fp64) scores rank them: kernels that score in lower precision keep a bound of
 *       each score's error and re-score in fp64 every candidate the bounds cannot separate from
 *       the k-th;
 *   y[b] = sum over i in R u M of Wd[:, i] * h[b, i]   (fp32 accumulation).
 *   mask_out: uint8 [n_cand], 1 where the candidate in that slot (slot order = the d_cand array)
 *             was selected; may be NULL.
 *   sel_out : int32 [k_candidate], channel ids of the selected candidates, ascending; may be NULL.
 * No allocation, no host synchronisation.  0 <= k_candidate <= n_cand.
 * One partition serves one stream at a time (its scratch and counters are shared by its steps).
 * Two steps of the same call sequence may differ in the last bit of y: partial sums are added to
 * the fp32 accumulator in the order the SMs deliver them; the mask does not depend on that order.
 * The default kernel for bf16 partitions with d in {2048, 4096, 5120} and at most 3072 candidates is
 * launched so that its CTAs may take over SMs from the previous kernel of the stream; callers that
 * keep other streams busy on the same device should choose POP_LAUNCH_COOPERATIVE (pop_set_config):
 * a step whose CTAs cannot all be resident ends with POP_ERR_TIMEOUT at the next
 * pop_partition_check, after at most pop_config_t.wait_budget_us per wait, instead of hanging.
 * Errors: POP_ERR_INVALID_ARG, POP_ERR_UNSUPPORTED (B too large for the shape), POP_ERR_CUDA.
 */
int pop_decode_step(pop_partition_t* p, const void* x, int B, int k_candidate,
                    void* y, uint8_t* mask_out, int32_t* sel_out, void* cuda_stream);

/*
 * Prefill importance scores without any allocation.  (The paper has no counterpart: this entry
 * point exists for the library's users, not for the method.)
 *
 * Some callers cannot allocate device memory at the moment they need the scores: code running
 * inside a memory pool whose budget is fixed up front, a serving loop that forbids allocator
 * calls on its hot path because they may synchronise the device, or a host whose allocator
 * is owned by another framework.  pop_prefill_partition is closed to them, since it allocates the
 * partition and stream-ordered temporaries.  This call computes the same I_i (Eq. 3) into a buffer
 * the caller already owns, and keeps its temporaries (2 x N doubles) in a fixed 512 KB array that is
 * part of the library image on every GPU that loads it.  It scores every channel in fp64 with the
 * library's plain per-channel kernel, not with the tensor-core pass or the blocked fp64 pass that
 * pop_prefill_partition uses: the results agree with that call's scores to fp64 rounding where it
 * reports an error bound of 0 and within its reported bound elsewhere (pop_partition_score_bounds), so
 * a caller that ranks these scores gets the same regions up to ties at the last bit; it is also several
 * times slower per layer (about 14 ms at hidden 4096, intermediate 11008, 512 prompt tokens).
 *   X [L, d], Wg [N, d], Wu [N, d], Wd [d, N]: device arrays of `dtype` as for
 *   pop_prefill_partition; scores_out: device double [N], caller-owned, written on `cuda_stream`.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.
 * N > POP_NOALLOC_MAX_N is rejected with POP_ERR_UNSUPPORTED (pop_last_cuda_error() names the
 * limit); other errors as pop_prefill_partition.
 * The first call on a device looks up the device address of the fixed array (a host-side
 * query, once per device, with that device current); make that first call outside any stream
 * capture.
 * All calls on one device share the array, and it keeps the previous call's contents (every
 * entry a call reads it has written first, so nothing needs clearing).  Two calls whose kernels
 * may overlap on the GPU (different streams, no ordering between them) race on it: order them.
 */
int pop_prefill_scores_noalloc(const void* X, int L, int d,
                               const void* Wg, const void* Wu, const void* Wd, int N,
                               pop_dtype_t dtype, double* scores_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* POP_H_ */
