// Shared declarations of the POP CUDA library (internal; the public C ABI is include/pop.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "pop.h"

typedef unsigned long long u64;
typedef unsigned int u32;

// ---------------------------------------------------------------------------------------------
// Partition object (host struct; every pointer below is device memory owned by it).
//
// Repacked layout ("slots"): slot s in [0, n_ret) is Retained channel idx_ret[s]; slot
// n_ret + c is Candidate channel idx_cand[c].  n_rc = n_ret + n_cand.
//
// POP_LAYOUT_ROWS (any dtype and shape)
//   GU  [n_rc][2][d]  gate row then up row of the slot's channel, contiguous (one 2*d*es block)
//   WdT [n_rc][d]     column of the down projection of the slot's channel, as a contiguous row
//   h   [POP_MAX_BATCH][n_rc]
//
// POP_LAYOUT_TILED (bf16, d a multiple of 1024; read by pop_decode_stream.cu).  The Retained part
// is stored as mma.m16n8k16 A fragments, 512 bytes per (16 x 16) tile, lane L's 16 bytes =
// {A[g][2t..2t+1], A[g+8][2t..], A[g][2t+8..], A[g+8][2t+8..]} with g = L / 4, t = L % 4:
//   GU  = GUt  [n_rt][d/16][32][16 B]      tile (rt, kt): rows 0..7 gate, rows 8..15 up of retained
//                                            slots 8 rt .. 8 rt + 7, columns = hidden 16 kt .. 16 kt + 15
//                                            tiles n_rt .. n_rt + n_ct - 1 hold the candidate slots the same way
//         GUc  [n_cand][2][d]              candidate gate/up rows, plain (read only to re-score exactly)
//   WdT = WdTt [4][n_cg][d/64][32][16 B]   tile (q, cg, mt): rows = outputs q d/4 + 16 mt .. + 15,
//                                            columns = retained slots 16 cg .. 16 cg + 15
//         WdTc [n_cand][d]                 candidate down rows, plain
//   n_rt = ceil(n_ret / 8), n_ct = ceil(n_cand / 8), n_cg = ceil(n_ret / 16), n_ret_pad = 16 n_cg;
//   slots past n_ret (n_cand) are zero.
//   h   [POP_MAX_BATCH][h_stride]: retained slots at [0, n_ret_pad) (padding stays 0), candidates
//       at n_ret_pad + c.
// ---------------------------------------------------------------------------------------------
enum { POP_LAYOUT_ROWS = 0, POP_LAYOUT_TILED = 1 };

struct pop_partition {
    int device;
    int d, N;
    pop_dtype_t dtype;
    int es;                       // element size in bytes
    int n_ret, n_cand, n_pruned, n_rc;
    int layout;                   // POP_LAYOUT_*
    int force_simple;             // rows layout: use the multi-kernel decode path even where the fused kernel would do
    int n_rt, n_ct, n_cg, n_ret_pad, h_stride;      // tiled layout only (h_stride: both)

    void* slab;                   // the one device allocation all pointers below point into
    size_t slab_bytes;
    void* GU;
    void* WdT;
    int32_t* idx_ret;
    int32_t* idx_cand;
    int32_t* idx_pruned;
    double* scores;               // [N] prefill I_i
    double* score_bounds;         // [N] bound of |scores[i] - exact I_i| (0 where the score is exact)
    double* norm_cand;            // [n_cand] ||Wd[:, i]||_2 of the candidate channels
    float* wnorm_cand;            // [2][n_cand] max |Wg[i][:]|, max |Wu[i][:]| of the candidate channels
    double* rpart;                // [4 n_cand][POP_MAX_BATCH] decode scratch: partial dot products of re-scoring jobs

    // decode scratch (no allocation at decode time)
    float* h;                     // intermediate activations of this step: [POP_MAX_BATCH][n_rc] floats (row layout);
                                  // tiled layout: [POP_MAX_BATCH][h_stride] 8-byte words (float bits, epoch of the step)
    u64* keys;                    // [n_cand] candidate scores as ordered 64-bit keys (row layout); tiled layout:
                                  // (streamed fp32 score, bound of its error) as two 32-bit patterns
    float* y_acc;                 // [POP_MAX_BATCH][d] fp32 accumulator, zero between steps
    int32_t* sel_slots;           // [n_cand] selected candidate slots (ascending), this step
    int32_t* rank_tmp;            // [N] prefill scratch: rank of every channel by score
    u32* sync;                    // [SYNC_WORDS] counters / flags, see pop_decode*.cu
    int sm_count;
    int coop;                     // device supports cooperative launch
    int max_smem_optin;
};

// Input-independent statistics of one weight set (Wg, Wu, Wd): what a prefill needs from the weights alone.
// The weights themselves are not copied: the caller keeps them alive and unchanged while the object is in use.
struct pop_weights {
    int device;
    int d, N;
    pop_dtype_t dtype;
    const void *Wg, *Wu, *Wd;
    void* block;                  // the one device allocation behind the arrays below
    double* norm;                 // [N] ||Wd[:, i]||_2 (the weight factor of Eq. 3)
    float* gnorm;                 // [n_pad] ||Wg[i]||_2 rounded up, 0 past N (bf16 with a tensor-core prefill, else NULL)
    float* unorm;                 // [n_pad]
    int have_maps;                // tensor maps of Wg and Wu below are valid
    alignas(64) unsigned char map_g[128];
    alignas(64) unsigned char map_u[128];
};

// What the prefill kernels take of it (pointers may come from a pop_weights or from a call's own temporaries).
struct WeightStats {
    const double* norm;
    const float* gnorm;
    const float* unorm;
    const void* map_g;            // encoded tensor maps of Wg / Wu (128 bytes each), or NULL: encode per call
    const void* map_u;
};

// Process-wide settings (pop_set_config); a snapshot is taken where a decision is made.
struct PopConfig {
    int decode_kernel;                    // POP_DECODE_AUTO / _FUSED / _SIMPLE: applies when a partition is created
    int launch_mode;                      // POP_LAUNCH_*: applies to every later step of the streaming kernel
    unsigned wait_budget_us;              // how long a device-side wait may last before the step gives up
    unsigned long long slab_cache_bytes;  // freed partition memory kept for reuse, at most
};
PopConfig pop_config_snapshot();

// sync[] word assignment (contended counters sit on separate 128-byte lines)
enum { SYNC_BARRIER = 0, SYNC_TICKET = 1, SYNC_ERROR = 2, SYNC_WORK = 3,
       SYNC_EPOCH = 32, SYNC_CAST_DONE = 64 /* CTAs done with their part of the final cast */, SYNC_CAND_DONE = 96,
       SYNC_Q0 = 128 /* + 32 q, q = 0..3 */, SYNC_QC0 = 256 /* + 32 q */, SYNC_RF_DONE = 384,
       SYNC_WORDS = 416 };

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
void pop_set_cuda_error(cudaError_t e, const char* what);

#define POP_CUDA(call)                                                    \
    do {                                                                  \
        cudaError_t e__ = (call);                                         \
        if (e__ != cudaSuccess) {                                         \
            pop_set_cuda_error(e__, #call);                               \
            return (e__ == cudaErrorMemoryAllocation) ? POP_ERR_ALLOC : POP_ERR_CUDA; \
        }                                                                 \
    } while (0)

// Every kernel launch of the library goes through POP_LAUNCHED() so that callers can report
// how many of the library's kernels ran (pop_kernel_launch_count()).
void pop_count_launch(int n);
#define POP_LAUNCHED()                         \
    do {                                       \
        POP_CUDA(cudaGetLastError());          \
        pop_count_launch(1);                   \
    } while (0)

// ---------------------------------------------------------------------------------------------
// launchers implemented in the .cu files (host functions; all enqueue on `st`)
// ---------------------------------------------------------------------------------------------
// pop_prefill.cu
int pop_launch_colnorm(const void* Wd, int d, int N, pop_dtype_t dt, double* norm /*[N]*/, cudaStream_t st);
int pop_launch_gather_rows(const void* X, int L, size_t row_bytes, int stride, void* Xp /*[ceil(L / stride)] rows*/, cudaStream_t st);
int pop_launch_prefill_s2_exact(const void* X, int L, int d, const void* Wg, const void* Wu, int N,
                                pop_dtype_t dt, const int32_t* chan_list /*NULL = all*/, int n_list,
                                double* s2 /*[N], entries of listed channels are overwritten*/, cudaStream_t st);
// exact fp64 energies as a register-blocked GEMM (d a multiple of 16); s2part: [pop_prefill_s2_gemm_splits(L)][N] scratch
bool pop_prefill_s2_gemm_supported(int d);
int pop_prefill_s2_gemm_splits(int L);
int pop_launch_prefill_s2_gemm(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                               double* s2part, double* s2, cudaStream_t st);
// the same pass, enqueued always but run only when *run_if_gt > threshold (a device-side decision)
int pop_launch_prefill_s2_gemm_if(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                                  double* s2part, double* s2, const int* run_if_gt, int threshold, cudaStream_t st);
// only the blocked pass (no sum over the token ranges), gated the same way
int pop_launch_prefill_s2_gemm_parts_if(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                                        double* s2part, const int* run_if_gt, int threshold, cudaStream_t st);
// scores[i] = sqrt(s2[i]) * norm[i]; also zeroes rank_to_zero[i] when that is not NULL
int pop_launch_scores(const double* s2, const double* norm, int N, double* scores, int32_t* rank_to_zero, cudaStream_t st);
// rank[i] += position of channel i in the order (score descending, channel id ascending); the caller has zeroed rank [N]
// earlier on the stream (the kernels that write the scores do it: scores_kernel, tc_finish_kernel, rescore_finish_kernel)
int pop_launch_ranks(const double* scores, int N, int32_t* rank, int sm_count, cudaStream_t st);
int pop_launch_partition(const double* scores, int N, int n_ret, int n_cand, int32_t* rank_zeroed /*[N]*/, int sm_count,
                         int32_t* idx_ret, int32_t* idx_cand, int32_t* idx_pruned, cudaStream_t st);
int pop_launch_partition_after_rescore(const double* scores, int N, int n_ret, int n_cand, int32_t* rank, int sm_count,
                                       const int32_t* list, const int* n_list, int max_list, int32_t* idx_ret,
                                       int32_t* idx_cand, int32_t* idx_pruned, cudaStream_t st);
int pop_launch_repack(const pop_partition* p, const void* Wg, const void* Wu, const void* Wd,
                      const double* norm /*[N]*/, cudaStream_t st);
int pop_launch_repack_tiled(const pop_partition* p, const void* Wg, const void* Wu, const void* Wd,
                            const double* norm /*[N]*/, cudaStream_t st);
// pop_prefill_tc.cu (bf16: activation energies on the tensor cores with error bounds, exact re-scoring of the
// channels the bounds cannot place)
#define POP_PREFILL_MAX_LIST 4096     // longest list the list re-scoring kernel takes; longer lists use the full fp64 pass
struct PrefillTcPlan { int n_ct, n_tt, n_pad, l_pad, n_parts, n_tb, max_list; };
struct PrefillTcScratch {
    void* H;               // [2][l_pad][n_pad] bf16 (high, low) intermediate activations of the prompt, or NULL
    float* xnorm;          // [l_pad]
    float* gnorm;          // [n_pad]
    float* unorm;          // [n_pad]
    double* s2part;        // [n_parts][n_pad]
    float* bpart;          // [n_parts][n_pad]
    u64* m_max;            // largest score bound (bits of a double)
    int32_t* list;         // [N] channels to re-score
    int* n_list;
    int32_t* rank;         // [N] rank of every channel by streamed score
    double* part;          // [max_list][n_tb]
    double* s2part_full;   // [pop_prefill_s2_gemm_splits(L)][N]
};
bool pop_prefill_tc_supported(int d, pop_dtype_t dt);
void pop_prefill_tc_plan(int L, int d, int N, PrefillTcPlan* plan);
// row norms of Wg and Wu (rounded up, zero past N up to n_pad) in one launch; encoded tensor maps of Wg and Wu
int pop_launch_weight_rownorms(const void* Wg, const void* Wu, int N, int n_pad, int d, float* gnorm, float* unorm, cudaStream_t st);
int pop_prefill_tc_encode_weight_maps(const void* Wg, const void* Wu, int N, int d, void* map_g, void* map_u);
int pop_launch_prefill_tc(const void* X, int L, int d, const void* Wg, const void* Wu, int N, const WeightStats& ws,
                          const PrefillTcScratch& s, double* scores, double* bounds, u32* status, int sm_count,
                          cudaStream_t st);
int pop_launch_prefill_rescore(const void* X, int L, int d, const void* Wg, const void* Wu, int N, const double* norm,
                               int n_ret, int n_cand, int n_third /*extra rank boundary, 0 = none*/, const PrefillTcScratch& s,
                               double* scores, double* bounds, int sm_count, cudaStream_t st);
// the prompt's own output from H (cleared outside the mask rank < n_active) and Wd [d, N], on the tensor cores
bool pop_prefill_output_supported(int d, int N, pop_dtype_t dt);
int pop_launch_prefill_output(void* H, int L, int d, const void* Wd, int N, const int32_t* rank, int n_active, void* Y,
                              u32* status, int sm_count, cudaStream_t st);
// pop_decode_stream.cu (bf16 partitions in the tiled layout)
bool pop_stream_layout_supported(int d, pop_dtype_t dt);
int pop_stream_max_candidates();          // the streaming kernel's selection warp holds this many candidate keys
int pop_launch_decode_stream(pop_partition* p, const void* x, int B, int k, void* y,
                             uint8_t* mask_out, int32_t* sel_out, cudaStream_t st);
// pop_decode_simple.cu (multi-kernel path, any accepted shape)
int pop_launch_decode_simple(pop_partition* p, const void* x, int B, int k, void* y,
                             uint8_t* mask_out, int32_t* sel_out, cudaStream_t st);
// pop_decode.cu (fused persistent kernel; returns POP_ERR_UNSUPPORTED for shapes it does not take)
int pop_launch_decode(pop_partition* p, const void* x, int B, int k, void* y,
                      uint8_t* mask_out, int32_t* sel_out, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int VEC = 4;                       // elements per 16-byte vector
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float to_f32(float v) { return v; }
    __device__ static __forceinline__ float from_f32(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int VEC = 8;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ static __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ static __forceinline__ __nv_bfloat16 from_f32(float v) { return __float2bfloat16_rn(v); }
};

// silu(z) = z / (1 + exp(-z)), in the precision of the argument.
__device__ __forceinline__ double silu_f64(double z) { return z / (1.0 + exp(-z)); }
__device__ __forceinline__ float silu_f32(float z) { return z / (1.0f + expf(-z)); }

__device__ __forceinline__ unsigned long long pop_global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Budget of a device-side wait in wall time.  The timer is read only every 64 polls (reading it is not free), so a
// wait that ends within 64 polls never touches it; with a budget of 0 the wait gives up at the first reading.
struct PopWaitClock {
    u32 polls;
    unsigned long long t0;
    __device__ __forceinline__ PopWaitClock() : polls(0u), t0(0ull) {}
    __device__ __forceinline__ bool expired(unsigned long long budget_ns) {
        if ((++polls & 63u) != 0u) return false;
        const unsigned long long now = pop_global_ns();
        if (polls == 64u) { t0 = now; return budget_ns == 0ull; }
        return now - t0 > budget_ns;
    }
};

// Scores are non-negative finite doubles: their bit patterns order like the values.
__device__ __forceinline__ u64 score_key(double s) { return (u64)__double_as_longlong(s); }

#endif  // __CUDACC__
