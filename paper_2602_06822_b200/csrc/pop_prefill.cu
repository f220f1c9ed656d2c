// Prefilling stage of POP (Sec. 3.3 "Prefilling Stage"; score of Sec. 3.4 Eq. 3):
//   column norms of the down projection, per-channel activation energy over the prompt,
//   importance scores, rank-select into Retained / Candidate / Pruned, weight repack.
#include "pop_common.cuh"
#include <stdlib.h>
#include "pop_select.cuh"

// ---------------------------------------------------------------------------------------------
// n_i = ||Wd[:, i]||_2  (the weight factor of Eq. 3: ||W[:, i] * s_i||_2 = |s_i| * ||W[:, i]||_2).
// Block (32 columns x 32 row strips); every column is summed in the same fixed order, so equal
// columns give bit-equal norms.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(1024) colnorm_kernel(const T* __restrict__ Wd, int d, int N,
                                                       double* __restrict__ norm) {
    __shared__ double part[32][33];
    const int cx = threadIdx.x, ry = threadIdx.y;
    const int c = blockIdx.x * 32 + cx;
    double acc = 0.0;
    if (c < N) {
        for (int j = ry; j < d; j += 32) {
            double v = (double)Elem<T>::to_f32(Wd[(size_t)j * N + c]);
            acc = fma(v, v, acc);
        }
    }
    part[ry][cx] = acc;
    __syncthreads();
    if (ry == 0 && c < N) {
        double s = 0.0;
#pragma unroll 1
        for (int r = 0; r < 32; ++r) s += part[r][cx];
        norm[c] = sqrt(s);
    }
}

// Every stride-th row of X [L, row_bytes] (rows 0, stride, 2 stride, ...) into Xp, contiguous: the probe tokens of a
// partial-probing prefill (Sec. 3.4).  16-byte vectors; row_bytes is a multiple of 16.
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ X, int rows_out, int vec_per_row, int stride,
                                                          uint4* __restrict__ Xp) {
    const size_t total = (size_t)rows_out * vec_per_row;
    for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
        const size_t r = o / vec_per_row, v = o - r * vec_per_row;
        Xp[o] = __ldg(X + r * (size_t)stride * vec_per_row + v);
    }
}

int pop_launch_gather_rows(const void* X, int L, size_t row_bytes, int stride, void* Xp, cudaStream_t st) {
    const int rows_out = (L + stride - 1) / stride, vec = (int)(row_bytes / 16);
    const size_t total = (size_t)rows_out * vec;
    if (total == 0) return POP_OK;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    gather_rows_kernel<<<blocks, 256, 0, st>>>((const uint4*)X, rows_out, vec, stride, (uint4*)Xp);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_colnorm(const void* Wd, int d, int N, pop_dtype_t dt, double* norm, cudaStream_t st) {
    dim3 blk(32, 32), grd((N + 31) / 32);
    if (dt == POP_F32) colnorm_kernel<float><<<grd, blk, 0, st>>>((const float*)Wd, d, N, norm);
    else colnorm_kernel<__nv_bfloat16><<<grd, blk, 0, st>>>((const __nv_bfloat16*)Wd, d, N, norm);
    POP_LAUNCHED();
    return POP_OK;
}

// ---------------------------------------------------------------------------------------------
// Exact (fp64) activation energy  s2[i] = sum_t H[t, i]^2,  H[t, i] = silu(Wg[i].X[t]) * (Wu[i].X[t])
// for the channels in chan_list (all channels when chan_list == NULL).
//
// One block owns 32 channels and walks over all tokens in tiles of 32; K is consumed in chunks
// of 32 staged in shared memory as doubles.  Thread (tx, ty) of the 16 x 16 block computes
// channels {tx, tx+16} x tokens {ty, ty+16}.  The per-channel sum over tokens is taken in a
// fixed order that is the same for every channel.
// ---------------------------------------------------------------------------------------------
#define S2_CT 32
#define S2_TT 32
#define S2_KT 32

template <typename T>
__global__ void __launch_bounds__(256) prefill_s2_exact_kernel(
    const T* __restrict__ X, int L, int d, const T* __restrict__ Wg, const T* __restrict__ Wu, int N,
    const int32_t* __restrict__ chan_list, int n_list, double* __restrict__ s2) {
    __shared__ double Xs[S2_TT][S2_KT + 1];
    __shared__ double Gs[S2_CT][S2_KT + 1];
    __shared__ double Us[S2_CT][S2_KT + 1];
    __shared__ int chan[S2_CT];
    __shared__ double red[16][S2_CT + 1];

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int c0 = blockIdx.x * S2_CT;
    if (tid < S2_CT) {
        int li = c0 + tid;
        chan[tid] = (li < n_list) ? (chan_list ? chan_list[li] : li) : -1;
    }
    __syncthreads();

    double e[2] = {0.0, 0.0};                     // energy of channels tx, tx+16 over this thread's tokens
    for (int t0 = 0; t0 < L; t0 += S2_TT) {
        double g[2][2] = {{0, 0}, {0, 0}}, u[2][2] = {{0, 0}, {0, 0}};
        for (int k0 = 0; k0 < d; k0 += S2_KT) {
            // stage X[t0..+32][k0..+32], Wg/Wu[chan][k0..+32] as doubles (zero outside bounds)
            for (int idx = tid; idx < S2_TT * S2_KT; idx += 256) {
                int r = idx / S2_KT, kk = idx % S2_KT, k = k0 + kk;
                int t = t0 + r;
                Xs[r][kk] = (t < L && k < d) ? (double)Elem<T>::to_f32(X[(size_t)t * d + k]) : 0.0;
                int ch = chan[r];
                bool ok = ch >= 0 && k < d;
                Gs[r][kk] = ok ? (double)Elem<T>::to_f32(Wg[(size_t)ch * d + k]) : 0.0;
                Us[r][kk] = ok ? (double)Elem<T>::to_f32(Wu[(size_t)ch * d + k]) : 0.0;
            }
            __syncthreads();
#pragma unroll 8
            for (int kk = 0; kk < S2_KT; ++kk) {
                double x0 = Xs[ty][kk], x1 = Xs[ty + 16][kk];
                double g0 = Gs[tx][kk], g1 = Gs[tx + 16][kk];
                double u0 = Us[tx][kk], u1 = Us[tx + 16][kk];
                g[0][0] = fma(g0, x0, g[0][0]); g[0][1] = fma(g0, x1, g[0][1]);
                g[1][0] = fma(g1, x0, g[1][0]); g[1][1] = fma(g1, x1, g[1][1]);
                u[0][0] = fma(u0, x0, u[0][0]); u[0][1] = fma(u0, x1, u[0][1]);
                u[1][0] = fma(u1, x0, u[1][0]); u[1][1] = fma(u1, x1, u[1][1]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                // tokens beyond L contribute silu(0) * 0 = 0
                double h = silu_f64(g[c][t]) * u[c][t];
                e[c] = fma(h, h, e[c]);
            }
    }
    red[ty][tx] = e[0];
    red[ty][tx + 16] = e[1];
    __syncthreads();
    if (tid < S2_CT && chan[tid] >= 0) {
        double s = 0.0;
#pragma unroll 1
        for (int r = 0; r < 16; ++r) s += red[r][tid];
        s2[chan[tid]] = s;
    }
}

int pop_launch_prefill_s2_exact(const void* X, int L, int d, const void* Wg, const void* Wu, int N,
                                pop_dtype_t dt, const int32_t* chan_list, int n_list, double* s2,
                                cudaStream_t st) {
    if (n_list <= 0) return POP_OK;
    dim3 grd((n_list + S2_CT - 1) / S2_CT);
    if (dt == POP_F32)
        prefill_s2_exact_kernel<float><<<grd, 256, 0, st>>>((const float*)X, L, d, (const float*)Wg,
                                                            (const float*)Wu, N, chan_list, n_list, s2);
    else
        prefill_s2_exact_kernel<__nv_bfloat16><<<grd, 256, 0, st>>>(
            (const __nv_bfloat16*)X, L, d, (const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu, N,
            chan_list, n_list, s2);
    POP_LAUNCHED();
    return POP_OK;
}

// ---------------------------------------------------------------------------------------------
// The same activation energy, exact in fp64, as a register-blocked GEMM for hidden sizes that
// are a multiple of 16: the fp64 pipe, not shared memory or the conversions, is what bounds it.
//
// Block = 256 threads = 8 warps; block tile = 256 tokens x 32 channels (gate and up at once);
// a warp owns 32 tokens x 32 channels, lane (tg, cg) = (lane / 8, lane % 8) a tile of 8 tokens x
// 4 channels x {gate, up} = 64 accumulators (channels 2 cg, 2 cg + 1, 16 + 2 cg, 17 + 2 cg, so that the
// 16-byte loads of the 8 lanes that are served together cover 128 contiguous bytes: no bank conflict).
// K is consumed in chunks of KT (16; 32 for bf16, which halves the block barriers), staged in shared
// memory as doubles ([k][token] and [k][channel], so a lane reads its operands as contiguous
// 16-byte pieces that the lanes of a warp share by broadcast), double-buffered with the next
// chunk's global loads in flight during the arithmetic.  blockIdx.y splits the tokens into
// ranges of tok_per_split; range y writes its partial energies to s2out[y * out_stride + channel],
// and the caller adds the ranges in a fixed order.
// ---------------------------------------------------------------------------------------------
#define G2_TOK 256
#define G2_CH 32
#define G2_KT 16

template <typename T, int KT>
__global__ void __launch_bounds__(256, 1) prefill_s2_gemm_kernel(
    const T* __restrict__ X, int L, int d, const T* __restrict__ Wg, const T* __restrict__ Wu,
    const int32_t* __restrict__ chan_list, int n_list, int tok_per_split, double* __restrict__ s2out, int out_stride,
    const int* __restrict__ run_if_gt, int threshold) {
    if (run_if_gt && *run_if_gt <= threshold) return;           // the same decision in every thread of the grid
    constexpr int EPV = 16 / sizeof(T);               // elements per 16-byte vector
    constexpr int XV = KT / EPV;                   // vectors per token row and chunk
    constexpr int WV = (KT / 2) / EPV;                // vectors per (matrix, channel, half chunk)
    extern __shared__ __align__(16) double g2_sm[];
    double* Xs = g2_sm;                               // [2][KT][G2_TOK]
    double* Gs = Xs + 2 * KT * G2_TOK;             // [2][KT][G2_CH]
    double* Us = Gs + 2 * KT * G2_CH;
    __shared__ int chan[G2_CH];
    __shared__ double red[8][G2_CH];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, tg = lane >> 3, cg = lane & 7;
    const int c0 = blockIdx.x * G2_CH;
    if (tid < G2_CH) {
        const int li = c0 + tid;
        chan[tid] = (li < n_list) ? (chan_list ? chan_list[li] : li) : -1;
    }
    __syncthreads();
    const int t_begin = blockIdx.y * tok_per_split, t_end = min(L, t_begin + tok_per_split);
    const int nk = d / KT;

    // staging roles: every thread one token row of X; threads 0..127 one (matrix, channel, half chunk) of W
    const int wm = tid >> 6, wc = (tid >> 1) & 31, wh = tid & 1;
    const int wch = tid < 128 ? chan[wc] : -1;
    const T* wrow = wch >= 0 ? (wm ? Wu : Wg) + (size_t)wch * d + wh * (KT / 2) : nullptr;

    double e[4] = {0.0, 0.0, 0.0, 0.0};
    for (int t0 = t_begin; t0 < t_end; t0 += G2_TOK) {
        const int tok = t0 + tid;
        const T* xrow = tok < t_end ? X + (size_t)tok * d : nullptr;
        uint4 xr[XV], wr[WV];
        auto fetch = [&](int kc) {
#pragma unroll
            for (int v = 0; v < XV; ++v)
                xr[v] = xrow ? __ldg(reinterpret_cast<const uint4*>(xrow + kc * KT) + v) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int v = 0; v < WV; ++v)
                wr[v] = wrow ? __ldg(reinterpret_cast<const uint4*>(wrow + kc * KT) + v) : make_uint4(0u, 0u, 0u, 0u);
        };
        auto stash = [&](int buf) {
#pragma unroll
            for (int v = 0; v < XV; ++v) {
                float f[EPV];
                Elem<T>::unpack(xr[v], f);
#pragma unroll
                for (int j = 0; j < EPV; ++j) Xs[(buf * KT + v * EPV + j) * G2_TOK + tid] = (double)f[j];
            }
            if (tid < 128) {
                double* dst = wm ? Us : Gs;
#pragma unroll
                for (int v = 0; v < WV; ++v) {
                    float f[EPV];
                    Elem<T>::unpack(wr[v], f);
#pragma unroll
                    for (int j = 0; j < EPV; ++j) dst[(buf * KT + wh * (KT / 2) + v * EPV + j) * G2_CH + wc] = (double)f[j];
                }
            }
        };
        double g[8][4], u[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) { g[j][c] = 0.0; u[j][c] = 0.0; }

        fetch(0);
        stash(0);
        __syncthreads();
#pragma unroll 1
        for (int kc = 0; kc < nk; ++kc) {
            const int buf = kc & 1;
            if (kc + 1 < nk) fetch(kc + 1);
            const double* xs = Xs + (size_t)buf * KT * G2_TOK + warp * 32 + tg * 8;
            const double* gs = Gs + (size_t)buf * KT * G2_CH + cg * 2;
            const double* us = Us + (size_t)buf * KT * G2_CH + cg * 2;
#pragma unroll
            for (int k = 0; k < KT; ++k) {
                double xv[8], gv[4], uv[4];
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    const double2 t2 = *reinterpret_cast<const double2*>(xs + k * G2_TOK + j);
                    xv[j] = t2.x; xv[j + 1] = t2.y;
                }
#pragma unroll
                for (int c = 0; c < 4; c += 2) {        // channels 2 cg, 2 cg + 1, then 16 + 2 cg, 17 + 2 cg
                    const double2 a2 = *reinterpret_cast<const double2*>(gs + k * G2_CH + c * 8);
                    const double2 b2 = *reinterpret_cast<const double2*>(us + k * G2_CH + c * 8);
                    gv[c] = a2.x; gv[c + 1] = a2.y; uv[c] = b2.x; uv[c + 1] = b2.y;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        g[j][c] = fma(gv[c], xv[j], g[j][c]);
                        u[j][c] = fma(uv[c], xv[j], u[j][c]);
                    }
            }
            if (kc + 1 < nk) stash(buf ^ 1);
            __syncthreads();
        }
        // tokens past the end contribute silu(0) * 0 = 0
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const double h = silu_f64(g[j][c]) * u[j][c];
                e[c] = fma(h, h, e[c]);
            }
    }
    // channel sums: over the 4 token groups of the warp, then over the 8 warps, in a fixed order
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        e[c] += __shfl_xor_sync(0xffffffffu, e[c], 8);
        e[c] += __shfl_xor_sync(0xffffffffu, e[c], 16);
    }
    if (tg == 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) red[warp][(c >> 1) * 16 + cg * 2 + (c & 1)] = e[c];
    }
    __syncthreads();
    if (tid < G2_CH && chan[tid] >= 0) {
        double sum = 0.0;
#pragma unroll 1
        for (int r = 0; r < 8; ++r) sum += red[r][tid];
        s2out[(size_t)blockIdx.y * out_stride + chan[tid]] = sum;
    }
}

// s2[i] = sum over the token ranges (ascending) of s2part[y][i]
__global__ void sum_ranges_kernel(const double* __restrict__ s2part, int nsplit, int N, double* __restrict__ s2,
                                  const int* __restrict__ run_if_gt, int threshold) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N || (run_if_gt && *run_if_gt <= threshold)) return;
    double sum = 0.0;
    for (int y = 0; y < nsplit; ++y) sum += s2part[(size_t)y * N + i];
    s2[i] = sum;
}

int pop_prefill_s2_gemm_splits(int L) { return L > 0 ? (L + G2_TOK - 1) / G2_TOK : 1; }

bool pop_prefill_s2_gemm_supported(int d) { return d >= G2_KT && d % G2_KT == 0; }

template <typename T, int KT>
static int launch_s2_gemm(const void* X, int L, int d, const void* Wg, const void* Wu, int N, double* s2part,
                          const int* run_if_gt, int threshold, cudaStream_t st) {
    auto kern = prefill_s2_gemm_kernel<T, KT>;
    const size_t smem = sizeof(double) * (2 * KT * G2_TOK + 4 * KT * G2_CH);
    static thread_local int cfg_dev = -1;
    int dev = 0;
    POP_CUDA(cudaGetDevice(&dev));
    if (cfg_dev != dev) {
        POP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        cfg_dev = dev;
    }
    dim3 grd((N + G2_CH - 1) / G2_CH, pop_prefill_s2_gemm_splits(L));
    kern<<<grd, 256, smem, st>>>((const T*)X, L, d, (const T*)Wg, (const T*)Wu, nullptr, N, G2_TOK, s2part, N, run_if_gt, threshold);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_prefill_s2_gemm_parts_if(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                                        double* s2part, const int* run_if_gt, int threshold, cudaStream_t st) {
    if (N <= 0) return POP_OK;
    if (dt == POP_F32) return launch_s2_gemm<float, G2_KT>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
    if (d % 32 == 0) return launch_s2_gemm<__nv_bfloat16, 32>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
    return launch_s2_gemm<__nv_bfloat16, G2_KT>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
}

int pop_launch_prefill_s2_gemm_if(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                                  double* s2part, double* s2, const int* run_if_gt, int threshold, cudaStream_t st) {
    if (N <= 0) return POP_OK;
    int rc;
    // K chunks of 32 for bf16 (half the block barriers of 16; measured 4.33 -> 4.14 ms at d 4096, N 11008, L 512)
    if (dt == POP_F32) rc = launch_s2_gemm<float, G2_KT>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
    else if (d % 32 == 0) rc = launch_s2_gemm<__nv_bfloat16, 32>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
    else rc = launch_s2_gemm<__nv_bfloat16, G2_KT>(X, L, d, Wg, Wu, N, s2part, run_if_gt, threshold, st);
    if (rc != POP_OK) return rc;
    sum_ranges_kernel<<<(N + 255) / 256, 256, 0, st>>>(s2part, pop_prefill_s2_gemm_splits(L), N, s2, run_if_gt, threshold);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_prefill_s2_gemm(const void* X, int L, int d, const void* Wg, const void* Wu, int N, pop_dtype_t dt,
                               double* s2part, double* s2, cudaStream_t st) {
    return pop_launch_prefill_s2_gemm_if(X, L, d, Wg, Wu, N, dt, s2part, s2, nullptr, 0, st);
}

// I_i = sqrt(s2_i) * n_i   (Eq. 3)
__global__ void scores_kernel(const double* __restrict__ s2, const double* __restrict__ norm, int N,
                              double* __restrict__ scores, int32_t* __restrict__ rank_to_zero) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) {
        scores[i] = sqrt(s2[i]) * norm[i];
        if (rank_to_zero) rank_to_zero[i] = 0;
    }
}

int pop_launch_scores(const double* s2, const double* norm, int N, double* scores, int32_t* rank_to_zero, cudaStream_t st) {
    scores_kernel<<<(N + 255) / 256, 256, 0, st>>>(s2, norm, N, scores, rank_to_zero);
    POP_LAUNCHED();
    return POP_OK;
}

// ---------------------------------------------------------------------------------------------
// Partition (Sec. 3.3): rank by (score descending, channel id ascending); the first n_ret channels are Retained,
// the next n_cand Candidate, the rest Pruned: the tau_high and tau_low thresholds of the paper taken by rank, with
// ties split by channel id.
//
// Ranks by counting: rank[i] = #{j : key_j > key_i} + #{j < i : key_j == key_i}, the channel's position in that
// total order.  N^2 comparisons are little work for the whole GPU (N = 11008: 121 M) and need no atomics on shared
// histogram bins, which is where a single-block radix select spends its time when the keys are the scores of
// similar channels.  Block (x, y): 512 channels i (two per thread) against the y-th slice of the j range, staged
// in shared memory; the partial counts meet in rank[] (zeroed earlier on the stream) through one atomic per channel and block.
// ---------------------------------------------------------------------------------------------
#define RANK_NT 256
#define RANK_TILE 1024

__global__ void __launch_bounds__(RANK_NT) rank_kernel(const u64* __restrict__ keys, int N, int j_chunk, int32_t* __restrict__ rank,
                                                       const int* __restrict__ run_if_gt, int threshold) {
    __shared__ u64 kj[RANK_TILE];
    if (run_if_gt && *run_if_gt <= threshold) return;           // the same decision in every thread of the grid
    const int tid = threadIdx.x;
    const int i_lo = blockIdx.x * (2 * RANK_NT), i0 = i_lo + tid, i1 = i0 + RANK_NT;
    const u64 k0 = i0 < N ? keys[i0] : ~0ull, k1 = i1 < N ? keys[i1] : ~0ull;
    int c0 = 0, c1 = 0;
    const int j_begin = blockIdx.y * j_chunk, j_end = min(N, j_begin + j_chunk);
    for (int t0 = j_begin; t0 < j_end; t0 += RANK_TILE) {
        const int tn = min(RANK_TILE, j_end - t0);
        __syncthreads();
        for (int j = tid; j < tn; j += RANK_NT) kj[j] = keys[t0 + j];
        __syncthreads();
        if (t0 + tn <= i_lo) {                            // every j of the tile precedes every i of the block: ties count
#pragma unroll 8
            for (int j = 0; j < tn; ++j) { const u64 k = kj[j]; c0 += (k >= k0); c1 += (k >= k1); }
        } else if (t0 >= i_lo + 2 * RANK_NT) {            // every j follows every i: ties do not count
#pragma unroll 8
            for (int j = 0; j < tn; ++j) { const u64 k = kj[j]; c0 += (k > k0); c1 += (k > k1); }
        } else {
#pragma unroll 4
            for (int j = 0; j < tn; ++j) {
                const u64 k = kj[j];
                const int jj = t0 + j;
                c0 += (k > k0) || (k == k0 && jj < i0);
                c1 += (k > k1) || (k == k1 && jj < i1);
            }
        }
    }
    if (i0 < N && c0) atomicAdd(&rank[i0], c0);
    if (i1 < N && c1) atomicAdd(&rank[i1], c1);
}

// Ranks of the listed channels only (the others keep theirs): rank[list[t]] += number of channels that precede it.
// Block (x, y): 128 listed channels against the y-th slice of all channels.  Runs when 0 < *n_list <= max_list.
__global__ void __launch_bounds__(128) rank_list_kernel(const u64* __restrict__ keys, int N, int j_chunk,
                                                        const int32_t* __restrict__ list, const int* __restrict__ n_list,
                                                        int max_list, int32_t* __restrict__ rank) {
    __shared__ u64 kj[RANK_TILE];
    const int n = *n_list;
    if (n <= 0 || n > max_list || (int)(blockIdx.x * 128) >= n) return;
    const int tid = threadIdx.x, t = blockIdx.x * 128 + tid;
    const int i = t < n ? list[t] : -1;
    const u64 ki = i >= 0 ? keys[i] : ~0ull;
    int c = 0;
    const int j_begin = blockIdx.y * j_chunk, j_end = min(N, j_begin + j_chunk);
    for (int t0 = j_begin; t0 < j_end; t0 += RANK_TILE) {
        const int tn = min(RANK_TILE, j_end - t0);
        __syncthreads();
        for (int j = tid; j < tn; j += 128) kj[j] = keys[t0 + j];
        __syncthreads();
#pragma unroll 4
        for (int j = 0; j < tn; ++j) {
            const u64 k = kj[j];
            c += (k > ki) || (k == ki && t0 + j < i);
        }
    }
    if (i >= 0 && c) atomicAdd(&rank[i], c);
}

static int launch_ranks(const double* scores, int N, int32_t* rank, int sm_count, const int* run_if_gt, int threshold, cudaStream_t st) {
    const int bx = (N + 2 * RANK_NT - 1) / (2 * RANK_NT);
    int by = (8 * sm_count + bx - 1) / bx;                                   // about eight blocks per SM in all (the kernel is bound by latency: four took 39 us at N = 11008)
    const int max_by = (N + 255) / 256;
    if (by > max_by) by = max_by;
    if (by < 1) by = 1;
    int j_chunk = (N + by - 1) / by;
    j_chunk = (j_chunk + 255) & ~255;                                        // slice boundaries on multiples of 256
    by = (N + j_chunk - 1) / j_chunk;
    rank_kernel<<<dim3(bx, by), RANK_NT, 0, st>>>(reinterpret_cast<const u64*>(scores), N, j_chunk, rank, run_if_gt, threshold);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_ranks(const double* scores, int N, int32_t* rank, int sm_count, cudaStream_t st) {
    return launch_ranks(scores, N, rank, sm_count, nullptr, 0, st);
}

// The three ascending index lists from the ranks: one block, every thread a contiguous chunk of channel ids.
#define PART_NT 1024

__global__ void __launch_bounds__(PART_NT) partition_kernel(const int32_t* __restrict__ rank, int N, int n_ret, int n_cand,
                                                            int32_t* __restrict__ idx_ret,
                                                            int32_t* __restrict__ idx_cand,
                                                            int32_t* __restrict__ idx_pruned) {
    __shared__ u32 sm[POP_SELECT_SMEM_WORDS(PART_NT)];
    const int tid = threadIdx.x;
    const int per = (N + PART_NT - 1) / PART_NT;
    const int lo = min(N, tid * per), hi = min(N, lo + per);
    const int n_rc = n_ret + n_cand;
    int cR = 0, cC = 0, cP = 0;
    for (int i = lo; i < hi; ++i) {
        const int r = rank[i];
        if (r < n_ret) ++cR; else if (r < n_rc) ++cC; else ++cP;
    }
    int tot;
    int pR = group_excl_scan<PART_NT>(cR, sm, tid, 0, tot);
    int pC = group_excl_scan<PART_NT>(cC, sm, tid, 0, tot);
    int pP = group_excl_scan<PART_NT>(cP, sm, tid, 0, tot);
    for (int i = lo; i < hi; ++i) {
        const int r = rank[i];
        if (r < n_ret) idx_ret[pR++] = i; else if (r < n_rc) idx_cand[pC++] = i; else idx_pruned[pP++] = i;
    }
}

int pop_launch_partition(const double* scores, int N, int n_ret, int n_cand, int32_t* rank_tmp /* zeroed */, int sm_count, int32_t* idx_ret,
                         int32_t* idx_cand, int32_t* idx_pruned, cudaStream_t st) {
    const int rc = pop_launch_ranks(scores, N, rank_tmp, sm_count, st);
    if (rc != POP_OK) return rc;
    partition_kernel<<<1, PART_NT, 0, st>>>(rank_tmp, N, n_ret, n_cand, idx_ret, idx_cand, idx_pruned);
    POP_LAUNCHED();
    return POP_OK;
}

// After a re-scoring of the listed channels: only they can have changed sides of a rank boundary, and a channel that
// was not listed is on the same side under the mixed scores as under its first rank (argument at
// select_uncertain_kernel), so only the listed channels are ranked again (their rank entries were cleared by
// rescore_finish_kernel).  When the list was longer than max_list every score was replaced: then all ranks were
// cleared and the full ranking runs instead.
int pop_launch_partition_after_rescore(const double* scores, int N, int n_ret, int n_cand, int32_t* rank, int sm_count,
                                       const int32_t* list, const int* n_list, int max_list, int32_t* idx_ret,
                                       int32_t* idx_cand, int32_t* idx_pruned, cudaStream_t st) {
    // lists are short (blocks past the list's end return at once), so the channel axis is cut finely
    int by = (N + 255) / 256;
    if (by > 128) by = 128;
    if (by < 1) by = 1;
    (void)sm_count;
    int j_chunk = (((N + by - 1) / by) + 255) & ~255;
    by = (N + j_chunk - 1) / j_chunk;
    rank_list_kernel<<<dim3((max_list + 127) / 128, by), 128, 0, st>>>(reinterpret_cast<const u64*>(scores), N, j_chunk, list, n_list,
                                                                      max_list, rank);
    POP_LAUNCHED();
    if (max_list < N) {
        const int rc = launch_ranks(scores, N, rank, sm_count, n_list, max_list, st);
        if (rc != POP_OK) return rc;
    }
    partition_kernel<<<1, PART_NT, 0, st>>>(rank, N, n_ret, n_cand, idx_ret, idx_cand, idx_pruned);
    POP_LAUNCHED();
    return POP_OK;
}

// ---------------------------------------------------------------------------------------------
// Repack: live rows of Wg/Wu interleaved per slot, live columns of Wd transposed into rows.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int slot_channel(int s, int n_ret, const int32_t* idx_ret, const int32_t* idx_cand) {
    return s < n_ret ? idx_ret[s] : idx_cand[s - n_ret];
}

// one block per slot; rows are d*es bytes, a multiple of 16.  The block of a candidate slot also leaves the
// candidate's weight factor of Eq. 3 in norm_cand and, when wmax is given (bf16, streaming decode kernel), the
// largest magnitudes of its gate and up rows in wmax[0][c], wmax[1][c]: with max |x| they bound any single product
// of the candidate's dot products (used by the error bound of its streamed score).
__global__ void __launch_bounds__(256) repack_gu_kernel(const uint4* __restrict__ Wg, const uint4* __restrict__ Wu,
                                                        int row_vecs, int n_ret, int n_cand,
                                                        const int32_t* __restrict__ idx_ret,
                                                        const int32_t* __restrict__ idx_cand,
                                                        uint4* __restrict__ GU, const double* __restrict__ norm,
                                                        double* __restrict__ norm_cand, float* __restrict__ wmax) {
    __shared__ float red[2][8];
    const int s = blockIdx.x;
    const int ch = slot_channel(s, n_ret, idx_ret, idx_cand);
    const uint4* g = Wg + (size_t)ch * row_vecs;
    const uint4* u = Wu + (size_t)ch * row_vecs;
    uint4* o = GU + (size_t)s * 2 * row_vecs;
    float mg = 0.f, mu = 0.f;
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        const uint4 a = g[v], b = u[v];
        o[v] = a;
        o[row_vecs + v] = b;
        if (wmax) {                                   // bf16 rows only
            float f[8];
            Elem<__nv_bfloat16>::unpack(a, f);
#pragma unroll
            for (int j = 0; j < 8; ++j) mg = fmaxf(mg, fabsf(f[j]));
            Elem<__nv_bfloat16>::unpack(b, f);
#pragma unroll
            for (int j = 0; j < 8; ++j) mu = fmaxf(mu, fabsf(f[j]));
        }
    }
    if (s < n_ret) return;
    const int c = s - n_ret;
    if (threadIdx.x == 0 && norm_cand) norm_cand[c] = norm[ch];
    if (wmax) {
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, off));
            mu = fmaxf(mu, __shfl_xor_sync(0xffffffffu, mu, off));
        }
        if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = mg; red[1][threadIdx.x >> 5] = mu; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < 8; ++w) { mg = fmaxf(mg, red[0][w]); mu = fmaxf(mu, red[1][w]); }
            wmax[c] = mg;
            wmax[n_cand + c] = mu;
        }
    }
}

// WdT[s][j] = Wd[j][channel(s)]: tile of 32 slots x 32 rows through shared memory
template <typename T>
__global__ void __launch_bounds__(1024) repack_wdt_kernel(const T* __restrict__ Wd, int d, int N, int n_rc,
                                                          int n_ret, const int32_t* __restrict__ idx_ret,
                                                          const int32_t* __restrict__ idx_cand,
                                                          T* __restrict__ WdT) {
    __shared__ T tile[32][33];
    const int s0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    int s = s0 + threadIdx.x, j = j0 + threadIdx.y;
    if (s < n_rc && j < d) {
        int ch = slot_channel(s, n_ret, idx_ret, idx_cand);
        tile[threadIdx.y][threadIdx.x] = Wd[(size_t)j * N + ch];
    }
    __syncthreads();
    s = s0 + threadIdx.y; j = j0 + threadIdx.x;
    if (s < n_rc && j < d) WdT[(size_t)s * d + j] = tile[threadIdx.x][threadIdx.y];
}

int pop_launch_repack(const pop_partition* p, const void* Wg, const void* Wu, const void* Wd,
                      const double* norm, cudaStream_t st) {
    if (p->n_rc > 0) {
        const int row_vecs = p->d * p->es / 16;
        repack_gu_kernel<<<p->n_rc, 256, 0, st>>>((const uint4*)Wg, (const uint4*)Wu, row_vecs, p->n_ret, p->n_cand,
                                                  p->idx_ret, p->idx_cand, (uint4*)p->GU, norm, p->norm_cand, nullptr);
        POP_LAUNCHED();
        dim3 blk(32, 32), grd((p->n_rc + 31) / 32, (p->d + 31) / 32);
        if (p->dtype == POP_F32)
            repack_wdt_kernel<float><<<grd, blk, 0, st>>>((const float*)Wd, p->d, p->N, p->n_rc, p->n_ret,
                                                          p->idx_ret, p->idx_cand, (float*)p->WdT);
        else
            repack_wdt_kernel<__nv_bfloat16><<<grd, blk, 0, st>>>((const __nv_bfloat16*)Wd, p->d, p->N, p->n_rc,
                                                                   p->n_ret, p->idx_ret, p->idx_cand,
                                                                   (__nv_bfloat16*)p->WdT);
        POP_LAUNCHED();
    }
    return POP_OK;
}

// ---------------------------------------------------------------------------------------------
// Repack into the tiled layout (see pop_common.cuh): the Retained rows as mma.m16n8k16 A
// fragments, the Candidate rows plain.  One thread writes one 16-byte fragment piece.
// ---------------------------------------------------------------------------------------------
// (tiles 0 .. n_rt - 1 hold the retained slots, tiles n_rt .. n_rt + n_ct - 1 the candidate slots)
__global__ void __launch_bounds__(256) repack_gut_kernel(const __nv_bfloat16* __restrict__ Wg,
                                                         const __nv_bfloat16* __restrict__ Wu, int d, int n_ret, int n_rt,
                                                         int n_cand, int n_ct, const int32_t* __restrict__ idx_ret,
                                                         const int32_t* __restrict__ idx_cand, uint4* __restrict__ GUt) {
    const int KT = d >> 4;
    const size_t total = (size_t)(n_rt + n_ct) * KT * 32;
    for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
        const int lane = (int)(o & 31);
        const size_t tile = o >> 5;
        const int kt = (int)(tile % KT), rt = (int)(tile / KT);
        const int g = lane >> 2, t = lane & 3;
        const bool cand = rt >= n_rt;
        const int slot = cand ? 8 * (rt - n_rt) + g : 8 * rt + g;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (slot < (cand ? n_cand : n_ret)) {
            const int ch = cand ? idx_cand[slot] : idx_ret[slot];
            const u32* gp = reinterpret_cast<const u32*>(Wg + (size_t)ch * d + (size_t)kt * 16);
            const u32* up = reinterpret_cast<const u32*>(Wu + (size_t)ch * d + (size_t)kt * 16);
            v.x = gp[t];        // row g     (gate), columns 2t, 2t+1
            v.y = up[t];        // row g + 8 (up),   columns 2t, 2t+1
            v.z = gp[t + 4];    // row g,     columns 2t+8, 2t+9
            v.w = up[t + 4];    // row g + 8, columns 2t+8, 2t+9
        }
        GUt[o] = v;
    }
}

__global__ void __launch_bounds__(256) repack_wdtt_kernel(const __nv_bfloat16* __restrict__ Wd, int d, int N,
                                                          int n_ret, int n_cg, const int32_t* __restrict__ idx_ret,
                                                          uint4* __restrict__ WdTt) {
    const int MT = d >> 6;                                   // m-tiles per quarter
    const size_t total = (size_t)4 * n_cg * MT * 32;
    const unsigned short* W = reinterpret_cast<const unsigned short*>(Wd);
    for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
        const int lane = (int)(o & 31);
        size_t tile = o >> 5;
        const int mt = (int)(tile % MT); tile /= MT;
        const int cg = (int)(tile % n_cg);
        const int q = (int)(tile / n_cg);
        const int g = lane >> 2, t = lane & 3;
        const int j0 = q * (d >> 2) + mt * 16 + g;           // output row of A rows g (and g + 8)
        u32 r[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = j0 + ((e & 1) ? 8 : 0);
            const int s0 = 16 * cg + 2 * t + ((e >> 1) ? 8 : 0);
            u32 lo = 0, hi = 0;
            if (s0 < n_ret) lo = W[(size_t)j * N + idx_ret[s0]];
            if (s0 + 1 < n_ret) hi = W[(size_t)j * N + idx_ret[s0 + 1]];
            r[e] = lo | (hi << 16);
        }
        WdTt[o] = make_uint4(r[0], r[1], r[2], r[3]);
    }
}

// ---------------------------------------------------------------------------------------------
// Both W_d outputs of the tiled layout in one pass over W_d: the retained fragments WdTt and the plain candidate rows
// WdTc.  Block (sg, jc) stages W_d[64 jc .. + 63][c_lo .. c_hi) in shared memory with coalesced 16-byte loads, where
// [c_lo, c_hi) is the span of channel ids from the first retained slot of slot group sg (128 retained slots) up to the
// first slot of the next group (the spans tile [0, N), so every candidate lies in exactly one of them), and builds
// from it the 8 x 4 fragment tiles of its slots and the 64-row pieces of the candidates inside the span.  W_d is read
// once (the pruned columns inside a span ride along); the former per-element column gathers from global memory cost
// twice the time.  A span too wide for the staging buffer (very sparse retained regions) is read from global memory
// directly, element by element, by the same code.
// ---------------------------------------------------------------------------------------------
#define RWD_ROWS 64
#define RWD_SLOTS 128
#define RWD_SPAN_MAX 512

// rows of the staged tile start 16 bytes aligned and an odd number of 16-byte units apart (8 rows fall on 8 bank groups)
__host__ __device__ __forceinline__ int rwd_pitch_vec(int nvec) { return (nvec + 1) | 1; }

template <bool STAGED>
__device__ __forceinline__ void rwd_emit(const unsigned short* __restrict__ W, const unsigned short* tile, int pitch,
                                         int c_lo8, int j0, int d, int N, int n_cg, int sg, const int* slot_ch,
                                         int ca, int cb, const int32_t* __restrict__ idx_cand, uint4* __restrict__ WdTt,
                                         __nv_bfloat16* __restrict__ WdTc) {
    const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
    // element (row jl of the block, channel offset off) of W_d
    auto rd = [&](int jl, int off) -> u32 {
        return STAGED ? (u32)tile[jl * pitch + off] : (u32)W[(size_t)(j0 + jl) * N + c_lo8 + off];
    };
    // retained fragments: warp = column group (16 slots), 4 m-tiles of 16 rows each, one 16-byte vector per lane and tile
    const int cg8 = tid >> 5, cg = 8 * sg + cg8;
    if (cg < n_cg) {
        int off[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int ch = slot_ch[16 * cg8 + 2 * t + (h & 1) + ((h >> 1) ? 8 : 0)];
            off[h] = ch < 0 ? -1 : ch - c_lo8;
        }
        const int MT = d >> 6, quarter_rows = d >> 2;
        const int q = j0 / quarter_rows, mt0 = (j0 - q * quarter_rows) >> 4;
        uint4* out = WdTt + (((size_t)q * n_cg + cg) * MT + mt0) * 32 + lane;
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            u32 r[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int jl = 16 * mt + g + ((e & 1) ? 8 : 0);
                const int oa = off[2 * (e >> 1)], ob = off[2 * (e >> 1) + 1];
                const u32 lo = oa >= 0 ? rd(jl, oa) : 0u, hi = ob >= 0 ? rd(jl, ob) : 0u;
                r[e] = lo | (hi << 16);
            }
            out[mt * 32] = make_uint4(r[0], r[1], r[2], r[3]);
        }
    }
    // candidate rows inside the span: 8 pieces of 8 rows each
    for (int w = tid; w < (cb - ca) * 8; w += 256) {
        const int c = ca + (w >> 3), rv = w & 7;
        const int off = __ldg(idx_cand + c) - c_lo8;
        u32 o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = rd(8 * rv + 2 * e, off) | (rd(8 * rv + 2 * e + 1, off) << 16);
        *reinterpret_cast<uint4*>(WdTc + (size_t)c * d + j0 + 8 * rv) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

__global__ void __launch_bounds__(256, 5) repack_wd_tiled_kernel(const __nv_bfloat16* __restrict__ Wd, int d, int N, int n_ret,
                                                              int n_cg, int n_cand, int span_cap, const int32_t* __restrict__ idx_ret,
                                                              const int32_t* __restrict__ idx_cand, uint4* __restrict__ WdTt,
                                                              __nv_bfloat16* __restrict__ WdTc) {
    extern __shared__ __align__(16) unsigned short rwd_tile[];     // [RWD_ROWS][pitch]
    __shared__ int slot_ch[RWD_SLOTS];
    __shared__ int span[2];                                        // first and last + 1 candidate of the span
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, sg = blockIdx.x, j0 = blockIdx.y * RWD_ROWS;
    const int n_sg = gridDim.x;
    const unsigned short* W = reinterpret_cast<const unsigned short*>(Wd);
    if (tid < RWD_SLOTS) {
        const int s = RWD_SLOTS * sg + tid;
        slot_ch[tid] = s < n_ret ? idx_ret[s] : -1;
    }
    if (tid < 2) span[tid] = 0;
    const int c_lo = sg == 0 ? 0 : __ldg(idx_ret + RWD_SLOTS * sg);
    const int c_hi = sg == n_sg - 1 ? N : __ldg(idx_ret + RWD_SLOTS * (sg + 1));
    const int c_lo8 = c_lo & ~7;
    const int nvec = (c_hi - c_lo8 + 7) >> 3;                       // 16-byte vectors per staged row (N is a multiple of 8)
    const bool staged = nvec * 8 <= span_cap + 8;      // the launch sized the staging buffer for spans of span_cap channels
    const int pitch = 8 * rwd_pitch_vec(nvec);
    __syncthreads();
    if (staged) {
        // a warp per row, lanes along the row: every load of a warp is one contiguous run
        const uint4* src = reinterpret_cast<const uint4*>(W + (size_t)(j0 + warp) * N + c_lo8) + lane;
        uint4* dst = reinterpret_cast<uint4*>(rwd_tile + warp * pitch) + lane;
        const size_t src_step = (size_t)N;                          // 8 rows, in 16-byte units
        const int dst_step = pitch;
        if (nvec <= 32) {
            uint4 x[RWD_ROWS / 8];
            if (lane < nvec) {
#pragma unroll
                for (int i = 0; i < RWD_ROWS / 8; ++i) x[i] = __ldg(src + i * src_step);
#pragma unroll
                for (int i = 0; i < RWD_ROWS / 8; ++i) dst[i * dst_step] = x[i];
            }
        } else {
            for (int cv = lane; cv < nvec; cv += 32) {
                uint4 x[RWD_ROWS / 8];
#pragma unroll
                for (int i = 0; i < RWD_ROWS / 8; ++i) x[i] = __ldg(src + i * src_step + (cv - lane));
#pragma unroll
                for (int i = 0; i < RWD_ROWS / 8; ++i) dst[i * dst_step + (cv - lane)] = x[i];
            }
        }
    }
    {   // candidates below the span and below its end, counted by all threads (independent loads, one latency)
        int below_lo = 0, below_hi = 0;
        for (int i = tid; i < n_cand; i += 256) {
            const int v = __ldg(idx_cand + i);
            below_lo += v < c_lo; below_hi += v < c_hi;
        }
        below_lo = __reduce_add_sync(0xffffffffu, below_lo); below_hi = __reduce_add_sync(0xffffffffu, below_hi);
        if (lane == 0) { atomicAdd(&span[0], below_lo); atomicAdd(&span[1], below_hi); }
    }
    __syncthreads();
    const int ca = span[0], cb = span[1];
    if (staged) rwd_emit<true>(W, rwd_tile, pitch, c_lo8, j0, d, N, n_cg, sg, slot_ch, ca, cb, idx_cand, WdTt, WdTc);
    else rwd_emit<false>(W, rwd_tile, pitch, c_lo8, j0, d, N, n_cg, sg, slot_ch, ca, cb, idx_cand, WdTt, WdTc);
}

static bool repack_wd_tiled_applies(const pop_partition* p) {
    return p->n_ret > 0 && p->N % 8 == 0 && p->d % (4 * RWD_ROWS) == 0;
}

int pop_launch_repack_tiled(const pop_partition* p, const void* Wg, const void* Wu, const void* Wd,
                            const double* norm, cudaStream_t st) {
    const size_t row = (size_t)p->d * 2;
    unsigned char* GUt = (unsigned char*)p->GU;
    unsigned char* GUc = GUt + (size_t)(p->n_rt + p->n_ct) * 16 * row;  // candidate rows
    unsigned char* WdTt = (unsigned char*)p->WdT;
    unsigned char* WdTc = WdTt + (size_t)p->n_ret_pad * row;
    if (p->n_rt + p->n_ct > 0) {
        const size_t total = (size_t)(p->n_rt + p->n_ct) * (p->d / 16) * 32;
        const int blocks = (int)((total + 255) / 256 < 148 * 64 ? (total + 255) / 256 : 148 * 64);
        repack_gut_kernel<<<blocks, 256, 0, st>>>((const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu, p->d, p->n_ret, p->n_rt,
                                                  p->n_cand, p->n_ct, p->idx_ret, p->idx_cand, (uint4*)GUt);
        POP_LAUNCHED();
    }
    const bool merged = repack_wd_tiled_applies(p);
    if (merged) {
        // The staging buffer is sized for spans a quarter wider than the average one (128 N / n_ret channels), at most
        // RWD_SPAN_MAX: a smaller buffer lets more blocks share an SM, and the kernel is bound by latency.
        long long cap = ((long long)RWD_SLOTS * p->N * 5 / 4) / p->n_ret + 16;
        int span_cap = (int)((cap + 7) / 8 * 8);
        if (span_cap > RWD_SPAN_MAX) span_cap = RWD_SPAN_MAX;
        const size_t smem = sizeof(unsigned short) * RWD_ROWS * 8 * rwd_pitch_vec(span_cap / 8 + 1);
        static thread_local int cfg_dev = -1;
        int dev = 0;
        POP_CUDA(cudaGetDevice(&dev));
        if (cfg_dev != dev) {
            const size_t smem_max = sizeof(unsigned short) * RWD_ROWS * 8 * rwd_pitch_vec(RWD_SPAN_MAX / 8 + 1);
            POP_CUDA(cudaFuncSetAttribute(repack_wd_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
            cfg_dev = dev;
        }
        dim3 grd((p->n_ret + RWD_SLOTS - 1) / RWD_SLOTS, p->d / RWD_ROWS);
        repack_wd_tiled_kernel<<<grd, 256, smem, st>>>((const __nv_bfloat16*)Wd, p->d, p->N, p->n_ret, p->n_cg, p->n_cand, span_cap,
                                                       p->idx_ret, p->idx_cand, (uint4*)WdTt, (__nv_bfloat16*)WdTc);
        POP_LAUNCHED();
    } else if (p->n_rt > 0) {
        const size_t total2 = (size_t)4 * p->n_cg * (p->d / 64) * 32;
        const int blocks2 = (int)((total2 + 255) / 256 < 148 * 64 ? (total2 + 255) / 256 : 148 * 64);
        repack_wdtt_kernel<<<blocks2, 256, 0, st>>>((const __nv_bfloat16*)Wd, p->d, p->N, p->n_ret, p->n_cg,
                                                    p->idx_ret, (uint4*)WdTt);
        POP_LAUNCHED();
    }
    if (p->n_cand > 0) {
        const int row_vecs = (int)(row / 16);
        repack_gu_kernel<<<p->n_cand, 256, 0, st>>>((const uint4*)Wg, (const uint4*)Wu, row_vecs, 0, p->n_cand, p->idx_cand,
                                                    p->idx_cand, (uint4*)GUc, norm, p->norm_cand, p->wnorm_cand);
        POP_LAUNCHED();
        if (!merged) {
            dim3 blk(32, 32), grd((p->n_cand + 31) / 32, (p->d + 31) / 32);
            repack_wdt_kernel<__nv_bfloat16><<<grd, blk, 0, st>>>((const __nv_bfloat16*)Wd, p->d, p->N, p->n_cand, 0,
                                                                   p->idx_cand, p->idx_cand, (__nv_bfloat16*)WdTc);
            POP_LAUNCHED();
        }
    }
    return POP_OK;
}
