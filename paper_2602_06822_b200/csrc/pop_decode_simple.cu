// Decoding step of POP, plain multi-kernel version (Sec. 3.3 "Decoding Stage", Sec. 3.4):
//   1. gate/up rows of Retained + Candidate slots, activation, candidate scores
//   2. exact top-k among the candidate scores
//   3. down projection over Retained + selected rows
//   4. cast of the fp32 accumulator to the output dtype
// It handles every shape the library accepts and serves as the path for shapes the fused
// persistent kernel (pop_decode.cu) does not take.
#include "pop_common.cuh"
#include "pop_select.cuh"

// ---------------------------------------------------------------------------------------------
// 1. one warp per slot.  Retained slots accumulate in fp32; Candidate slots accumulate in fp64
//    because their scores decide the mask.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) gateup_simple_kernel(const uint4* __restrict__ GU, const uint4* __restrict__ x,
                                                            int B, int row_vecs, int n_ret, int n_rc,
                                                            const double* __restrict__ norm_cand,
                                                            float* __restrict__ h, u64* __restrict__ keys) {
    constexpr int VEC = Elem<T>::VEC;
    const int lane = threadIdx.x & 31;
    const int slot = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (slot >= n_rc) return;
    const uint4* gr = GU + (size_t)slot * 2 * row_vecs;
    const uint4* ur = gr + row_vecs;
    const bool cand = slot >= n_ret;
    double energy = 0.0;
    for (int b = 0; b < B; ++b) {
        const uint4* xb = x + (size_t)b * row_vecs;
        double hv;
        if (cand) {
            double ag = 0.0, au = 0.0;
            for (int v = lane; v < row_vecs; v += 32) {
                float fg[VEC], fu[VEC], fx[VEC];
                Elem<T>::unpack(gr[v], fg); Elem<T>::unpack(ur[v], fu); Elem<T>::unpack(xb[v], fx);
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    double xd = (double)fx[j];
                    ag = fma((double)fg[j], xd, ag);
                    au = fma((double)fu[j], xd, au);
                }
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) {
                ag += __shfl_xor_sync(0xffffffffu, ag, off);
                au += __shfl_xor_sync(0xffffffffu, au, off);
            }
            hv = silu_f64(ag) * au;
        } else {
            float ag = 0.f, au = 0.f;
            for (int v = lane; v < row_vecs; v += 32) {
                float fg[VEC], fu[VEC], fx[VEC];
                Elem<T>::unpack(gr[v], fg); Elem<T>::unpack(ur[v], fu); Elem<T>::unpack(xb[v], fx);
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    ag = fmaf(fg[j], fx[j], ag);
                    au = fmaf(fu[j], fx[j], au);
                }
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) {
                ag += __shfl_xor_sync(0xffffffffu, ag, off);
                au += __shfl_xor_sync(0xffffffffu, au, off);
            }
            hv = (double)(silu_f32(ag) * au);
        }
        if (lane == 0) h[(size_t)b * n_rc + slot] = (float)hv;
        energy = fma(hv, hv, energy);
    }
    if (cand && lane == 0) keys[slot - n_ret] = score_key(norm_cand[slot - n_ret] * sqrt(energy));
}

// ---------------------------------------------------------------------------------------------
// 2. top-k among the candidate keys (one block)
// ---------------------------------------------------------------------------------------------
#define SEL_NT 1024
__global__ void __launch_bounds__(SEL_NT) select_simple_kernel(const u64* __restrict__ keys, int n_cand, int k,
                                                               const int32_t* __restrict__ idx_cand,
                                                               int32_t* __restrict__ sel_slots,
                                                               uint8_t* __restrict__ mask_out,
                                                               int32_t* __restrict__ sel_out) {
    __shared__ u32 sm[POP_SELECT_SMEM_WORDS(SEL_NT)];
    const int tid = threadIdx.x;
    u64 thr = ~0ull;
    int need = 0;
    if (k > 0) radix_select_kth<SEL_NT>(keys, n_cand, k, sm, tid, 0, thr, need);
    select_walk<SEL_NT>(keys, n_cand, thr, need, sm, tid, 0, [&](int i, bool s, int pos) {
        if (mask_out) mask_out[i] = s ? 1 : 0;
        if (s) {
            sel_slots[pos] = i;
            if (sel_out) sel_out[pos] = idx_cand[i];
        }
    });
}

// ---------------------------------------------------------------------------------------------
// 3. y_acc[b][:] += sum over this block's rows of h[b][slot] * WdT[slot][:]
//    rows: Retained slots 0..n_ret-1, then n_ret + sel_slots[0..k-1]
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) down_simple_kernel(const uint4* __restrict__ WdT, const float* __restrict__ h,
                                                          const int32_t* __restrict__ sel_slots, int B, int d,
                                                          int row_vecs, int n_ret, int n_rc, int k, int rows_per_block,
                                                          float* __restrict__ y_acc) {
    constexpr int VEC = Elem<T>::VEC;
    const int n_act = n_ret + k;
    const int r0 = blockIdx.x * rows_per_block, r1 = min(n_act, r0 + rows_per_block);
    for (int v = threadIdx.x; v < row_vecs; v += blockDim.x) {
        for (int b = 0; b < B; ++b) {
            float acc[VEC];
#pragma unroll
            for (int j = 0; j < VEC; ++j) acc[j] = 0.f;
            for (int r = r0; r < r1; ++r) {
                const int slot = r < n_ret ? r : n_ret + sel_slots[r - n_ret];
                const float hv = h[(size_t)b * n_rc + slot];
                float w[VEC];
                Elem<T>::unpack(WdT[(size_t)slot * row_vecs + v], w);
#pragma unroll
                for (int j = 0; j < VEC; ++j) acc[j] = fmaf(hv, w[j], acc[j]);
            }
#pragma unroll
            for (int j = 0; j < VEC; ++j) atomicAdd(&y_acc[(size_t)b * d + v * VEC + j], acc[j]);
        }
    }
}

// 4. y = cast(y_acc); y_acc = 0 for the next step
template <typename T>
__global__ void finalize_simple_kernel(float* __restrict__ y_acc, T* __restrict__ y, int n) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { y[i] = Elem<T>::from_f32(y_acc[i]); y_acc[i] = 0.f; }
}

template <typename T>
static int decode_simple_t(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                           int32_t* sel_out, cudaStream_t st) {
    const int row_vecs = p->d * p->es / 16;
    if (p->n_rc > 0) {
        gateup_simple_kernel<T><<<(p->n_rc + 7) / 8, 256, 0, st>>>((const uint4*)p->GU, (const uint4*)x, B, row_vecs,
                                                                  p->n_ret, p->n_rc, p->norm_cand, p->h, p->keys);
        POP_LAUNCHED();
    }
    if (p->n_cand > 0) {
        select_simple_kernel<<<1, SEL_NT, 0, st>>>(p->keys, p->n_cand, k, p->idx_cand, p->sel_slots, mask_out, sel_out);
        POP_LAUNCHED();
    }
    const int n_act = p->n_ret + k;
    if (n_act > 0) {
        const int rpb = 16;
        down_simple_kernel<T><<<(n_act + rpb - 1) / rpb, 256, 0, st>>>((const uint4*)p->WdT, p->h, p->sel_slots, B, p->d,
                                                                       row_vecs, p->n_ret, p->n_rc, k, rpb, p->y_acc);
        POP_LAUNCHED();
    }
    finalize_simple_kernel<T><<<(B * p->d + 255) / 256, 256, 0, st>>>(p->y_acc, (T*)y, B * p->d);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_decode_simple(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                             int32_t* sel_out, cudaStream_t st) {
    if (p->dtype == POP_F32) return decode_simple_t<float>(p, x, B, k, y, mask_out, sel_out, st);
    return decode_simple_t<__nv_bfloat16>(p, x, B, k, y, mask_out, sel_out, st);
}
