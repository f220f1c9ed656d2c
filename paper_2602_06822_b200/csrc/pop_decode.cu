// Fused decode step of POP (Sec. 3.3 "Decoding Stage", Sec. 3.4) as ONE persistent cooperative
// kernel: one CTA per SM, weights streamed through a shared-memory ring by bulk asynchronous
// copies (TMA engine, mbarrier completion), one grid-wide barrier between the two projections.
//
//   phase 1  gate/up rows of the Retained + Candidate slots -> h = silu(g) * u, candidate scores
//            (tiles of TC slots, tile t handled by CTA t mod G, so that the CTAs read one
//            contiguous window of HBM at any time and the fp64 candidate rows are spread evenly)
//   barrier  every CTA has published its h values and candidate keys
//   phase 2  y += h_i * WdT[i, :] over the Retained rows (known before the barrier: the producer
//            keeps prefetching them into the ring while the CTA waits) and over the k selected
//            Candidate rows; the selection (exact radix top-k on fp64 scores) is computed
//            redundantly per CTA by four otherwise idle warps while the Retained rows stream.
//   finish   partial y vectors are added into an fp32 accumulator with vector reductions at L2;
//            the CTA that finishes last casts it to the output dtype and re-arms the counters.
//
// Warp roles: warps [0, ncw) consumers, warp ncw producer (one elected lane), then 4 selector warps.
// In phase 1 every consumer warp owns a fixed set of 16-byte column chunks of every row (x for
// those columns lives in registers); the per-row partial dot products of the warps are combined
// at the end of the phase in a fixed order (bit-reproducible; equal rows give equal results).
// In phase 2 the same column ownership makes each lane the owner of fixed output columns.
//
// Every wait (mbarrier, grid barrier) is bounded: when a limit expires the kernel raises
// sync[SYNC_ERROR], stops issuing copies, drains the copies in flight and returns.
#include "pop_common.cuh"
#include <stdlib.h>
#include <string.h>

#include "pop_select.cuh"

namespace {

constexpr int SEL_NT = 128;                 // selector threads (4 warps)
constexpr int STAGE_TARGET = 32 * 1024;     // bytes per ring stage aimed for
constexpr int KEYS_SMEM_MAX = 4096;         // candidate keys kept in shared memory up to this many

enum { ERR_MBAR_FULL = 1, ERR_MBAR_EMPTY = 2, ERR_GRID_BARRIER = 3, ERR_SELECT = 4 };

struct DecodeParams {
    const unsigned char* GU;
    const unsigned char* WdT;
    const void* x;
    void* y;
    const double* norm_cand;
    const int32_t* idx_cand;
    float* h;
    u64* keys;
    float* y_acc;
    u32* sync;
    uint8_t* mask_out;
    int32_t* sel_out;
    int d, n_ret, n_cand, n_rc, k, B;
    int row_bytes, TC, TR, nstage, stage_bytes;
    int T1, T2r, T2c;
    int ncw, MC, MCC, capr, capc, keys_in_smem;
    int off_x, off_pf, off_pd, off_h2, off_mysel, off_keys, off_selsm, off_bars;
    unsigned long long wait_ns;    // budget of every device-side wait
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 smem_u32(const void* p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u32 bar, u32 count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u32 bar, u32 bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u32 bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u32 bar, u32 parity) {
    u32 ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ u64 make_evict_first_policy() {
    u64 pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// Bulk asynchronous copy global -> this CTA's shared memory; completion is counted in bytes on `bar`.
// dst, src and bytes are multiples of 16.
__device__ __forceinline__ void bulk_g2s(u32 dst, const void* src, u32 bytes, u32 bar, u64 pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ u32 ld_acquire_gpu(const u32* p) {
    u32 v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ uint4 lds128(u32 addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void named_bar(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Bounded mbarrier wait.  Returns false (and raises the error flags) when it gives up.
__device__ __forceinline__ bool mbar_wait(u32 bar, u32 parity, volatile int* abort_flag, u32* gerr, int code,
                                          unsigned long long wait_ns) {
    PopWaitClock spins;
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (spins.expired(wait_ns)) {
            *abort_flag = 1;
            atomicExch(gerr, (u32)code);
            return false;
        }
    }
    return true;
}

// Bounded wait until *counter >= target (grid barrier).
__device__ __forceinline__ bool grid_wait(const u32* counter, u32 target, volatile int* abort_flag, u32* gerr,
                                          unsigned long long wait_ns) {
    PopWaitClock spins;
    while (ld_acquire_gpu(counter) < target) {
        if (*abort_flag) return false;
        if (spins.expired(wait_ns)) {
            *abort_flag = 1;
            atomicExch(gerr, (u32)ERR_GRID_BARRIER);
            return false;
        }
        __nanosleep(64);
    }
    return true;
}

template <int NV>
__device__ __forceinline__ void warp_allreduce(float (&v)[NV]) {
#pragma unroll
    for (int off = 16; off; off >>= 1)
#pragma unroll
        for (int i = 0; i < NV; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], off);
}
template <int NV>
__device__ __forceinline__ void warp_allreduce(double (&v)[NV]) {
#pragma unroll
    for (int off = 16; off; off >>= 1)
#pragma unroll
        for (int i = 0; i < NV; ++i) v[i] += __shfl_xor_sync(0xffffffffu, v[i], off);
}

// ---------------------------------------------------------------------------------------------
// The kernel.  T element type, BT batch capacity of this instantiation (B <= BT), CPW column
// chunks (of 32 lanes x 16 bytes) owned by each consumer warp.
// ---------------------------------------------------------------------------------------------
template <typename T, int BT, int CPW>
__global__ void __launch_bounds__(672, 1) pop_decode_fused_kernel(const DecodeParams P) {
    constexpr int VEC = Elem<T>::VEC;
    constexpr int ES = (int)sizeof(T);
    constexpr bool IS_BF16 = (ES == 2);
    extern __shared__ __align__(128) unsigned char smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, G = gridDim.x;
    const int ncw = P.ncw, NTC = ncw * 32;              // consumer threads
    const int d = P.d, n_ret = P.n_ret, n_rc = P.n_rc, TC = P.TC, TR = P.TR, B = P.B;

    unsigned char* ring = smem;
    T* xs = reinterpret_cast<T*>(smem + P.off_x);                 // [BT][d]
    float* pf = reinterpret_cast<float*>(smem + P.off_pf);        // [MC][2][BT][ncw]
    double* pd = reinterpret_cast<double*>(smem + P.off_pd);      // [MCC][2][BT][ncw]
    float* h2 = reinterpret_cast<float*>(smem + P.off_h2);        // [(capr + capc)][BT]
    int* mysel = reinterpret_cast<int*>(smem + P.off_mysel);      // [capc] candidate slots of this CTA's tiles
    u64* keys_s = reinterpret_cast<u64*>(smem + P.off_keys);
    u32* selsm = reinterpret_cast<u32*>(smem + P.off_selsm);
    u64* bars = reinterpret_cast<u64*>(smem + P.off_bars);        // full[nstage], empty[nstage], selbar
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * P.nstage + 1);
    volatile int* last_flag = abort_flag + 1;
    const u32 full0 = smem_u32(bars), empty0 = smem_u32(bars + P.nstage), selbar = smem_u32(bars + 2 * P.nstage);
    u32* gerr = P.sync + SYNC_ERROR;

    // this CTA's share of the three tile sequences
    const int n1 = cta < P.T1 ? (P.T1 - cta + G - 1) / G : 0;
    const int j0r = ((cta - P.T1) % G + G) % G;
    const int n2r = j0r < P.T2r ? (P.T2r - j0r + G - 1) / G : 0;
    const int j0c = ((cta - P.T1 - P.T2r) % G + G) % G;
    const int n2c = j0c < P.T2c ? (P.T2c - j0c + G - 1) / G : 0;

    if (tid == 0) {
        for (int s = 0; s < P.nstage; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, (u32)ncw);
        }
        mbar_init(selbar, 1);
        *abort_flag = 0;
        *last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // x -> shared memory (rows b >= B are zero)
    {
        const int vec_per_row = d / VEC;
        const uint4* xg = reinterpret_cast<const uint4*>(P.x);
        uint4* xv = reinterpret_cast<uint4*>(xs);
        for (int i = tid; i < BT * vec_per_row; i += blockDim.x) {
            int b = i / vec_per_row;
            xv[i] = b < B ? xg[i] : make_uint4(0, 0, 0, 0);
        }
    }
    __syncthreads();

    if (warp == ncw) {
        // ===================================================================== producer
        if (lane == 0) {
            const u64 pol = make_evict_first_policy();
            const u32 ring_u = smem_u32(ring);
            int n = 0;
            bool ok = true;
            for (int i = 0; i < n1 && ok; ++i, ++n) {
                const int s = n % P.nstage, use = n / P.nstage;
                ok = mbar_wait(empty0 + 8 * s, (use & 1) ^ 1, abort_flag, gerr, ERR_MBAR_EMPTY, P.wait_ns);
                if (!ok) break;
                const int ch0 = (cta + i * G) * TC;
                const int nch = min(TC, n_rc - ch0);
                const u32 bytes = (u32)nch * 2u * (u32)P.row_bytes;
                mbar_expect_tx(full0 + 8 * s, bytes);
                bulk_g2s(ring_u + s * P.stage_bytes, P.GU + (size_t)ch0 * 2 * P.row_bytes, bytes, full0 + 8 * s, pol);
            }
            for (int i = 0; i < n2r && ok; ++i, ++n) {
                const int s = n % P.nstage, use = n / P.nstage;
                ok = mbar_wait(empty0 + 8 * s, (use & 1) ^ 1, abort_flag, gerr, ERR_MBAR_EMPTY, P.wait_ns);
                if (!ok) break;
                const int r0 = (j0r + i * G) * TR;
                const int nr = min(TR, n_ret - r0);
                const u32 bytes = (u32)nr * (u32)P.row_bytes;
                mbar_expect_tx(full0 + 8 * s, bytes);
                bulk_g2s(ring_u + s * P.stage_bytes, P.WdT + (size_t)r0 * P.row_bytes, bytes, full0 + 8 * s, pol);
            }
            if (n2c > 0 && ok) ok = mbar_wait(selbar, 0, abort_flag, gerr, ERR_SELECT, P.wait_ns);
            for (int i = 0; i < n2c && ok; ++i, ++n) {
                const int s = n % P.nstage, use = n / P.nstage;
                ok = mbar_wait(empty0 + 8 * s, (use & 1) ^ 1, abort_flag, gerr, ERR_MBAR_EMPTY, P.wait_ns);
                if (!ok) break;
                const int p0 = (j0c + i * G) * TR;
                const int nr = min(TR, P.k - p0);
                mbar_expect_tx(full0 + 8 * s, (u32)nr * (u32)P.row_bytes);
                for (int r = 0; r < nr; ++r) {
                    const int slot = n_ret + mysel[i * TR + r];
                    bulk_g2s(ring_u + s * P.stage_bytes + r * P.row_bytes, P.WdT + (size_t)slot * P.row_bytes,
                             (u32)P.row_bytes, full0 + 8 * s, pol);
                }
            }
            if (*abort_flag) {
                // drain: every stage this thread filled must have landed before the CTA may exit
                for (int m = max(0, n - P.nstage); m < n; ++m) {
                    const int s = m % P.nstage, use = m / P.nstage;
                    PopWaitClock spins;
                    while (!mbar_try_wait(full0 + 8 * s, use & 1) && !spins.expired(P.wait_ns)) {}
                }
            }
        }
    } else if (warp > ncw) {
        // ===================================================================== selectors
        const int st = tid - (ncw + 1) * 32;                   // 0..127
        const bool need = P.n_cand > 0 && (n2c > 0 || (cta == 0 && (P.mask_out || P.sel_out)));
        if (need) {
            bool ok = true;
            if (P.k > 0) {
                if (st == 0) ok = grid_wait(P.sync + SYNC_BARRIER, (u32)G, abort_flag, gerr, P.wait_ns);
                group_sync<SEL_NT>(2);
                ok = !*abort_flag;
            }
            if (ok) {
                u64 thr = ~0ull;
                int need_eq = 0;
                const u64* keys = P.keys;
                if (P.k > 0) {
                    if (P.keys_in_smem) {
                        for (int i = st; i < P.n_cand; i += SEL_NT) keys_s[i] = __ldcg(P.keys + i);
                        keys = keys_s;
                        group_sync<SEL_NT>(2);
                    }
                    radix_select_kth<SEL_NT>(keys, P.n_cand, P.k, selsm, st, 2, thr, need_eq);
                }
                const bool write_out = cta == 0;
                const int shift = P.T1 + P.T2r;
                select_walk<SEL_NT>(keys, P.n_cand, thr, need_eq, selsm, st, 2, [&](int i, bool s, int pos) {
                    if (write_out && P.mask_out) P.mask_out[i] = s ? 1 : 0;
                    if (s) {
                        if (write_out && P.sel_out) P.sel_out[pos] = P.idx_cand[i];
                        const int tile = pos / TR;
                        if ((tile + shift) % G == cta) mysel[((tile - j0c) / G) * TR + (pos - tile * TR)] = i;
                    }
                });
            }
            __threadfence_block();
            group_sync<SEL_NT>(2);
            if (st == 0) mbar_arrive(selbar);
        }
    } else {
        // ===================================================================== consumers
        const int tc = tid;                                     // consumer thread id, 0..NTC-1
        bool ok = true;
        int n = 0;
        // columns owned by this lane: chunk c covers elements [(c*ncw + warp)*32*VEC + lane*VEC, +VEC)
        int col[CPW];
        bool colok[CPW];
#pragma unroll
        for (int c = 0; c < CPW; ++c) {
            col[c] = ((c * ncw + warp) * 32 + lane) * VEC;
            colok[c] = col[c] < d;
        }
        // x of the owned columns, in registers
        float xr[CPW][BT][VEC];
#pragma unroll
        for (int c = 0; c < CPW; ++c)
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                if (colok[c]) {
                    uint4 v = *reinterpret_cast<const uint4*>(xs + (size_t)b * d + col[c]);
                    Elem<T>::unpack(v, xr[c][b]);
                } else {
#pragma unroll
                    for (int j = 0; j < VEC; ++j) xr[c][b][j] = 0.f;
                }
            }

        // ------------------------------------------------------------------ phase 1
        const int tcand0 = n_ret / TC;                          // first tile that holds a candidate slot
        const int i_first = tcand0 <= cta ? 0 : (tcand0 - cta + G - 1) / G;
        const u32 ring_u = smem_u32(ring);
        for (int i = 0; i < n1; ++i, ++n) {
            const int s = n % P.nstage, use = n / P.nstage;
            if (ok) ok = mbar_wait(full0 + 8 * s, use & 1, abort_flag, gerr, ERR_MBAR_FULL, P.wait_ns);
            if (!ok) break;
            const int ch0 = (cta + i * G) * TC;
            const int nch = min(TC, n_rc - ch0);
            const u32 base = ring_u + s * P.stage_bytes;
            for (int j = 0; j < nch; ++j) {
                const int slot = ch0 + j;
                const u32 grow = base + (u32)(2 * j) * P.row_bytes, urow = grow + P.row_bytes;
                const int lc = i * TC + j;
                if (slot < n_ret) {
                    float acc[2 * BT];
#pragma unroll
                    for (int q = 0; q < 2 * BT; ++q) acc[q] = 0.f;
#pragma unroll
                    for (int c = 0; c < CPW; ++c) {
                        if (colok[c]) {
                            float wg[VEC], wu[VEC];
                            Elem<T>::unpack(lds128(grow + col[c] * ES), wg);
                            Elem<T>::unpack(lds128(urow + col[c] * ES), wu);
#pragma unroll
                            for (int b = 0; b < BT; ++b)
#pragma unroll
                                for (int v = 0; v < VEC; ++v) {
                                    acc[b] = fmaf(wg[v], xr[c][b][v], acc[b]);
                                    acc[BT + b] = fmaf(wu[v], xr[c][b][v], acc[BT + b]);
                                }
                        }
                    }
                    warp_allreduce<2 * BT>(acc);
                    if (lane == 0) {
#pragma unroll
                        for (int b = 0; b < BT; ++b) {
                            pf[((lc * 2 + 0) * BT + b) * ncw + warp] = acc[b];
                            pf[((lc * 2 + 1) * BT + b) * ncw + warp] = acc[BT + b];
                        }
                    }
                } else {
                    double acc[2 * BT];
#pragma unroll
                    for (int q = 0; q < 2 * BT; ++q) acc[q] = 0.0;
#pragma unroll
                    for (int c = 0; c < CPW; ++c) {
                        if (colok[c]) {
                            float wg[VEC], wu[VEC];
                            Elem<T>::unpack(lds128(grow + col[c] * ES), wg);
                            Elem<T>::unpack(lds128(urow + col[c] * ES), wu);
#pragma unroll
                            for (int b = 0; b < BT; ++b)
#pragma unroll
                                for (int v = 0; v < VEC; ++v) {
                                    if (IS_BF16) {
                                        // a product of two bf16 values is exact in fp32
                                        acc[b] += (double)(wg[v] * xr[c][b][v]);
                                        acc[BT + b] += (double)(wu[v] * xr[c][b][v]);
                                    } else {
                                        const double xd = (double)xr[c][b][v];
                                        acc[b] = fma((double)wg[v], xd, acc[b]);
                                        acc[BT + b] = fma((double)wu[v], xd, acc[BT + b]);
                                    }
                                }
                        }
                    }
                    warp_allreduce<2 * BT>(acc);
                    const int lcc = lc - i_first * TC;
                    if (lane == 0) {
#pragma unroll
                        for (int b = 0; b < BT; ++b) {
                            pd[((lcc * 2 + 0) * BT + b) * ncw + warp] = acc[b];
                            pd[((lcc * 2 + 1) * BT + b) * ncw + warp] = acc[BT + b];
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);
        }
        named_bar(1, NTC);
        // combine the warps' partial dot products in a fixed order; publish h and candidate keys
        if (ok && !*abort_flag) {
            for (int lc = tc; lc < n1 * TC; lc += NTC) {
                const int i = lc / TC, j = lc - i * TC;
                const int slot = (cta + i * G) * TC + j;
                if (slot >= n_rc) continue;
                if (slot < n_ret) {
                    for (int b = 0; b < B; ++b) {
                        float g = 0.f, u = 0.f;
                        for (int w = 0; w < ncw; ++w) {
                            g += pf[((lc * 2 + 0) * BT + b) * ncw + w];
                            u += pf[((lc * 2 + 1) * BT + b) * ncw + w];
                        }
                        P.h[(size_t)b * n_rc + slot] = silu_f32(g) * u;
                    }
                } else {
                    const int lcc = lc - i_first * TC;
                    double energy = 0.0;
                    for (int b = 0; b < B; ++b) {
                        double g = 0.0, u = 0.0;
                        for (int w = 0; w < ncw; ++w) {
                            g += pd[((lcc * 2 + 0) * BT + b) * ncw + w];
                            u += pd[((lcc * 2 + 1) * BT + b) * ncw + w];
                        }
                        const double hv = silu_f64(g) * u;
                        P.h[(size_t)b * n_rc + slot] = (float)hv;
                        energy = fma(hv, hv, energy);
                    }
                    P.keys[slot - n_ret] = score_key(P.norm_cand[slot - n_ret] * sqrt(energy));
                }
            }
        }
        __threadfence();
        named_bar(1, NTC);
        // ------------------------------------------------------------------ grid barrier
        if (tc == 0) {
            atomicAdd(P.sync + SYNC_BARRIER, 1u);
            grid_wait(P.sync + SYNC_BARRIER, (u32)G, abort_flag, gerr, P.wait_ns);
        }
        named_bar(1, NTC);
        ok = ok && !*abort_flag;

        // ------------------------------------------------------------------ phase 2
        float acc[CPW][BT][VEC];
#pragma unroll
        for (int c = 0; c < CPW; ++c)
#pragma unroll
            for (int b = 0; b < BT; ++b)
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[c][b][v] = 0.f;

        if (ok) {
            for (int idx = tc; idx < n2r * TR * BT; idx += NTC) {
                const int b = idx % BT, rr = idx / BT;
                const int i = rr / TR, r = rr - i * TR;
                const int row = (j0r + i * G) * TR + r;
                h2[idx] = (b < B && row < n_ret) ? __ldcg(P.h + (size_t)b * n_rc + row) : 0.f;
            }
        }
        named_bar(1, NTC);
        for (int i = 0; i < n2r; ++i, ++n) {
            const int s = n % P.nstage, use = n / P.nstage;
            if (ok) ok = mbar_wait(full0 + 8 * s, use & 1, abort_flag, gerr, ERR_MBAR_FULL, P.wait_ns);
            if (!ok) break;
            const int r0 = (j0r + i * G) * TR;
            const int nr = min(TR, n_ret - r0);
            const u32 base = ring_u + s * P.stage_bytes;
            for (int r = 0; r < nr; ++r) {
                float hv[BT];
#pragma unroll
                for (int b = 0; b < BT; ++b) hv[b] = h2[(i * TR + r) * BT + b];
#pragma unroll
                for (int c = 0; c < CPW; ++c) {
                    if (colok[c]) {
                        float w[VEC];
                        Elem<T>::unpack(lds128(base + (u32)r * P.row_bytes + col[c] * ES), w);
#pragma unroll
                        for (int b = 0; b < BT; ++b)
#pragma unroll
                            for (int v = 0; v < VEC; ++v) acc[c][b][v] = fmaf(hv[b], w[v], acc[c][b][v]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);
        }
        if (n2c > 0) {
            if (ok) ok = mbar_wait(selbar, 0, abort_flag, gerr, ERR_SELECT, P.wait_ns);
            float* h2c = h2 + P.capr * BT;
            if (ok) {
                for (int idx = tc; idx < n2c * TR * BT; idx += NTC) {
                    const int b = idx % BT, rr = idx / BT;
                    const int i = rr / TR, r = rr - i * TR;
                    const int pos = (j0c + i * G) * TR + r;
                    h2c[idx] = (b < B && pos < P.k) ? __ldcg(P.h + (size_t)b * n_rc + n_ret + mysel[rr]) : 0.f;
                }
            }
            named_bar(1, NTC);
            for (int i = 0; i < n2c; ++i, ++n) {
                const int s = n % P.nstage, use = n / P.nstage;
                if (ok) ok = mbar_wait(full0 + 8 * s, use & 1, abort_flag, gerr, ERR_MBAR_FULL, P.wait_ns);
                if (!ok) break;
                const int p0 = (j0c + i * G) * TR;
                const int nr = min(TR, P.k - p0);
                const u32 base = ring_u + s * P.stage_bytes;
                for (int r = 0; r < nr; ++r) {
                    float hv[BT];
#pragma unroll
                    for (int b = 0; b < BT; ++b) hv[b] = h2c[(i * TR + r) * BT + b];
#pragma unroll
                    for (int c = 0; c < CPW; ++c) {
                        if (colok[c]) {
                            float w[VEC];
                            Elem<T>::unpack(lds128(base + (u32)r * P.row_bytes + col[c] * ES), w);
#pragma unroll
                            for (int b = 0; b < BT; ++b)
#pragma unroll
                                for (int v = 0; v < VEC; ++v) acc[c][b][v] = fmaf(hv[b], w[v], acc[c][b][v]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * s);
            }
        }
        // partial y of this CTA -> fp32 accumulator (vector reductions performed at L2)
        if (ok && (n2r > 0 || n2c > 0)) {
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                if (colok[c]) {
#pragma unroll
                    for (int b = 0; b < BT; ++b) {
                        if (b < B) {
                            float* dst = P.y_acc + (size_t)b * d + col[c];
#pragma unroll
                            for (int v = 0; v < VEC; v += 4)
                                red_add_v4(dst + v, acc[c][b][v], acc[c][b][v + 1], acc[c][b][v + 2], acc[c][b][v + 3]);
                        }
                    }
                }
            }
        }
        __threadfence();
    }

    // ========================================================================= finish
    __syncthreads();
    if (tid == 0) {
        const u32 ticket = atomicAdd(P.sync + SYNC_TICKET, 1u);
        __threadfence();
        *last_flag = (ticket == (u32)G - 1u) ? 1 : 0;
    }
    __syncthreads();
    if (*last_flag) {
        // every CTA has added its partial sums: cast to the output dtype and clear the accumulator
        T* y = reinterpret_cast<T*>(P.y);
        for (int i = tid; i < B * d; i += blockDim.x) {
            const float v = __ldcg(P.y_acc + i);
            y[i] = Elem<T>::from_f32(v);
            P.y_acc[i] = 0.f;
        }
        __syncthreads();
        if (tid == 0) {
            P.sync[SYNC_BARRIER] = 0;
            P.sync[SYNC_TICKET] = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
template <typename T, int BT, int CPW>
int launch_fused(const DecodeParams& P, int G, int threads, size_t smem_bytes, cudaStream_t st) {
    auto kern = pop_decode_fused_kernel<T, BT, CPW>;
    // per instantiation and device: opt in to the shared-memory size, check that one CTA fits an SM
    static thread_local int cfg_dev = -1, cfg_threads = 0, cfg_ok = 0;
    static thread_local size_t cfg_smem = 0;
    int dev = 0;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev != cfg_dev || smem_bytes != cfg_smem || threads != cfg_threads) {
        POP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        int per_sm = 0;
        POP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem_bytes));
        cfg_dev = dev; cfg_smem = smem_bytes; cfg_threads = threads; cfg_ok = per_sm >= 1;
    }
    if (!cfg_ok) return POP_ERR_UNSUPPORTED;
    DecodeParams Pc = P;
    void* args[] = {(void*)&Pc};
    POP_CUDA(cudaLaunchCooperativeKernel((const void*)kern, dim3(G), dim3(threads), args, smem_bytes, st));
    pop_count_launch(1);
    return POP_OK;
}

template <typename T>
int dispatch_fused(const DecodeParams& P, int BT, int CPW, int G, int threads, size_t smem, cudaStream_t st) {
#define POP_CASE(bt, cpw) if (BT == bt && CPW == cpw) return launch_fused<T, bt, cpw>(P, G, threads, smem, st);
    POP_CASE(1, 1) POP_CASE(1, 2) POP_CASE(1, 4)
    POP_CASE(2, 1) POP_CASE(2, 2) POP_CASE(2, 4)
#undef POP_CASE
    return POP_ERR_UNSUPPORTED;
}

inline int align_up(int v, int a) { return (v + a - 1) / a * a; }

}  // namespace

int pop_launch_decode(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                      int32_t* sel_out, cudaStream_t st) {
    if (!p->coop || p->n_rc <= 0 || p->n_ret + k <= 0) return POP_ERR_UNSUPPORTED;
    if (B > 2) return POP_ERR_UNSUPPORTED;
    if (p->force_simple) return POP_ERR_UNSUPPORTED;
    const int stage_target = STAGE_TARGET;
    const int BT = B;
    const int es = p->es, d = p->d, VEC = 16 / es;
    const int chunks = (d + 32 * VEC - 1) / (32 * VEC);
    // consumer warps / chunks per warp: least padding, CPW in {1, 2, 4}
    const int ncw_pref = 16;                                  // preferred number of consumer warps
    const int order[] = {ncw_pref, 8, 10, 12, 16, 6, 7, 9, 11, 5, 4};
    int ncw = 0, CPW = 0, best = 1 << 30;
    for (int o : order) {
        int c = (chunks + o - 1) / o;
        c = c <= 1 ? 1 : (c <= 2 ? 2 : (c <= 4 ? 4 : 0));
        if (!c) continue;
        const int waste = c * o - chunks;
        if (waste < best) { best = waste; ncw = o; CPW = c; }
    }
    if (!ncw) return POP_ERR_UNSUPPORTED;

    DecodeParams P;
    memset(&P, 0, sizeof(P));
    P.GU = (const unsigned char*)p->GU; P.WdT = (const unsigned char*)p->WdT; P.x = x; P.y = y;
    P.norm_cand = p->norm_cand; P.idx_cand = p->idx_cand; P.h = p->h; P.keys = p->keys; P.y_acc = p->y_acc;
    P.sync = p->sync; P.mask_out = mask_out; P.sel_out = sel_out;
    P.d = d; P.n_ret = p->n_ret; P.n_cand = p->n_cand; P.n_rc = p->n_rc; P.k = k; P.B = B;
    P.row_bytes = d * es;
    const int pair = 2 * P.row_bytes;
    P.TC = stage_target / pair > 0 ? stage_target / pair : 1;
    if (P.TC > 16) P.TC = 16;
    P.TR = 2 * P.TC;
    P.stage_bytes = P.TC * pair;
    const int G = p->sm_count;
    P.T1 = (p->n_rc + P.TC - 1) / P.TC;
    P.T2r = (p->n_ret + P.TR - 1) / P.TR;
    P.T2c = (k + P.TR - 1) / P.TR;
    P.ncw = ncw;
    P.MC = ((P.T1 + G - 1) / G) * P.TC;
    const int tcand0 = p->n_ret / P.TC;
    P.MCC = p->n_cand > 0 ? (((P.T1 - tcand0) + G - 1) / G + 1) * P.TC : 0;
    P.capr = ((P.T2r + G - 1) / G) * P.TR;
    P.capc = ((P.T2c + G - 1) / G) * P.TR;
    P.keys_in_smem = p->n_cand <= KEYS_SMEM_MAX;
    P.wait_ns = 1000ull * (unsigned long long)pop_config_snapshot().wait_budget_us;

    // shared-memory layout after the ring
    int off = 0;
    P.off_x = off; off = align_up(off + BT * d * es, 16);
    P.off_pf = off; off = align_up(off + P.MC * 2 * BT * ncw * 4, 16);
    P.off_pd = off; off = align_up(off + P.MCC * 2 * BT * ncw * 8, 16);
    P.off_h2 = off; off = align_up(off + (P.capr + P.capc) * BT * 4, 16);
    P.off_mysel = off; off = align_up(off + P.capc * 4, 16);
    P.off_keys = off; off = align_up(off + (P.keys_in_smem ? p->n_cand * 8 : 0), 16);
    P.off_selsm = off; off = align_up(off + POP_SELECT_SMEM_WORDS(SEL_NT) * 4, 16);
    P.off_bars = off;
    const int max_stages = 16;
    const int fixed = off;                                   // bars come last, sized below
    const int avail = p->max_smem_optin - 1024;
    int nstage = (avail - fixed - (2 * max_stages + 2) * 8) / P.stage_bytes;
    if (nstage > max_stages) nstage = max_stages;
    if (nstage < 3) return POP_ERR_UNSUPPORTED;
    P.nstage = nstage;
    const int ring_bytes = nstage * P.stage_bytes;           // stage_bytes is a multiple of 32
    P.off_x += ring_bytes; P.off_pf += ring_bytes; P.off_pd += ring_bytes; P.off_h2 += ring_bytes;
    P.off_mysel += ring_bytes; P.off_keys += ring_bytes; P.off_selsm += ring_bytes; P.off_bars += ring_bytes;
    const size_t smem = (size_t)P.off_bars + (2 * nstage + 2) * 8;
    const int threads = (ncw + 1) * 32 + SEL_NT;

    if (p->dtype == POP_F32) return dispatch_fused<float>(P, BT, CPW, G, threads, smem, st);
    return dispatch_fused<__nv_bfloat16>(P, BT, CPW, G, threads, smem, st);
}
