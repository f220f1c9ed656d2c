// Decode step of POP (Sec. 3.3 "Decoding Stage", Sec. 3.4) for bf16 partitions in the tiled
// layout: ONE persistent kernel without any grid-wide barrier.  The step is cut into work units
// that CTAs claim from device-side counters; a unit that depends on another unit's result waits
// for that unit's flag only, so fast SMs run ahead instead of idling at a barrier.
//
//   phase-1 unit, Candidate   8 candidate channels: gate/up rows in fp64 (their scores decide the
//                             mask), h = silu(g) * u, score keys.  These units come first in the
//                             queue; the CTA that completes the last of them runs the exact
//                             radix top-k at once, while everybody else streams Retained rows.
//   phase-1 unit, Retained    8 retained channels: 16 rows (8 gate + 8 up) x d on the tensor
//                             cores (mma.m16n8k16, bf16 x bf16 -> fp32; the batch is the n dimension),
//                             h published with a per-unit ready flag.
//   phase-2 unit, Retained    16 retained channels x one quarter of the d outputs, again as
//                             m16n8k16 tiles; h enters as a bf16 (high, low) pair in two columns
//                             of the n dimension, so that y keeps fp32 accuracy.
//   phase-2 unit, Candidate   16 selected candidate rows x one quarter of d (only selected rows
//                             are read), gathered by row id, transposed by ldmatrix.
//
// Every consumer warp owns a private ring in shared memory that it fills with 16-byte
// cp.async copies (each lane copies the very bytes it will read back as its mma A fragment: the
// tiled layout stores fragments lane-contiguously) and drains NG-1 groups later.  A scheduler
// warp claims units, waits for their dependencies and stages the small operands (h fragments,
// selected row ids) so that consumer warps never poll global memory.
//
// CTAs are pinned to a quarter of the output columns in phase 2 (they move to another quarter
// when theirs is exhausted), partial y goes to an fp32 accumulator with vector reductions at L2;
// the CTA that finishes last casts it, re-arms the counters and advances the epoch that
// validates the flags.  Every wait is bounded; on expiry the kernel raises sync[SYNC_ERROR],
// drains its copies and returns.
#include "pop_common.cuh"
#include <stdlib.h>
#include <string.h>

#include "pop_select.cuh"

namespace {

constexpr int NCW = 16;                    // consumer warps
constexpr int NTC = NCW * 32;              // consumer threads
constexpr int NTHREADS = NTC + 32;         // + scheduler warp
constexpr int ND = 8;                      // unit descriptors in flight per CTA
constexpr int MAXG = 4;                    // copy groups per unit at most
constexpr u32 SPIN_LIMIT = 1u << 22;       // polls (with a short sleep) before a wait gives up: seconds
constexpr u32 BAR_SPIN_LIMIT = 1u << 20;   // mbarrier try_wait calls (each suspends for a while) before giving up
constexpr int SLOT = 512;                  // bytes one warp copies per cp.async instruction

enum { T_P1_CAND = 0, T_P1_RET = 1, T_P2_RET = 2, T_P2_CAND = 3, T_END = 4 };
enum { ERR_DESC = 11, ERR_CTA_BARRIER = 12, ERR_FLAG = 13, ERR_SELECT_FLAG = 14, ERR_THROTTLE = 15 };

struct StreamParams {
    const unsigned char* GUt;      // [n_rt][d/16][32][16 B]   retained gate/up fragments
    const unsigned char* GUc;      // [n_cand][2][d]           candidate gate/up rows
    const unsigned char* WdTt;     // [4][n_cg][d/64][32][16 B] retained down fragments, quarter-major
    const unsigned char* WdTc;     // [n_cand][d]              candidate down rows
    const __nv_bfloat16* x;
    __nv_bfloat16* y;
    const double* norm_cand;
    const int32_t* idx_cand;
    float* h;                      // [POP_MAX_BATCH][h_stride]
    u64* keys;
    float* y_acc;
    int32_t* sel_slots;
    u32* sync;
    u32* flags;                    // [n_rt] epoch at which the unit's h was published
    uint8_t* mask_out;
    int32_t* sel_out;
    int d, B, k, n_ret, n_cand, n_rt, n_cg, n_ret_pad, h_stride;
    int Uc, U1, n_cu, NG, p2_macro;
    int off_part, off_hfrag, off_rows, off_ystage, off_dsum, off_ctrl, scratch_keys;
};

struct Ctrl {
    int4 desc[ND];
    u64 bar_s1, bar_s2;
    volatile int filled;
    volatile int abort;
    volatile int do_select;
    int last;
    volatile int cons_m[NCW];
    volatile int cons_g[NCW];
    u32 selsm[POP_SELECT_SMEM_WORDS(NTC)];
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ u32 smem_u32(const void* p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp16(u32 dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp16_zero(u32 dst, const void* valid_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, 0;" ::"r"(dst), "l"(valid_src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void cp_wait_pending(int n) {      // n in [0, 7]
    switch (n) {
        case 0: cp_wait<0>(); break;
        case 1: cp_wait<1>(); break;
        case 2: cp_wait<2>(); break;
        case 3: cp_wait<3>(); break;
        case 4: cp_wait<4>(); break;
        case 5: cp_wait<5>(); break;
        case 6: cp_wait<6>(); break;
        default: cp_wait<7>(); break;
    }
}
__device__ __forceinline__ uint4 lds128(u32 addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(u32 addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 ldmatrix_x4_trans(u32 addr) {
    uint4 v;
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// D (16 x 8, fp32) += A (16 x 16, bf16, row) * B (16 x 8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint4& a, u32 b0, u32 b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
__device__ __forceinline__ u32 ld_acquire_gpu(const u32* p) {
    u32 v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(u32* p, u32 v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void mbar_init(u32 bar, u32 count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
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
__device__ __forceinline__ void named_bar(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// h as a bf16 pair: part 0 = nearest bf16, part 1 = nearest bf16 of the remainder.
__device__ __forceinline__ u32 split_bits(float v, int part) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 r = part ? __float2bfloat16_rn(v - __bfloat162float(hi)) : hi;
    return (u32)__bfloat16_as_ushort(r);
}
__device__ __forceinline__ u32 pack2(u32 lo, u32 hi) { return lo | (hi << 16); }

// Barrier among the NCW consumer warps with a bounded wait (an mbarrier: a warp that gave up
// elsewhere cannot leave the others waiting for ever).  `uses` counts completed phases.
__device__ __forceinline__ bool cta_barrier(u32 bar, int& uses, int lane, Ctrl* ctrl, u32* gerr) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const u32 parity = (u32)uses & 1u;
    ++uses;
    u32 spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++spins > BAR_SPIN_LIMIT) {
            ctrl->abort = 1;
            atomicExch(gerr, (u32)ERR_CTA_BARRIER);
            return false;
        }
    }
    return true;
}

// ---------------------------------------------------------------------------------------------
// The kernel.  GS = d / 1024 = 512-byte slots per warp and copy group; NBLK = n-blocks of 8
// columns used in phase 2 (batch <= 4 * NBLK).
// ---------------------------------------------------------------------------------------------
template <int GS, int NBLK>
__global__ void __launch_bounds__(NTHREADS, 1) pop_decode_stream_kernel(const StreamParams P) {
    constexpr int S = 4 * GS;              // slots per warp in a phase-1 unit
    constexpr int CPR = 2 * GS;            // 16-byte chunks per candidate row and warp in phase 2
    constexpr int BCAP = 4 * NBLK;         // batch capacity
    extern __shared__ __align__(128) unsigned char smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, G = gridDim.x;
    const int g8 = lane >> 2, t4 = lane & 3;
    const int d = P.d, B = P.B, KT = d >> 4;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + P.off_ctrl);
    uint2* hfrag = reinterpret_cast<uint2*>(smem + P.off_hfrag);   // [ND][MAXG][NBLK][32]
    int* rows = reinterpret_cast<int*>(smem + P.off_rows);          // [ND][16]
    u32* gerr = P.sync + SYNC_ERROR;
    const u32 bar_s1 = smem_u32(&ctrl->bar_s1), bar_s2 = smem_u32(&ctrl->bar_s2);

    if (tid == 0) {
        ctrl->filled = 0; ctrl->abort = 0; ctrl->do_select = 0; ctrl->last = 0;
        mbar_init(bar_s1, NCW);
        mbar_init(bar_s2, NCW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < NCW) { ctrl->cons_m[tid] = 0; ctrl->cons_g[tid] = 0; }
    const u32 epoch = ld_acquire_gpu(P.sync + SYNC_EPOCH) + 1u;
    __syncthreads();

    if (warp == NCW) {
        // ================================================================= scheduler warp
        int stage = 0, nstatic = 0, qoff = 0, pend_lo = 0, pend_hi = 0, pend_q = 0;   // lane 0's state
        int filled = 0, sched_groups = 0;
        const int myq = cta & 3;
        const int nq_groups = P.n_cg + P.n_cu;
        bool done = false, ok = true;
        while (!done && ok) {
            // room in the descriptor ring and in the look-ahead window?
            u32 spins = 0;
            for (;;) {
                int cm = lane < NCW ? ctrl->cons_m[lane] : 0x7fffffff;
                int cg = lane < NCW ? ctrl->cons_g[lane] : 0x7fffffff;
#pragma unroll
                for (int off = 16; off; off >>= 1) {
                    cm = min(cm, __shfl_xor_sync(0xffffffffu, cm, off));
                    cg = min(cg, __shfl_xor_sync(0xffffffffu, cg, off));
                }
                if (filled - cm < ND && sched_groups - cg < P.NG + MAXG) break;
                if (ctrl->abort) { ok = false; break; }
                if (++spins > SPIN_LIMIT) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_THROTTLE); ok = false; break; }
                __nanosleep(40);
            }
            if (!ok) break;
            // claim the next unit
            int type = T_END, a = 0, b = 0, ng = 0;
            if (lane == 0) {
                for (;;) {
                    if (pend_lo < pend_hi) {
                        if (pend_lo < P.n_cg) {
                            ng = min(pend_hi, P.n_cg) - pend_lo;
                            type = T_P2_RET; a = pend_lo; b = pend_q; pend_lo += ng;
                        } else {
                            type = T_P2_CAND; a = pend_lo - P.n_cg; b = pend_q; ng = 1; pend_lo += 1;
                        }
                        break;
                    }
                    if (stage == 0) {
                        int p;
                        if (nstatic < 2) { p = cta + nstatic * G; ++nstatic; }
                        else p = 2 * G + (int)atomicAdd(P.sync + SYNC_P1, 1u);
                        if (p < P.U1) {
                            if (p < P.Uc) { type = T_P1_CAND; a = p; } else { type = T_P1_RET; a = p - P.Uc; }
                            ng = MAXG;
                            break;
                        }
                        stage = 1;
                    }
                    if (qoff >= 4 || nq_groups == 0) { type = T_END; break; }
                    const int q = (myq + qoff) & 3;
                    const int p = (int)atomicAdd(P.sync + SYNC_Q0 + 32 * q, (u32)P.p2_macro);
                    if (p < nq_groups) { pend_lo = p; pend_hi = min(p + P.p2_macro, nq_groups); pend_q = q; }
                    else ++qoff;
                }
            }
            type = __shfl_sync(0xffffffffu, type, 0);
            a = __shfl_sync(0xffffffffu, a, 0);
            b = __shfl_sync(0xffffffffu, b, 0);
            ng = __shfl_sync(0xffffffffu, ng, 0);
            const int dslot = filled % ND;
            if (type == T_P2_RET) {
                // wait for the h of the unit's channels: phase-1 units 2a .. 2(a+ng)-1
                const int rt0 = 2 * a, rt1 = min(2 * (a + ng), P.n_rt);
                if (lane < rt1 - rt0) {
                    u32 sp = 0;
                    while (ld_acquire_gpu(P.flags + rt0 + lane) != epoch) {
                        if (ctrl->abort) { ok = false; break; }
                        if (++sp > SPIN_LIMIT) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_FLAG); ok = false; break; }
                        __nanosleep(64);
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                for (int gi = 0; gi < ng; ++gi) {
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb) {
                        const int n = g8 + 8 * nb, bb = n >> 1, part = n & 1;
                        u32 b0 = 0, b1 = 0;
                        if (bb < B) {
                            const float* hp = P.h + (size_t)bb * P.h_stride + 16 * (a + gi);
                            const float v0 = __ldcg(hp + 2 * t4), v1 = __ldcg(hp + 2 * t4 + 1);
                            const float v2 = __ldcg(hp + 2 * t4 + 8), v3 = __ldcg(hp + 2 * t4 + 9);
                            b0 = pack2(split_bits(v0, part), split_bits(v1, part));
                            b1 = pack2(split_bits(v2, part), split_bits(v3, part));
                        }
                        hfrag[((dslot * MAXG + gi) * NBLK + nb) * 32 + lane] = make_uint2(b0, b1);
                    }
                }
            } else if (type == T_P2_CAND) {
                if (lane == 0) {
                    u32 sp = 0;
                    while (ld_acquire_gpu(P.sync + SYNC_SEL_READY) != epoch) {
                        if (ctrl->abort) { ok = false; break; }
                        if (++sp > SPIN_LIMIT) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_SELECT_FLAG); ok = false; break; }
                        __nanosleep(64);
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                int sc = -1;                                   // candidate slot of row `lane` of the unit
                if (lane < 16) {
                    const int pos = 16 * a + lane;
                    if (pos < P.k) sc = __ldcg(P.sel_slots + pos);
                    rows[dslot * 16 + lane] = sc;
                }
#pragma unroll
                for (int nb = 0; nb < NBLK; ++nb) {
                    const int n = g8 + 8 * nb, bb = n >> 1, part = n & 1;
                    float v[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int kk = 2 * t4 + (e & 1) + (e >> 1) * 8;
                        const int s = __shfl_sync(0xffffffffu, sc, kk);
                        v[e] = (s >= 0 && bb < B) ? __ldcg(P.h + (size_t)bb * P.h_stride + P.n_ret_pad + s) : 0.f;
                    }
                    hfrag[((dslot * MAXG + 0) * NBLK + nb) * 32 + lane] =
                        make_uint2(pack2(split_bits(v[0], part), split_bits(v[1], part)),
                                   pack2(split_bits(v[2], part), split_bits(v[3], part)));
                }
            }
            if (lane == 0) ctrl->desc[dslot] = make_int4(type, a, b, ng);
            __syncwarp();
            __threadfence_block();
            ++filled;
            sched_groups += ng;
            if (lane == 0) ctrl->filled = filled;
            if (type == T_END) done = true;
        }
    } else {
        // ================================================================= consumer warps
        const int w = warp;
        const u32 ring0 = smem_u32(smem) + (u32)w * (u32)(P.NG * GS * SLOT);   // this warp's ring
        const int NG = P.NG;

        // x as mma B fragments for this warp's k range [w * S * 16, (w + 1) * S * 16)
        u32 xf[S][2];
#pragma unroll
        for (int s = 0; s < S; ++s) {
            if (g8 < B) {
                const u32* xp = reinterpret_cast<const u32*>(P.x + (size_t)g8 * d + (size_t)(w * S + s) * 16);
                xf[s][0] = __ldg(xp + t4);
                xf[s][1] = __ldg(xp + t4 + 4);
            } else {
                xf[s][0] = 0u; xf[s][1] = 0u;
            }
        }

        // ---- pipeline state (identical in all lanes of the warp)
        int n = 0;                      // groups consumed
        int icount = 0;                 // groups issued
        int im = 0, ig = 0;             // issue position: unit index, group within the unit
        int4 idesc = make_int4(T_END, 0, 0, 0);
        bool ihave = false, iend = false, ok = true;
        int late_upto = -1;             // groups up to this index were issued late: drain fully before reading
        int cm = 0;                     // units consumed
        int uses_s1 = 0, uses_s2 = 0, pbuf = 0;

        // Issues the copies of the next group if its descriptor is there.  block: wait for it.
        auto issue_one = [&](bool block) -> bool {
            if (!ihave) {
                u32 sp = 0;
                while (ctrl->filled <= im) {
                    if (!block) return false;
                    if (ctrl->abort) { ok = false; return false; }
                    if (++sp > SPIN_LIMIT) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_DESC); ok = false; return false; }
                    __nanosleep(20);
                }
                __threadfence_block();
                idesc = ctrl->desc[im % ND];
                ihave = true; ig = 0;
            }
            if (idesc.x == T_END) { iend = true; return false; }
            const u32 dst0 = ring0 + (u32)((icount % NG) * GS * SLOT);
            const int a = idesc.y, b = idesc.z;
            if (idesc.x == T_P1_RET) {
                const unsigned char* src = P.GUt + ((size_t)a * KT + (size_t)(w * S + ig * GS)) * SLOT + lane * 16;
#pragma unroll
                for (int j = 0; j < GS; ++j) cp16(dst0 + j * SLOT + lane * 16, src + j * SLOT);
            } else if (idesc.x == T_P1_CAND) {
                const int cs = 8 * a + (w >> 1);
                if (cs < P.n_cand) {
                    const unsigned char* src = P.GUc + ((size_t)cs * 2 + (w & 1)) * (size_t)d * 2 + (size_t)(ig * GS) * SLOT + lane * 16;
#pragma unroll
                    for (int j = 0; j < GS; ++j) cp16(dst0 + j * SLOT + lane * 16, src + j * SLOT);
                } else {
#pragma unroll
                    for (int j = 0; j < GS; ++j) cp16_zero(dst0 + j * SLOT + lane * 16, P.GUc);
                }
            } else if (idesc.x == T_P2_RET) {
                const unsigned char* src = P.WdTt + (((size_t)b * P.n_cg + (size_t)(a + ig)) * (size_t)(KT >> 2) + (size_t)(w * GS)) * SLOT + lane * 16;
#pragma unroll
                for (int j = 0; j < GS; ++j) cp16(dst0 + j * SLOT + lane * 16, src + j * SLOT);
            } else {   // T_P2_CAND: 16 rows x CPR chunks, row r at chunk (r * CPR + c), swizzled when CPR == 8
                const int* rw = rows + (im % ND) * 16;
#pragma unroll
                for (int j = 0; j < GS; ++j) {
                    const int f = j * 32 + lane, r = f / CPR, c = f - r * CPR;
                    const int sc = rw[r];
                    const int cc = (CPR == 8) ? (c ^ (r & 7)) : c;
                    const u32 dst = dst0 + (u32)((r * CPR + cc) * 16);
                    if (sc >= 0)
                        cp16(dst, P.WdTc + (size_t)sc * (size_t)d * 2 + ((size_t)b * (d >> 2) + (size_t)(w * GS * 16)) * 2 + c * 16);
                    else
                        cp16_zero(dst, P.WdTc);
                }
            }
            ++icount; ++ig;
            if (ig == idesc.w) { ihave = false; ++im; }
            return true;
        };

        // One pipeline step: top the ring up, commit, wait for group n.  Returns its base address.
        auto step = [&]() -> u32 {
            while (icount < n + NG && !iend) {
                const int j = icount;
                if (!issue_one(icount <= n)) break;      // group n itself must be issued: block for it
                if (j < n + NG - 1) late_upto = max(late_upto, j);
            }
            cp_commit();
            if (n <= late_upto) cp_wait<0>(); else cp_wait_pending(NG - 1);
            return ring0 + (u32)((n % NG) * GS * SLOT);
        };

        // prologue: NG - 1 commits, group i in commit i when its descriptor is there.  Only the
        // first group may block: a later unit's descriptor can depend on work this very CTA
        // still has to do (a selected-candidate unit waits for the selection, which waits for
        // every candidate unit), so the consumer side never waits for more than the group it
        // is about to read.
        for (int i = 0; i < NG - 1 && ok; ++i) {
            if (!iend && icount <= i) {
                const int j = icount;
                if (issue_one(i == 0) && j < i) late_upto = max(late_upto, j);
            }
            cp_commit();
        }

        // phase-2 accumulators: [m-tile][n-block][4]
        float acc[GS][NBLK][4];
#pragma unroll
        for (int i = 0; i < GS; ++i)
#pragma unroll
            for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][nb][e] = 0.f;
        int cq = -1;                                         // quarter the accumulators belong to

        // partial y of quarter q -> global fp32 accumulator
        auto flush = [&](int q) {
            float* ys = reinterpret_cast<float*>(smem + P.off_ystage) + w * (GS * 16);
            for (int bb = 0; bb < B; ++bb) {
                const int nb = bb >> 2, tt = bb & 3;
#pragma unroll
                for (int nbs = 0; nbs < NBLK; ++nbs) {
                    if (nbs == nb && t4 == tt) {
#pragma unroll
                        for (int i = 0; i < GS; ++i) {
                            ys[i * 16 + g8] = acc[i][nbs][0] + acc[i][nbs][1];
                            ys[i * 16 + g8 + 8] = acc[i][nbs][2] + acc[i][nbs][3];
                        }
                    }
                }
                __syncwarp();
                if (lane < GS * 4) {
                    const float4 v = *reinterpret_cast<const float4*>(ys + lane * 4);
                    red_add_v4(P.y_acc + (size_t)bb * d + (size_t)q * (d >> 2) + w * (GS * 16) + lane * 4, v.x, v.y, v.z, v.w);
                }
                __syncwarp();
            }
        };

        while (ok) {
            // descriptor of the unit to consume
            {
                u32 sp = 0;
                while (ctrl->filled <= cm) {
                    if (ctrl->abort) { ok = false; break; }
                    if (++sp > SPIN_LIMIT) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_DESC); ok = false; break; }
                    __nanosleep(20);
                }
                if (!ok) break;
                __threadfence_block();
            }
            const int4 cd = ctrl->desc[cm % ND];
            const int dslot = cm % ND;
            if (cd.x == T_END) break;

            if (cd.x == T_P1_RET) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const u32 base = step() + lane * 16;
                    if (!ok) break;
#pragma unroll
                    for (int j = 0; j < GS; ++j) {
                        const uint4 av = lds128(base + j * SLOT);
                        mma_bf16(c, av, xf[q * GS + j][0], xf[q * GS + j][1]);
                    }
                    ++n;
                }
                if (!ok) break;
                float* part = reinterpret_cast<float*>(smem + P.off_part) + (size_t)((pbuf * NCW + w) * 16) * 8;
                part[g8 * 8 + 2 * t4] = c[0];
                part[g8 * 8 + 2 * t4 + 1] = c[1];
                part[(g8 + 8) * 8 + 2 * t4] = c[2];
                part[(g8 + 8) * 8 + 2 * t4 + 1] = c[3];
                if (!cta_barrier(bar_s1, uses_s1, lane, ctrl, gerr)) { ok = false; break; }
                if (tid < 64) {
                    // fixed-order sum over the warps' k ranges; thread = (channel, batch column)
                    const int ch = tid >> 3, nn = tid & 7;
                    const float* pb = reinterpret_cast<const float*>(smem + P.off_part) + (size_t)(pbuf * NCW * 16) * 8;
                    float gs = 0.f, us = 0.f;
#pragma unroll
                    for (int ww = 0; ww < NCW; ++ww) {
                        gs += pb[(ww * 16 + ch) * 8 + nn];
                        us += pb[(ww * 16 + ch + 8) * 8 + nn];
                    }
                    const int slot = 8 * cd.y + ch;
                    if (nn < B && slot < P.n_ret) P.h[(size_t)nn * P.h_stride + slot] = silu_f32(gs) * us;
                    __threadfence();
                    named_bar(2, 64);
                    if (tid == 0) st_release_gpu(P.flags + cd.y, epoch);
                }
                pbuf ^= 1;
            } else if (cd.x == T_P1_CAND) {
                // warp w = row (channel w / 2, gate or up) of the unit, exact in fp64
                double dacc[BCAP];
#pragma unroll
                for (int bb = 0; bb < BCAP; ++bb) dacc[bb] = 0.0;
                const int cs = 8 * cd.y + (w >> 1);
#pragma unroll 1
                for (int q = 0; q < 4; ++q) {
                    const u32 base = step() + lane * 16;
                    if (!ok) break;
                    if (cs < P.n_cand) {
#pragma unroll 1
                        for (int j = 0; j < GS; ++j) {
                            float wf[8];
                            Elem<__nv_bfloat16>::unpack(lds128(base + j * SLOT), wf);
                            const int e0 = ((q * GS + j) * 32 + lane) * 8;
#pragma unroll
                            for (int bb = 0; bb < BCAP; ++bb) {
                                if (bb < B) {
                                    float xv[8];
                                    Elem<__nv_bfloat16>::unpack(__ldg(reinterpret_cast<const uint4*>(P.x + (size_t)bb * d + e0)), xv);
#pragma unroll
                                    for (int v = 0; v < 8; ++v) dacc[bb] = fma((double)wf[v], (double)xv[v], dacc[bb]);
                                }
                            }
                        }
                    }
                    ++n;
                }
                if (!ok) break;
#pragma unroll
                for (int bb = 0; bb < BCAP; ++bb)
#pragma unroll
                    for (int off = 16; off; off >>= 1) dacc[bb] += __shfl_xor_sync(0xffffffffu, dacc[bb], off);
                double* dsum = reinterpret_cast<double*>(smem + P.off_dsum);       // [NCW][8]
                if (lane == 0) {
#pragma unroll
                    for (int bb = 0; bb < BCAP; ++bb) dsum[w * 8 + bb] = dacc[bb];
                }
                if (!cta_barrier(bar_s1, uses_s1, lane, ctrl, gerr)) { ok = false; break; }
                if (w == 0) {
                    if (lane < 8) {
                        const int c2 = 8 * cd.y + lane;
                        if (c2 < P.n_cand) {
                            double energy = 0.0;
                            for (int bb = 0; bb < B; ++bb) {
                                const double hv = silu_f64(dsum[(2 * lane) * 8 + bb]) * dsum[(2 * lane + 1) * 8 + bb];
                                P.h[(size_t)bb * P.h_stride + P.n_ret_pad + c2] = (float)hv;
                                energy = fma(hv, hv, energy);
                            }
                            P.keys[c2] = score_key(P.norm_cand[c2] * sqrt(energy));
                        }
                        __threadfence();
                    }
                    __syncwarp();
                    if (lane == 0) {
                        const u32 prev = atomicAdd(P.sync + SYNC_CAND_DONE, 1u);
                        ctrl->do_select = (prev == (u32)P.Uc - 1u) ? 1 : 0;
                        __threadfence();
                    }
                }
                if (!cta_barrier(bar_s2, uses_s2, lane, ctrl, gerr)) { ok = false; break; }
                if (ctrl->do_select) {
                    // every candidate score of the step is published: exact top-k by all consumer threads
                    u64 thr = ~0ull;
                    int need_eq = 0;
                    const u64* keys = P.keys;
                    if (P.k > 0) {
                        if (P.scratch_keys) {
                            u64* ks = reinterpret_cast<u64*>(smem + P.off_part);
                            for (int i = tid; i < P.n_cand; i += NTC) ks[i] = __ldcg(P.keys + i);
                            keys = ks;
                            named_bar(1, NTC);
                        }
                        radix_select_kth<NTC>(keys, P.n_cand, P.k, ctrl->selsm, tid, 1, thr, need_eq);
                    }
                    select_walk<NTC>(keys, P.n_cand, thr, need_eq, ctrl->selsm, tid, 1, [&](int i, bool s, int pos) {
                        if (P.mask_out) P.mask_out[i] = s ? 1 : 0;
                        if (s) {
                            P.sel_slots[pos] = i;
                            if (P.sel_out) P.sel_out[pos] = P.idx_cand[i];
                        }
                    });
                    __threadfence();
                    named_bar(1, NTC);
                    if (tid == 0) st_release_gpu(P.sync + SYNC_SEL_READY, epoch);
                }
            } else {
                // ---- phase 2
                if (cd.z != cq) {
                    if (cq >= 0) {
                        flush(cq);
#pragma unroll
                        for (int i = 0; i < GS; ++i)
#pragma unroll
                            for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                                for (int e = 0; e < 4; ++e) acc[i][nb][e] = 0.f;
                    }
                    cq = cd.z;
                }
                const u32 hf0 = smem_u32(hfrag) + (u32)(dslot * MAXG * NBLK * 32 + lane) * 8u;
                if (cd.x == T_P2_RET) {
                    for (int gi = 0; gi < cd.w; ++gi) {
                        const u32 base = step() + lane * 16;
                        if (!ok) break;
                        uint2 hb[NBLK];
#pragma unroll
                        for (int nb = 0; nb < NBLK; ++nb) hb[nb] = lds64(hf0 + (u32)((gi * NBLK + nb) * 32) * 8u);
#pragma unroll
                        for (int i = 0; i < GS; ++i) {
                            const uint4 av = lds128(base + i * SLOT);
#pragma unroll
                            for (int nb = 0; nb < NBLK; ++nb) mma_bf16(acc[i][nb], av, hb[nb].x, hb[nb].y);
                        }
                        ++n;
                    }
                } else {
                    const u32 base = step();
                    if (!ok) break;
                    __syncwarp();                       // lanes read what other lanes copied
                    uint2 hb[NBLK];
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb) hb[nb] = lds64(hf0 + (u32)(nb * 32) * 8u);
                    const int mi = lane >> 3;
                    const int r = ((mi >> 1) << 3) + (lane & 7);
#pragma unroll
                    for (int i = 0; i < GS; ++i) {
                        const int c = 2 * i + (mi & 1);
                        const int cc = (CPR == 8) ? (c ^ (r & 7)) : c;
                        const uint4 av = ldmatrix_x4_trans(base + (u32)((r * CPR + cc) * 16));
#pragma unroll
                        for (int nb = 0; nb < NBLK; ++nb) mma_bf16(acc[i][nb], av, hb[nb].x, hb[nb].y);
                    }
                    ++n;
                    __syncwarp();
                }
                if (!ok) break;
            }
            ++cm;
            if (lane == 0) { ctrl->cons_m[w] = cm; ctrl->cons_g[w] = n; }
        }
        cp_wait<0>();
        if (ok && !ctrl->abort && cq >= 0) flush(cq);
        __threadfence();
    }

    // ========================================================================= finish
    __syncthreads();
    if (tid == 0) {
        const u32 ticket = atomicAdd(P.sync + SYNC_TICKET, 1u);
        __threadfence();
        ctrl->last = (ticket == (u32)G - 1u) ? 1 : 0;
    }
    __syncthreads();
    if (ctrl->last) {
        // every CTA has added its partial sums: cast, clear the accumulator, re-arm the counters
        for (int i = tid; i < B * d; i += NTHREADS) {
            const float v = __ldcg(P.y_acc + i);
            P.y[i] = __float2bfloat16_rn(v);
            P.y_acc[i] = 0.f;
        }
        __syncthreads();
        if (tid == 0) {
            P.sync[SYNC_TICKET] = 0;
            P.sync[SYNC_P1] = 0;
            P.sync[SYNC_CAND_DONE] = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) P.sync[SYNC_Q0 + 32 * q] = 0;
            __threadfence();
            st_release_gpu(P.sync + SYNC_EPOCH, epoch);
        }
    }
}

inline int align_up(int v, int a) { return (v + a - 1) / a * a; }

template <int GS, int NBLK>
int launch_stream(StreamParams& P, const pop_partition* p, cudaStream_t st) {
    auto kern = pop_decode_stream_kernel<GS, NBLK>;
    // shared-memory layout: [ring][part][hfrag][rows][ystage][dsum][ctrl]
    const int part_bytes = 2 * NCW * 16 * 8 * 4;
    const int hfrag_bytes = ND * MAXG * NBLK * 32 * 8;
    const int rows_bytes = ND * 16 * 4;
    const int ystage_bytes = NCW * GS * 16 * 4;
    const int dsum_bytes = NCW * 8 * 8;
    const int fixed = align_up(part_bytes, 128) + align_up(hfrag_bytes, 128) + align_up(rows_bytes, 128) +
                      align_up(ystage_bytes, 128) + align_up(dsum_bytes, 128) + align_up((int)sizeof(Ctrl), 128);
    const int group_bytes = NCW * GS * SLOT;
    int NG = (p->max_smem_optin - 1024 - fixed) / group_bytes;
    if (NG > 8) NG = 8;
    if (NG < 3) return POP_ERR_UNSUPPORTED;
    P.NG = NG;
    int off = NG * group_bytes;
    P.off_part = off; off += align_up(part_bytes, 128);
    P.off_hfrag = off; off += align_up(hfrag_bytes, 128);
    P.off_rows = off; off += align_up(rows_bytes, 128);
    P.off_ystage = off; off += align_up(ystage_bytes, 128);
    P.off_dsum = off; off += align_up(dsum_bytes, 128);
    P.off_ctrl = off; off += align_up((int)sizeof(Ctrl), 128);
    const size_t smem_bytes = (size_t)off;
    // the selection may copy the keys into the (then idle) part + hfrag area
    P.scratch_keys = (size_t)p->n_cand * 8 <= (size_t)part_bytes ? 1 : 0;

    static thread_local int cfg_dev = -1, cfg_ok = 0;
    static thread_local size_t cfg_smem = 0;
    int dev = 0;
    POP_CUDA(cudaGetDevice(&dev));
    if (dev != cfg_dev || smem_bytes != cfg_smem) {
        POP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes));
        int per_sm = 0;
        POP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NTHREADS, smem_bytes));
        cfg_dev = dev; cfg_smem = smem_bytes; cfg_ok = per_sm >= 1;
    }
    if (!cfg_ok) return POP_ERR_UNSUPPORTED;
    kern<<<p->sm_count, NTHREADS, smem_bytes, st>>>(P);
    POP_LAUNCHED();
    return POP_OK;
}

}  // namespace

bool pop_stream_layout_supported(int d, pop_dtype_t dt) {
    if (dt != POP_BF16 || d % 1024 != 0) return false;
    const int gs = d / 1024;
    return gs == 2 || gs == 4 || gs == 5 || gs == 8;
}

int pop_launch_decode_stream(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                             int32_t* sel_out, cudaStream_t st) {
    if (p->layout != POP_LAYOUT_TILED) return POP_ERR_UNSUPPORTED;
    static const int p2_macro_env = getenv("POP_P2_MACRO") ? atoi(getenv("POP_P2_MACRO")) : 2;
    StreamParams P;
    memset(&P, 0, sizeof(P));
    const size_t row = (size_t)p->d * 2;
    P.GUt = (const unsigned char*)p->GU;
    P.GUc = P.GUt + (size_t)p->n_rt * 16 * row;
    P.WdTt = (const unsigned char*)p->WdT;
    P.WdTc = P.WdTt + (size_t)p->n_ret_pad * row;
    P.x = (const __nv_bfloat16*)x; P.y = (__nv_bfloat16*)y;
    P.norm_cand = p->norm_cand; P.idx_cand = p->idx_cand; P.h = p->h; P.keys = p->keys; P.y_acc = p->y_acc;
    P.sel_slots = p->sel_slots; P.sync = p->sync; P.flags = p->flags; P.mask_out = mask_out; P.sel_out = sel_out;
    P.d = p->d; P.B = B; P.k = k; P.n_ret = p->n_ret; P.n_cand = p->n_cand; P.n_rt = p->n_rt; P.n_cg = p->n_cg;
    P.n_ret_pad = p->n_ret_pad; P.h_stride = p->h_stride;
    P.Uc = (p->n_cand + 7) / 8;
    P.U1 = P.Uc + p->n_rt;
    P.n_cu = (k + 15) / 16;
    P.p2_macro = p2_macro_env < 1 ? 1 : (p2_macro_env > MAXG ? MAXG : p2_macro_env);
    if (P.Uc == 0) {
        // no candidate unit will ever run the selection: nothing to select, publish that at once
        // (mask_out has no entries, k == 0)
    }
    const int gs = p->d / 1024;
    const int nblk = B <= 4 ? 1 : 2;
#define POP_CASE(G_, N_) if (gs == G_ && nblk == N_) return launch_stream<G_, N_>(P, p, st);
    POP_CASE(2, 1) POP_CASE(2, 2) POP_CASE(4, 1) POP_CASE(4, 2) POP_CASE(5, 1) POP_CASE(5, 2) POP_CASE(8, 1) POP_CASE(8, 2)
#undef POP_CASE
    return POP_ERR_UNSUPPORTED;
}
