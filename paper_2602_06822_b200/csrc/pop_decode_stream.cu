// Decode step of POP (Sec. 3.3 "Decoding Stage", Sec. 3.4) for bf16 partitions in the tiled
// layout: ONE persistent kernel without any grid-wide barrier.  The step is cut into work units;
// a unit that depends on another unit's result waits for that result only, so fast SMs run ahead
// instead of idling at a barrier.
//
//   phase-1 unit, Candidate   8 candidate channels: 16 rows (8 gate + 8 up) x d on the tensor
//                             cores (mma.m16n8k16, bf16 x bf16 -> fp32; the batch is the n dimension),
//                             together with the largest magnitudes met, from which a bound of the
//                             error of the score follows.  These units come first.
//   phase-1 unit, Retained    8 retained channels, the same way, without the bounds.
//   phase-2 unit, Retained    1 to 4 groups of 16 retained channels x one quarter of the d outputs,
//                             again as m16n8k16 tiles; h enters as a bf16 (high, low) pair in two
//                             columns of the n dimension, so that y keeps fp32 accuracy.
//   phase-2 unit, Candidate   the selected rows among 32 candidates (one word of the mask) x one
//                             quarter of d: only selected rows are read, gathered by row id and
//                             transposed by ldmatrix.
//
// Phase 1 is dealt out statically (unit i of CTA c is unit c + i G); phase 2 is claimed from
// per-quarter counters in shrinking chunks, which evens out what phase 1 left uneven.
//
// Warps of a CTA:
//   8 consumer warps  each covers 1/8 of the k range (phase 1) or of the output columns of the quarter
//                     (phase 2).  The tiled layout stores mma A fragments lane-contiguously, so in
//                     phase 1 a lane's 16-byte global load IS its fragment: weights go from HBM to
//                     registers to the tensor core, two batches of loads per lane taking turns.  In
//                     phase 2 each warp owns a private ring in shared memory that it fills with
//                     16-byte cp.async copies and drains NG - 1 groups later (gathered candidate rows
//                     need shared memory anyway: they are transposed by ldmatrix).
//   scheduler warp    claims phase-2 units, waits for their dependencies and stages the small operands
//                     (h fragments, selected row ids), so consumer warps never poll global memory.
//   reducer warp      adds the consumer warps' partial sums of a phase-1 unit, applies the activation
//                     and publishes h as 8-byte words (value, epoch of the step): a word carries its
//                     own validity, so there are no ready flags and no fences on the consumer side.
//   selection warp    the top-k of the candidates, replicated: every CTA computes the same mask from
//                     the same streamed scores and keeps it in its own shared memory.  Candidates
//                     whose streamed score is within the error bounds of the k-th are re-scored
//                     exactly in fp64 (these jobs are dealt out over the CTAs), so the mask is the
//                     one exact arithmetic gives.
//
// Partial y goes to an fp32 accumulator with vector reductions at L2; the CTA that finishes last
// casts it, re-arms the counters and advances the epoch.  Every wait is bounded; on expiry the
// kernel raises sync[SYNC_ERROR], drains its copies and returns.
#include "pop_common.cuh"
#include <string.h>

#include "pop_select.cuh"

namespace {

constexpr int NCW = 8;                     // consumer warps (16 / NCW must be an integer)
constexpr int NTC = NCW * 32;              // consumer threads
constexpr int W_SCHED = NCW;               // scheduler warp
constexpr int W_RED = NCW + 1;             // reducer warp
constexpr int W_SEL = NCW + 2;             // selection warp
constexpr int NTHREADS = NTC + 96;
constexpr int NPB_MAX = 4;                 // partial-sum buffers between the consumer warps and the reducer warp
constexpr int ND = 8;                      // unit descriptors in flight per CTA
constexpr int MAXG = 4;                    // copy groups per unit at most
constexpr int SLOT = 512;                  // bytes one warp copies per cp.async instruction
constexpr int RING_GROUPS = 3;             // depth of a consumer warp's copy ring in phase 2 (deeper rings measured slower)
constexpr int P2_MACRO = 4;                // largest phase-2 claim, in groups of 16 retained channels
constexpr int P2_WINDOW = 2 * MAXG;        // groups the scheduler may stage beyond the copy ring (shallower measured slower)
// Candidate keys per lane of a selection warp (n_cand <= 32 * KPL): the kernel is built for two sizes, because the
// larger one costs the common case (partition fraction 0.1: about 1100 candidates) 1.3 us per step.
constexpr int KPL_SMALL = 48, KPL_LARGE = 96;
constexpr int SEL_BATCH = 24;              // keys a lane fetches at once (independent loads); KPL is a multiple of it

enum { T_P1_CAND = 0, T_P1_RET = 1, T_P2_RET = 2, T_P2_CAND = 3, T_END = 4 };
enum { ERR_DESC = 11, ERR_PART_FULL = 12, ERR_FLAG = 13, ERR_SELECT_FLAG = 14, ERR_THROTTLE = 15, ERR_PART_FREE = 16,
       ERR_REFINE = 17, ERR_CAND_DONE = 18 };

struct StreamParams {
    const unsigned char* GUt;      // [n_rt][d/16][32][16 B]   retained gate/up fragments
    const unsigned char* GUc;      // [n_cand][2][d]           candidate gate/up rows
    const unsigned char* WdTt;     // [4][n_cg][d/64][32][16 B] retained down fragments, quarter-major
    const unsigned char* WdTc;     // [n_cand][d]              candidate down rows
    const __nv_bfloat16* x;
    __nv_bfloat16* y;
    const double* norm_cand;
    const float* wmax_cand;        // [2][n_cand] max |Wg[i][:]|, max |Wu[i][:]|
    const int32_t* idx_cand;
    u64* h;                        // [POP_MAX_BATCH][h_stride] (float bits, epoch of the step that wrote them): a value
                                   // carries its own validity, so publishing it needs no fence and no flag
    uint2* km;                     // [n_cand] streamed score of each candidate and a bound of its error (two fp32 bit patterns)
    double* rpart;                 // [n_cand * RPARTS][POP_MAX_BATCH] partial dot products of the re-scoring jobs
    float* y_acc;
    u32* sync;
    uint8_t* mask_out;
    int32_t* sel_out;
    int d, B, k, n_ret, n_cand, n_rt, n_cg, n_ret_pad, h_stride;
    int Uc, U1, n_cu, NG, NPB, p2_macro, window;
    unsigned long long wait_ns;    // budget of every device-side wait
    double cstep;                  // error bound of one warp's partial dot product / the largest magnitude in it
    int off_part, off_hfrag, off_rows, off_ystage, off_sel, off_ctrl;
};

template <int KPL>
struct CtrlT {
    int4 desc[ND];
    u64 bar_full[NPB_MAX];         // the consumer warps' partial sums in buffer b are complete (NCW arrivals)
    int2 part_hdr[NPB_MAX];        // (type, unit id) of the unit in buffer b
    volatile int filled;           // descriptors published by the scheduler
    volatile int abort;
    volatile int reduced;          // phase-1 units the reducer is done with
    int last;
    volatile int cons_m[NCW];
    volatile int cons_g[NCW];
    int cmt[NCW][8];               // consumer warps: commit index of each ring position
    float xmax[POP_MAX_BATCH];     // max |x[b][:]|
    u32 epoch;                     // epoch of this step (set by the scheduler warp)
    volatile int p1_started;       // phase-1 units the consumer warps have started (direct-load phase 1)
    volatile int sel_ready;        // rowmask holds the candidates decided by the streamed scores; umask marks the open words
    volatile int sel_final;        // this CTA's copy of the selection (rowmask) is final
    u32 umask[KPL];                // bit l of word j: candidate 32 j + l awaits its exact score
    u32 rowmask[KPL];              // bit l of word j: candidate 32 j + l is selected in this step
    u32 selsm[POP_SELECT_SMEM_WORDS(32)];
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
__device__ __forceinline__ uint4 ldg_stream(const void* p) {       // read-once global data, not kept in L1
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
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

// h as a bf16 pair: part 0 = nearest bf16, part 1 = nearest bf16 of the remainder.
__device__ __forceinline__ u32 split_bits(float v, int part) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 r = part ? __float2bfloat16_rn(v - __bfloat162float(hi)) : hi;
    return (u32)__bfloat16_as_ushort(r);
}
__device__ __forceinline__ u32 pack2(u32 lo, u32 hi) { return lo | (hi << 16); }

__device__ __forceinline__ u64 h_word(float v, u32 epoch) { return (u64)__float_as_uint(v) | ((u64)epoch << 32); }

#define POP_RAISE(code) do { ctrl->abort = 1; atomicExch(gerr, (u32)(code)); } while (0)

// Polls an h word until it carries the epoch of this step (bounded; ok = false on expiry or abort).
template <typename Ctrl>
__device__ __noinline__ u64 poll_h(const u64* p, u32 epoch, Ctrl* ctrl, u32* gerr, unsigned long long wait_ns, bool& ok) {
    PopWaitClock sp;
    for (;;) {
        const u64 hw = __ldcg(p);
        if ((u32)(hw >> 32) == epoch) return hw;
        if (ctrl->abort) { ok = false; return 0ull; }
        if (sp.expired(wait_ns)) { POP_RAISE(ERR_FLAG); ok = false; return 0ull; }
        __nanosleep(64);
    }
}

// The final pass of a CTA that finishes last: y = bf16(y_acc), y_acc = 0 over its part of the accumulator, in rounds of CB 16-byte loads per thread, all in flight together
// (the CTA is alone on this, and a round costs a trip to L2).  A function of its own so that its registers do not weigh
// on the kernel's main loops.
template <int CB>
__device__ __noinline__ void cast_y(float* y_acc, __nv_bfloat16* y, int lo4, int n4, int tid) {      // 16-byte groups [lo4, n4)
    float4* ya = reinterpret_cast<float4*>(y_acc);
    uint2* yo = reinterpret_cast<uint2*>(y);
    for (int i0 = lo4 + tid; i0 < n4; i0 += NTHREADS * CB) {
        float4 v[CB];
#pragma unroll
        for (int u = 0; u < CB; ++u)
            if (i0 + u * NTHREADS < n4) v[u] = __ldcg(ya + i0 + u * NTHREADS);
#pragma unroll
        for (int u = 0; u < CB; ++u) {
            const int i = i0 + u * NTHREADS;
            if (i < n4) {
                yo[i] = make_uint2(pack2(split_bits(v[u].x, 0), split_bits(v[u].y, 0)), pack2(split_bits(v[u].z, 0), split_bits(v[u].w, 0)));
                ya[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
}

// Event timestamps for performance work: compiled in only with -DPOP_STREAM_TRACE (a build of its own);
// slot `id` of the calling CTA gets the time at which its lane 0 passed the marker.
#ifdef POP_STREAM_TRACE
constexpr int TRACE_SLOTS = 32;
__device__ unsigned long long g_trace[1024 * TRACE_SLOTS];
__device__ __forceinline__ unsigned long long trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define POP_TRACE(id) do { if (lane == 0) g_trace[cta * TRACE_SLOTS + (id)] = trace_now(); } while (0)
#define POP_TRACE_VALUE(id, v) do { if (lane == 0) g_trace[cta * TRACE_SLOTS + (id)] = (unsigned long long)(v); } while (0)
#else
#define POP_TRACE(id) do { } while (0)
#define POP_TRACE_VALUE(id, v) do { } while (0)
#endif

// ---------------------------------------------------------------------------------------------
// Exact (fp64) re-scoring of an uncertain candidate, cut into RPARTS * B jobs: job (e, b) with
// e = (uncertain candidate number e / RPARTS, part e % RPARTS); a part is a 1/(RPARTS/2) segment
// of the candidate's gate row (parts < RPARTS/2) or up row.  The warp that runs it leaves the fp64
// dot product with x[b] over that segment in P.rpart[e][b].  All loads of a job are issued before
// the first is used (one memory round trip).  A product of two bf16 values is exact
// in fp32; sums in fp64.
// ---------------------------------------------------------------------------------------------
constexpr int RPARTS = 4;
constexpr int RVEC = 8;                    // 16-byte vectors per lane in flight for each of the two operands

__device__ __noinline__ void refine_job(const StreamParams& P, int c, int e, int bb, int lane) {
    const int d = P.d;
    const int seg = d / (RPARTS / 2);                          // elements per segment
    const int segv = seg >> 3;                                 // 16-byte vectors per segment
    const int part = e % RPARTS;
    const int which = part / (RPARTS / 2), sidx = part % (RPARTS / 2);
    const uint4* wr = reinterpret_cast<const uint4*>(P.GUc + ((size_t)c * 2 + which) * (size_t)d * 2) + (size_t)sidx * segv;
    {
        const uint4* xr = reinterpret_cast<const uint4*>(P.x + (size_t)bb * d) + (size_t)sidx * segv;
        double a0 = 0.0, a1 = 0.0;
#pragma unroll 1
        for (int v0 = lane; v0 < segv; v0 += 32 * RVEC) {
            uint4 rw[RVEC], rx[RVEC];
#pragma unroll
            for (int t = 0; t < RVEC; ++t) {
                const bool in = v0 + 32 * t < segv;
                rw[t] = in ? __ldg(wr + v0 + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
                rx[t] = in ? __ldg(xr + v0 + 32 * t) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int t = 0; t < RVEC; ++t) {
                float fw[8], fx[8];
                Elem<__nv_bfloat16>::unpack(rw[t], fw);
                Elem<__nv_bfloat16>::unpack(rx[t], fx);
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    a0 += (double)(fw[j] * fx[j]);
                    a1 += (double)(fw[j + 1] * fx[j + 1]);
                }
            }
        }
        a0 += a1;
#pragma unroll
        for (int off = 16; off; off >>= 1) a0 += __shfl_xor_sync(0xffffffffu, a0, off);
        if (lane == 0) P.rpart[(size_t)e * POP_MAX_BATCH + bb] = a0;
    }
}

// ---------------------------------------------------------------------------------------------
// Top-k of the candidates by (score descending, channel id ascending), decided on EXACT scores.
// Every CTA's selection warp runs this same program on the same data and arrives at the same
// mask, which it keeps in its own shared memory: nothing has to be published, and the warps that
// stream weights never wait for another CTA's selection.  Only the fp64 re-scoring is shared out
// (job e goes to CTA e mod G) and exchanged through global memory.
//
// The streamed scores a_i (fp32, P.km) are approximate, each with a bound m_i of its error
// (m = max m_i).  Let [tau_lo, tau_hi] be a bucket of key values that holds the k-th largest a_i.
// a_i > tau_hi + 2m  => i is in the exact top-k (fewer than k candidates have a_j > tau_hi, and
// every other one has an exact score below i's); a_i < tau_lo - 2m => i is not (the k candidates
// with a_j >= tau_lo all beat it).  The candidates in between are re-scored in fp64 from their
// plain rows and ranked exactly among themselves; the best k - |IN| of them complete the top-k.
//
// One warp pays about 10 ns per dependent instruction, so the code is written for few
// instructions (rolled loops; lane owns candidates lane + 32 j) and fetches in batches of
// independent loads.
// ---------------------------------------------------------------------------------------------
template <int KPL>
__device__ __noinline__ bool selection_main(const StreamParams& P, CtrlT<KPL>* ctrl, unsigned char* smem, int lane,
                                            int cta, int G) {
    static_assert(KPL % SEL_BATCH == 0, "the key fetch loop runs in whole batches");
    const int n = P.n_cand, k = P.k;
    const int rows = (n + 31) >> 5;
    u32* gerr = P.sync + SYNC_ERROR;
    u32* hist = ctrl->selsm;
    const u32 hist_u = smem_u32(hist);
    u32* const keys_sm = reinterpret_cast<u32*>(smem + P.off_sel);            // [KPL][32]
    int* const ulist = reinterpret_cast<int*>(keys_sm + KPL * 32);             // [KPL * 32] uncertain candidates, ascending
    u64* const uex = reinterpret_cast<u64*>(ulist + KPL * 32);                 // [KPL * 32] their exact keys
    u32* const rowmask = ctrl->rowmask;
    u32* const kr = keys_sm + lane;                                            // this lane's keys at stride 32
    const u32 lt = (1u << lane) - 1u;

    for (int j = lane; j < KPL; j += 32) {
        const int left = n - 32 * j;
        rowmask[j] = (k >= n && left > 0) ? (left >= 32 ? 0xffffffffu : ((1u << left) - 1u)) : 0u;
    }
    __syncwarp();
    if (k > 0 && n > 0) {
        // all candidate units of the step reduced (their h, keys and bounds are visible after the acquire)
        bool ok = true;
        if (lane == 0) {
            PopWaitClock sp;
            while (ld_acquire_gpu(P.sync + SYNC_CAND_DONE) < (u32)P.Uc) {
                if (ctrl->abort) { ok = false; break; }
                if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_CAND_DONE); ok = false; break; }
                __nanosleep(200);
            }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) return false;
    }
    POP_TRACE(1);
    if (k > 0 && k < n) {
        float mm = 0.f;
        u32 kor = 0u, kand = ~0u;
#pragma unroll 1
        for (int j0 = 0; j0 < rows; j0 += SEL_BATCH) {
            uint2 kv[SEL_BATCH];
#pragma unroll
            for (int t = 0; t < SEL_BATCH; ++t) {
                const int i = lane + 32 * (j0 + t);
                kv[t] = i < n ? __ldcg(P.km + i) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int t = 0; t < SEL_BATCH; ++t) {
                kr[32 * (j0 + t)] = kv[t].x;
                if (lane + 32 * (j0 + t) < n) { kor |= kv[t].x; kand &= kv[t].x; }
                mm = fmaxf(mm, __uint_as_float(kv[t].y));
            }
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, off));
            kor |= __shfl_xor_sync(0xffffffffu, kor, off);
            kand &= __shfl_xor_sync(0xffffffffu, kand, off);
        }
        POP_TRACE(19);
        // The k-th largest key up to its low bits: radix passes of 8 bits, skipping digits that all keys share,
        // at most two counted passes, and the second only while more than a few keys agree with the k-th largest on
        // the digits looked at: every key of that bucket is re-scored exactly, so a bucket of a few keys costs
        // nothing, and a counted pass costs this one warp 2.6 us.
        const u32 differ = kor ^ kand;
        u32 prefix = 0, mask = 0;
        int rem = k, counted = 0, bucket = n;
#pragma unroll 1
        for (int shift = 24; shift >= 0 && counted < 2 && bucket > 24; shift -= 8) {
            if (((differ >> shift) & 255u) == 0u) {
                prefix |= kor & (255u << shift);
                mask |= 255u << shift;
                continue;
            }
            for (int i = lane; i < 256; i += 32) hist[i] = 0;
            __syncwarp();
#pragma unroll 1
            for (int j8 = 0; j8 < rows; j8 += 12) {
                // twelve keys at a time: their loads from shared memory are issued together
                u32 key[12];
#pragma unroll
                for (int t = 0; t < 12; ++t) key[t] = kr[32 * (j8 + t < KPL ? j8 + t : 0)];
#pragma unroll
                for (int t = 0; t < 12; ++t)
                    if (j8 + t < rows && lane + 32 * (j8 + t) < n && (key[t] & mask) == prefix)
                        asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(hist_u + 4u * ((key[t] >> shift) & 255u)), "r"(1u) : "memory");
            }
            __syncwarp();
            u32 c[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = hist[8 * lane + j]; tot += c[j]; }
            u32 incl = tot;                                 // inclusive suffix sum over lanes
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const u32 t = __shfl_down_sync(0xffffffffu, incl, off);
                if (lane + off < 32) incl += t;
            }
            const u32 above = incl - tot;
            u32 found = 0xffffffffu, cumf = 0, cntf = 0;
            if (above < (u32)rem && (u32)rem <= above + tot) {
                u32 cum = above;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (found == 0xffffffffu && cum + c[j] >= (u32)rem) { found = 8 * lane + j; cumf = cum; cntf = c[j]; }
                    cum += c[j];
                }
            }
            const int src = __ffs(__ballot_sync(0xffffffffu, found != 0xffffffffu)) - 1;
            found = __shfl_sync(0xffffffffu, found, src);
            cumf = __shfl_sync(0xffffffffu, cumf, src);
            bucket = (int)__shfl_sync(0xffffffffu, cntf, src);
            rem -= (int)cumf;
            prefix |= found << shift;
            mask |= 255u << shift;
            ++counted;
            __syncwarp();
        }
        // fewer than k keys lie above the bucket [prefix, prefix | ~mask], at least k at or above its lower end
        POP_TRACE(20);
        // thresholds as key bit patterns, rounded away from the bucket (keys are non-negative floats: they order
        // like their bit patterns)
        const double m2 = 2.0 * (double)mm;
        const float t_in = __double2float_ru((double)__uint_as_float(prefix | ~mask) + m2);
        const float t_out = __double2float_rd((double)__uint_as_float(prefix) - m2);
        const u32 thr_in = __float_as_uint(t_in);
        const u32 thr_out = t_out > 0.f ? __float_as_uint(t_out) : 0u;
        int nin = 0, nu = 0;
#pragma unroll 4
        for (int j = 0; j < rows; ++j) {
            const int i = lane + 32 * j;
            const u32 key = kr[32 * j];
            const bool is_in = i < n && key > thr_in;
            const bool is_un = i < n && !is_in && !(key < thr_out);
            const u32 bu = __ballot_sync(0xffffffffu, is_un);
            const u32 bi = __ballot_sync(0xffffffffu, is_in);
            if (is_un) ulist[nu + __popc(bu & lt)] = i;
            if (lane == 0) { rowmask[j] = bi; ctrl->umask[j] = bu; }
            nu += __popc(bu);
            nin += __popc(bi);
        }
        // The words of the mask without an open candidate are final already: the scheduler may hand them out
        // while the few open candidates are re-scored.
        __threadfence_block();
        __syncwarp();
        if (lane == 0) ctrl->sel_ready = 1;
        POP_TRACE(2);
        POP_TRACE_VALUE(16, nu);
        if (nu > 0) {
            const int njobs = nu * RPARTS * P.B;
            int mine = 0;
#pragma unroll 1
            for (int jb = cta; jb < njobs; jb += G) {
                const int e = jb / P.B;
                refine_job(P, ulist[e / RPARTS], e, jb - e * P.B, lane);
                ++mine;
            }
            bool ok = true;
            POP_TRACE(3);
            if (lane == 0) {
                if (mine) { __threadfence(); atomicAdd(P.sync + SYNC_RF_DONE, (u32)mine); }
                PopWaitClock sp;
                while (ld_acquire_gpu(P.sync + SYNC_RF_DONE) < (u32)njobs) {
                    if (ctrl->abort) { ok = false; break; }
                    if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_REFINE); ok = false; break; }
                    __nanosleep(100);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) return false;
            POP_TRACE(4);
            // exact scores from the parts (fixed order), lane = uncertain candidate
#pragma unroll 1
            for (int e = lane; e < nu; e += 32) {
                const int c = ulist[e];
                double energy = 0.0;
                for (int bb = 0; bb < P.B; ++bb) {
                    double g = 0.0, u = 0.0;
#pragma unroll
                    for (int q = 0; q < RPARTS / 2; ++q) {
                        g += __ldcg(P.rpart + ((size_t)e * RPARTS + q) * POP_MAX_BATCH + bb);
                        u += __ldcg(P.rpart + ((size_t)e * RPARTS + RPARTS / 2 + q) * POP_MAX_BATCH + bb);
                    }
                    const double hv = silu_f64(g) * u;
                    energy = fma(hv, hv, energy);
                }
                uex[e] = score_key(P.norm_cand[c] * sqrt(energy));
            }
            __syncwarp();
            // the best ku of the uncertain set by (exact score descending, channel id ascending); ulist ascends, so
            // position order is channel order
            const int ku = k - nin;
            if (nu <= 64) {
                // a few candidates: every lane ranks its own against all
#pragma unroll 1
                for (int e = lane; e < nu; e += 32) {
                    const u64 ke = uex[e];
                    int r = 0;
#pragma unroll 1
                    for (int f = 0; f < nu; ++f) {
                        const u64 kf = uex[f];
                        r += (kf > ke || (kf == ke && f < e)) ? 1 : 0;
                    }
                    if (r < ku) {
                        const int ce = ulist[e];
                        atomicOr(&rowmask[ce >> 5], 1u << (ce & 31));
                    }
                }
            } else if (ku > 0) {
                // many (scores that the bounds cannot tell apart, e.g. all equal): a radix select on the exact keys
                // instead of nu^2 / 32 comparisons per lane, then one ordered walk for the ties at the threshold
                u64 thr = 0;
                int need_eq = 0;
                radix_select_kth<32>(uex, nu, ku < nu ? ku : nu, hist, lane, 1, thr, need_eq);
                int eq_seen = 0;
#pragma unroll 1
                for (int e0 = 0; e0 < nu; e0 += 32) {
                    const int e = e0 + lane;
                    const bool valid = e < nu;
                    const u64 ke = valid ? uex[e] : 0ull;
                    const bool is_eq = valid && ke == thr;
                    const u32 beq = __ballot_sync(0xffffffffu, is_eq);
                    if (valid && (ke > thr || (is_eq && eq_seen + __popc(beq & lt) < need_eq))) {
                        const int ce = ulist[e];
                        atomicOr(&rowmask[ce >> 5], 1u << (ce & 31));
                    }
                    eq_seen += __popc(beq);
                }
            }
            __syncwarp();
        }
    }
    __threadfence_block();
    __syncwarp();
    if (lane == 0) ctrl->sel_final = 1;
    POP_TRACE(5);
    // outputs: row j of the mask by CTA j mod G
#pragma unroll 1
    for (int j = cta; j < rows; j += G) {
        int base = 0;
        for (int jj = lane; jj < j; jj += 32) base += __popc(rowmask[jj]);
#pragma unroll
        for (int off = 16; off; off >>= 1) base += __shfl_xor_sync(0xffffffffu, base, off);
        const u32 m = rowmask[j];
        const int i = 32 * j + lane;
        if (i < n) {
            const bool sel = (m >> lane) & 1u;
            if (P.mask_out) P.mask_out[i] = sel ? 1 : 0;
            if (sel && P.sel_out) P.sel_out[base + __popc(m & lt)] = __ldg(P.idx_cand + i);
        }
    }
    POP_TRACE(6);
    return true;
}

// ---------------------------------------------------------------------------------------------
// The kernel.  GS = d / 1024 = 512-byte slots per warp and copy group; NBLK = n-blocks of 8
// columns used in phase 2 (batch <= 4 * NBLK).
// ---------------------------------------------------------------------------------------------
template <int GS, int NBLK, int KPL>
__global__ void __launch_bounds__(NTHREADS, 1) pop_decode_stream_kernel(const StreamParams P) {
    using Ctrl = CtrlT<KPL>;
    constexpr int GSL = GS * (16 / NCW);   // 512-byte slots per warp and copy group
    constexpr int S = 4 * GSL;             // slots per warp in a phase-1 unit
    constexpr int CPR = 2 * GSL;            // 16-byte chunks per candidate row and warp in phase 2
    constexpr int BCAP = 4 * NBLK;         // batch capacity
    extern __shared__ __align__(128) unsigned char smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cta = blockIdx.x, G = gridDim.x;
    const int g8 = lane >> 2, t4 = lane & 3;
    const int d = P.d, B = P.B, KT = d >> 4;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + P.off_ctrl);
    uint2* hfrag = reinterpret_cast<uint2*>(smem + P.off_hfrag);   // [ND][MAXG][NBLK][32]
    int* rows = reinterpret_cast<int*>(smem + P.off_rows);          // [ND][32]
    u32* gerr = P.sync + SYNC_ERROR;
    const int NPB = P.NPB;
    constexpr int PART_W = 2 * 16 * BCAP;   // floats a warp deposits per phase-1 unit: 16 rows x BCAP sums, then magnitudes

    if (tid == 0) {
        ctrl->filled = 0; ctrl->abort = 0; ctrl->reduced = 0; ctrl->last = 0;
        ctrl->sel_final = 0; ctrl->sel_ready = 0; ctrl->p1_started = 0;
        for (int b = 0; b < NPB_MAX; ++b) mbar_init(smem_u32(&ctrl->bar_full[b]), NCW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < NCW) { ctrl->cons_m[tid] = 0; ctrl->cons_g[tid] = 0; }
    // When launched with programmatic stream serialization the CTA may have started while the previous kernel of
    // the stream was still running: nothing that a kernel of the stream may have written is touched before that kernel
    // is complete.  The repacked weights are the exception: they are written once, by the kernels that build the
    // partition, which do not release their dependents early (so this kernel cannot have started before they
    // completed), and never again; the consumer warps therefore issue the loads of their first phase-1 unit before the
    // wait, which takes the first trip to HBM out of the step.  The next kernel may be placed from the wait on (it takes
    // an SM only once a CTA of this one has left it).
    constexpr int PRE_GSL = GS * (16 / NCW), PRE_S = 4 * PRE_GSL, PRE_BS = PRE_S % 16 == 0 ? 8 : 5;
    uint4 preA[PRE_BS], preB[PRE_BS];
    if (warp < NCW && cta < P.U1) {
        const int tile0 = cta < P.Uc ? P.n_rt + cta : cta - P.Uc;      // this CTA's first unit (candidate tiles follow the retained ones)
        const unsigned char* s0 = P.GUt + ((size_t)tile0 * (size_t)(P.d >> 4) + (size_t)(warp * PRE_S)) * SLOT + lane * 16;
#pragma unroll
        for (int j = 0; j < PRE_BS; ++j) preA[j] = ldg_stream(s0 + j * SLOT);
#pragma unroll
        for (int j = 0; j < PRE_BS; ++j) preB[j] = ldg_stream(s0 + (PRE_BS + j) * SLOT);
        // the rest of that unit is asked into L2 meanwhile (the SM may sit at the wait below for several microseconds
        // while the previous kernel's last CTAs finish, with HBM partly idle)
        // (asking for the CTA's second unit as well measured slower)
        if (PRE_S > 2 * PRE_BS && lane == 0)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(s0 + 2 * PRE_BS * SLOT), "r"((u32)((PRE_S - 2 * PRE_BS) * SLOT)) : "memory");
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#ifdef POP_STREAM_TRACE
    if (tid < TRACE_SLOTS) g_trace[cta * TRACE_SLOTS + tid] = 0ull;
#endif
    __syncthreads();
    if (warp == 0) POP_TRACE(0);

    if (warp == W_SCHED) {
        // ================================================================= scheduler warp
        const u32 epoch = ld_acquire_gpu(P.sync + SYNC_EPOCH) + 1u;
        if (lane == 0) ctrl->epoch = epoch;
        int stage = 1, qoff = 0, pend_lo = 0, pend_hi = 0, pend_q = 0;   // lane 0's state (stage 1: retained groups, 2: what is left of the candidate units)
        bool sel_waited = false;
        int spec_amt = 0, cand_exh = 0;     // cand_exh bit q: the candidate units of quarter q are all claimed
        constexpr int NDEFER = 16;
        int defer[NDEFER], ndefer = 0;      // claimed candidate units (word | quarter << 16) that wait for the final mask
        const int cpq = (G + 3) >> 2;      // CTAs that start on the same quarter
        u32 spec = 0;                      // result of a claim issued ahead of its use
        bool spec_valid = false;
        int filled = 0, sched_groups = 0;
        const int myq = cta & 3;
        bool done = false, ok = true;
        {
            // Phase 2 is claimed dynamically, and what is claimed is committed to this CTA: the first claim waits
            // until the consumer warps are two units from the end of their phase 1, late enough to see which
            // CTAs are ahead, early enough for the first descriptors to be staged when they get there.
            const int p1_count = cta < P.U1 ? (P.U1 - cta + G - 1) / G : 0;
            PopWaitClock sp;
            while (ctrl->p1_started < p1_count - 1) {
                if (ctrl->abort) { ok = false; break; }
                if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_THROTTLE); ok = false; break; }
                __nanosleep(200);
            }
        }
        while (!done && ok) {
            // room in the descriptor ring and in the look-ahead window?
            PopWaitClock spins;
            for (;;) {
                int cm = lane < NCW ? ctrl->cons_m[lane] : 0x7fffffff;
                int cg = lane < NCW ? ctrl->cons_g[lane] : 0x7fffffff;
#pragma unroll
                for (int off = 16; off; off >>= 1) {
                    cm = min(cm, __shfl_xor_sync(0xffffffffu, cm, off));
                    cg = min(cg, __shfl_xor_sync(0xffffffffu, cg, off));
                }
                if (filled - cm < ND && sched_groups - cg < P.NG + P.window) break;
                if (ctrl->abort) { ok = false; break; }
                if (spins.expired(P.wait_ns)) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_THROTTLE); ok = false; break; }
                __nanosleep(40);
            }
            if (!ok) break;
            // claim the next unit
            int type = T_END, a = 0, b = 0, ng = 0;
            if (lane == 0) {
                for (;;) {
                    if (pend_lo < pend_hi) {
                        ng = pend_hi - pend_lo;
                        type = T_P2_RET; a = pend_lo; b = pend_q; pend_lo += ng;
                        break;
                    }
                    if (stage == 1) {
                        // retained groups of this CTA's quarter, then what is left of the other quarters
                        if (qoff >= 4 || P.n_cg == 0) { stage = 2; qoff = 0; spec_valid = false; POP_TRACE(8); continue; }
                        // Once the selection is final, the selected candidate rows of the quarter this CTA works on
                        // come first: they are small gathered units, better placed where retained groups follow
                        // than at the very end.
                        if (ndefer > 0 && ctrl->sel_final) {
                            // a unit put off for its open candidates: the mask is final now
                            __threadfence_block();
                            const int pq = defer[--ndefer];
                            const int pc = pq & 0xffff;
                            const int cnt = __popc(ctrl->rowmask[pc]);
                            if (cnt == 0) continue;
                            type = T_P2_CAND; a = pc; b = pq >> 16; ng = (cnt + 15) >> 4;
                            break;
                        }
                        {
                            const int q = (myq + qoff) & 3;
                            if (P.n_cu > 0 && !((cand_exh >> q) & 1) && ndefer < NDEFER && (ctrl->sel_final || ctrl->sel_ready)) {
                                __threadfence_block();
                                const int pc = (int)atomicAdd(P.sync + SYNC_QC0 + 32 * q, 1u);
                                if (pc < P.n_cu) {
                                    if (!ctrl->sel_final && ctrl->umask[pc] != 0u) {
                                        defer[ndefer++] = pc | (q << 16);      // a word with an open candidate: after the final mask
                                        continue;
                                    }
                                    const int cnt = __popc(ctrl->rowmask[pc]);
                                    if (cnt == 0) continue;
                                    type = T_P2_CAND; a = pc; b = q; ng = (cnt + 15) >> 4;
                                    break;
                                }
                                cand_exh |= 1 << q;
                            }
                        }
                        // Claims shrink towards the end of a quarter (large ones keep the claim rate low, small ones
                        // even out the finish): up to p2_macro groups while plenty are left, then 2, then 1.
                        const int q = (myq + qoff) & 3;
                        const int amt0 = spec_valid ? spec_amt : P.p2_macro;
                        const u32 pu = spec_valid ? spec : atomicAdd(P.sync + SYNC_Q0 + 32 * q, (u32)amt0);
                        spec_valid = false;
                        const int p = (int)pu;
                        if (p < P.n_cg) {
                            pend_lo = p; pend_hi = min(p + amt0, P.n_cg); pend_q = q;
                            // the next claim on this quarter is issued now and used when this range is drained, so
                            // that its latency overlaps the staging of this range
                            const int left = P.n_cg - pend_hi;
                            spec_amt = left >= 6 * cpq ? P.p2_macro : (left >= 2 * cpq ? min(2, P.p2_macro) : 1);
                            spec = atomicAdd(P.sync + SYNC_Q0 + 32 * q, (u32)spec_amt);
                            spec_valid = true;
                        } else {
                            ++qoff;
                        }
                        continue;
                    }
                    // stage 2: the candidate units left: those put off, then what nobody has claimed
                    if (P.n_cu == 0 || (qoff >= 4 && ndefer == 0)) { type = T_END; break; }
                    if (!sel_waited) {
                        PopWaitClock sp;
                        while (!ctrl->sel_final) {
                            if (ctrl->abort) { type = -1; break; }
                            if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_SELECT_FLAG); type = -1; break; }
                            __nanosleep(64);
                        }
                        if (type < 0) break;
                        __threadfence_block();
                        sel_waited = true;
                        POP_TRACE(9);
                    }
                    if (ndefer > 0) {
                        const int pq = defer[--ndefer];
                        const int pc = pq & 0xffff;
                        const int cnt = __popc(ctrl->rowmask[pc]);
                        if (cnt == 0) continue;
                        type = T_P2_CAND; a = pc; b = pq >> 16; ng = (cnt + 15) >> 4;
                        break;
                    }
                    const int q = (myq + qoff) & 3;
                    if ((cand_exh >> q) & 1) { ++qoff; continue; }
                    const u32 pu = spec_valid ? spec : atomicAdd(P.sync + SYNC_QC0 + 32 * q, 1u);
                    spec_valid = false;
                    if ((int)pu < P.n_cu) {
                        spec = atomicAdd(P.sync + SYNC_QC0 + 32 * q, 1u);
                        spec_valid = true;
                        const int cnt = __popc(ctrl->rowmask[pu]);
                        if (cnt == 0) continue;
                        type = T_P2_CAND; a = (int)pu; b = q; ng = (cnt + 15) >> 4;
                        break;
                    }
                    ++qoff;
                }
            }
            type = __shfl_sync(0xffffffffu, type, 0);
            a = __shfl_sync(0xffffffffu, a, 0);
            b = __shfl_sync(0xffffffffu, b, 0);
            ng = __shfl_sync(0xffffffffu, ng, 0);
            if (type < 0) { ok = false; break; }
            const int dslot = filled % ND;
            if (type == T_P2_RET) {
                // h of the unit's channels, as mma B fragments.  All words of the unit are fetched at once (one
                // memory round trip per unit); a word not yet written in this step (its epoch tag is old) is
                // then polled until the phase-1 unit that owns it has published it.
                u64 hw[MAXG][NBLK][4];
#pragma unroll
                for (int gi = 0; gi < MAXG; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int bb = (g8 + 8 * nb) >> 1;
                            const int ch = 16 * (a + gi) + 2 * t4 + (e & 1) + (e >> 1) * 8;
                            const bool live = gi < ng && bb < B && ch < P.n_ret;       // padding channels are zero
                            hw[gi][nb][e] = live ? __ldcg(P.h + (size_t)bb * P.h_stride + ch) : ((u64)epoch << 32);
                        }
#pragma unroll
                for (int gi = 0; gi < MAXG; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if ((u32)(hw[gi][nb][e] >> 32) != epoch) {
                                const int bb = (g8 + 8 * nb) >> 1;
                                const int ch = 16 * (a + gi) + 2 * t4 + (e & 1) + (e >> 1) * 8;
                                hw[gi][nb][e] = poll_h(P.h + (size_t)bb * P.h_stride + ch, epoch, ctrl, gerr, P.wait_ns, ok);
                            }
                        }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int gi = 0; gi < MAXG; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb) {
                        if (gi < ng) {
                            const int part = (g8 + 8 * nb) & 1;
                            float v[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) v[e] = __uint_as_float((u32)hw[gi][nb][e]);
                            hfrag[((dslot * MAXG + gi) * NBLK + nb) * 32 + lane] =
                                make_uint2(pack2(split_bits(v[0], part), split_bits(v[1], part)),
                                           pack2(split_bits(v[2], part), split_bits(v[3], part)));
                        }
                    }
            } else if (type == T_P2_CAND) {
                // row list of the unit: the selected ones among candidates 32 a .. 32 a + 31, padded with -1
                const u32 m = ctrl->rowmask[a];
                int* rw = rows + dslot * 32;
                rw[lane] = -1;
                __syncwarp();
                if ((m >> lane) & 1u) rw[__popc(m & ((1u << lane) - 1u))] = 32 * a + lane;
                __syncwarp();
                // their h as mma B fragments (written by the reducers of the candidate units, all of which the
                // selection has waited for; the epoch tag is checked all the same)
                // All words of the unit are fetched at once (one memory round trip), then any word whose tag is old
                // is polled.  A mask word selects at most 32 rows: two groups.
                u64 hw[2][NBLK][4];
#pragma unroll
                for (int gi = 0; gi < 2; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int bb = (g8 + 8 * nb) >> 1;
                            const int sc = gi < ng ? rw[16 * gi + 2 * t4 + (e & 1) + (e >> 1) * 8] : -1;
                            hw[gi][nb][e] = (sc >= 0 && bb < B) ? __ldcg(P.h + (size_t)bb * P.h_stride + P.n_ret_pad + sc)
                                                                : ((u64)epoch << 32);       // value 0
                        }
#pragma unroll
                for (int gi = 0; gi < 2; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if ((u32)(hw[gi][nb][e] >> 32) != epoch) {
                                const int bb = (g8 + 8 * nb) >> 1;
                                const int sc = rw[16 * gi + 2 * t4 + (e & 1) + (e >> 1) * 8];
                                hw[gi][nb][e] = poll_h(P.h + (size_t)bb * P.h_stride + P.n_ret_pad + sc, epoch, ctrl, gerr, P.wait_ns, ok);
                            }
                        }
#pragma unroll
                for (int gi = 0; gi < 2; ++gi)
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb) {
                        if (gi < ng) {
                            const int part = (g8 + 8 * nb) & 1;
                            float v[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) v[e] = __uint_as_float((u32)hw[gi][nb][e]);
                            hfrag[((dslot * MAXG + gi) * NBLK + nb) * 32 + lane] =
                                make_uint2(pack2(split_bits(v[0], part), split_bits(v[1], part)),
                                           pack2(split_bits(v[2], part), split_bits(v[3], part)));
                        }
                    }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
            }
            if (lane == 0) ctrl->desc[dslot] = make_int4(type, a, b, ng);
            __syncwarp();
            __threadfence_block();
            ++filled;
            sched_groups += ng;
            if (lane == 0) ctrl->filled = filled;
            if (type == T_END) done = true;
        }
        POP_TRACE(10);
    } else if (warp == W_RED) {
        // ================================================================= reducer warp
        // Turns the consumer warps' partial sums of a phase-1 unit into h (and, for a candidate unit,
        // the approximate score keys with their error bounds) and counts the candidate units done.
        // The consumer warps never wait for it.
        const u32 epoch = ld_acquire_gpu(P.sync + SYNC_EPOCH) + 1u;
        // max |x[b][:]| for the error bounds of the candidate scores.  All loads of a row are in flight together (up to 20
        // vectors per lane at d = 5120): one trip to memory per batch row (a loop of four loads at a time made this warp
        // start on the first candidate unit 19 us late at batch 8).
        for (int bb = 0; bb < B; ++bb) {
            const uint4* xv = reinterpret_cast<const uint4*>(P.x + (size_t)bb * d);
            constexpr int XV = 4 * GS;                       // d / 8 / 32 vectors per lane (d = 1024 GS)
            uint4 xr[XV];
#pragma unroll
            for (int v = 0; v < XV; ++v) xr[v] = __ldg(xv + lane + 32 * v);
            float mx = 0.f;
#pragma unroll
            for (int v = 0; v < XV; ++v) {
                float f[8];
                Elem<__nv_bfloat16>::unpack(xr[v], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) mx = fmaxf(mx, fabsf(f[e]));
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            if (lane == 0) ctrl->xmax[bb] = mx;
        }
        __syncwarp();
        const float* part = reinterpret_cast<const float*>(smem + P.off_part);   // [NPB][NCW][PART_W]
        int u = 0;                                   // phase-1 units reduced so far
        const int p1_count = cta < P.U1 ? (P.U1 - cta + G - 1) / G : 0;   // phase 1 is dealt out statically
        bool ok = true;
        while (ok && u < p1_count) {
            const int buf = u % NPB;
            const u32 bar = smem_u32(&ctrl->bar_full[buf]);
            const u32 parity = (u32)(u / NPB) & 1u;
            PopWaitClock sp;
            while (!mbar_try_wait(bar, parity)) {
                if (ctrl->abort) { ok = false; break; }
                if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_PART_FULL); ok = false; break; }
                __nanosleep(100);
            }
            if (!ok) break;
            const int2 hdr = ctrl->part_hdr[buf];
            const float* pb = part + (size_t)buf * NCW * PART_W;
            const bool is_cand = hdr.x == T_P1_CAND;
            // thread = (channel, batch column); 8 * BCAP outputs
            for (int o = lane; o < 8 * BCAP; o += 32) {
                const int ch = o / BCAP, nn = o - ch * BCAP;
                if (!is_cand) {
                    float gs = 0.f, us = 0.f;                      // fixed-order sum over the warps' k ranges
#pragma unroll
                    for (int ww = 0; ww < NCW; ++ww) {
                        gs += pb[ww * PART_W + ch * BCAP + nn];
                        us += pb[ww * PART_W + (ch + 8) * BCAP + nn];
                    }
                    const int slot = 8 * hdr.y + ch;
                    if (nn < B && slot < P.n_ret) P.h[(size_t)nn * P.h_stride + slot] = h_word(silu_f32(gs) * us, epoch);
                } else {
                    // Candidate unit: approximate score and a bound of its error.  The warps' partial sums are
                    // added in fp64 (exact for all practical purposes); each partial sum comes from S tensor-core
                    // steps whose error is bounded through the magnitudes seen (P.cstep).  From there on the value runs
                    // in fp32 (this one warp is what the candidate units of a CTA wait for, and fp64 exponentials,
                    // divisions and square roots made it the slowest stage at larger batches); what that costs in
                    // accuracy is added to the bound, and every bound is rounded up.
                    const int c2 = 8 * hdr.y + ch;
                    const bool live = c2 < P.n_cand && nn < B;
                    double e2 = 0.0, d2 = 0.0;
                    if (live) {
                        const float xm = ctrl->xmax[nn];
                        const float pmg = P.wmax_cand[c2] * xm * 1.000001f;
                        const float pmu = P.wmax_cand[P.n_cand + c2] * xm * 1.000001f;
                        double gs = 0.0, us = 0.0;
                        float dg = 0.f, du = 0.f;
#pragma unroll
                        for (int ww = 0; ww < NCW; ++ww) {
                            gs += (double)pb[ww * PART_W + ch * BCAP + nn];
                            us += (double)pb[ww * PART_W + (ch + 8) * BCAP + nn];
                            dg += fmaxf(pb[ww * PART_W + 16 * BCAP + ch * BCAP + nn], pmg);
                            du += fmaxf(pb[ww * PART_W + 16 * BCAP + (ch + 8) * BCAP + nn], pmu);
                        }
                        const float cs = __double2float_ru(P.cstep * 1.000002);      // (the fp32 sums above: 8 x 2^-24)
                        dg *= cs;
                        du *= cs;
                        const float gf = (float)gs, uf = (float)us;
                        const float sg = silu_f32(gf);
                        const float hv = sg * uf;
                        P.h[(size_t)nn * P.h_stride + P.n_ret_pad + c2] = h_word(hv, epoch);
                        // |silu'| <= 1.1.  fp32 from the sums on: the rounding of gs moves silu by at most (1 + |gs|) / 2
                        // last places, expf, the addition and the division by 3 more, in all below 4e-6 of the value
                        // for gs > -30; below -30 the value itself is under 3e-12 |us|.
                        const float dh = (1.1f * dg * (fabsf(uf) + du) + fabsf(sg) * du + 4e-6f * fabsf(hv) + 1e-11f * fabsf(uf)) * 1.000002f + 1e-37f;
                        e2 = (double)hv * (double)hv;
                        d2 = (double)dh * (double)dh;
                    }
                    // sum over the batch columns of the channel (BCAP consecutive lanes)
#pragma unroll
                    for (int off = 1; off < BCAP; off <<= 1) {
                        e2 += __shfl_xor_sync(0xffffffffu, e2, off);
                        d2 += __shfl_xor_sync(0xffffffffu, d2, off);
                    }
                    if (nn == 0 && c2 < P.n_cand) {
                        // square roots in fp32 where the operand is an ordinary fp32 number (relative error 1e-7)
                        auto root = [](double v) -> double {
                            return (v > 1e-30 && v < 1e30) ? (double)sqrtf((float)v) : sqrt(v);
                        };
                        const double nc = P.norm_cand[c2];
                        const double key = nc * root(e2);
                        const float kf = (float)key;
                        // bound of |fp32 key - exact score|, rounded up
                        const float mf = __double2float_ru(nc * root(d2) * (1.0 + 1e-6) + key * 4e-7);
                        P.km[c2] = make_uint2(__float_as_uint(kf), __float_as_uint(mf));
                    }
                }
            }
            if (is_cand) __threadfence();                    // h, scores and bounds before the count below
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                ctrl->reduced = u + 1;
                if (is_cand) atomicAdd(P.sync + SYNC_CAND_DONE, 1u);    // what the selection warps wait for
            }
            if (is_cand) POP_TRACE(17);
            ++u;
        }
        POP_TRACE(14);
    } else if (warp == W_SEL) {
        // ================================================================= selection warp
        selection_main<KPL>(P, ctrl, smem, lane, cta, G);
    } else {
        // ================================================================= consumer warps
        const int w = warp;
        const u32 ring0 = smem_u32(smem) + (u32)w * (u32)(P.NG * GSL * SLOT);   // this warp's ring
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
        int ncommit = 0;                // cp.async groups committed so far
        volatile int* cmt = ctrl->cmt[w];   // per ring position: the commit that carries its copies
        int iring = 0, cring = 0;       // ring positions of the next group to issue / to consume
        const unsigned char* isrc = nullptr;   // issue side: this lane's source of the unit's next group
        int istep = 0;
        int cm = 0;                     // units consumed
        int p1seq = 0;                  // phase-1 units consumed

        // Issues the copies of the next group if its descriptor is there.  block: wait for it.
        auto issue_one = [&](bool block) -> bool {
            if (!ihave) {
                PopWaitClock sp;
                while (ctrl->filled <= im) {
                    if (!block) return false;
                    if (ctrl->abort) { ok = false; return false; }
                    if (sp.expired(P.wait_ns)) { ctrl->abort = 1; atomicExch(gerr, (u32)ERR_DESC); ok = false; return false; }
                    __nanosleep(20);
                }
                __threadfence_block();
                idesc = ctrl->desc[im % ND];
                ihave = true; ig = 0;
                // this lane's source address of the unit's first group and the step from group to group
                if (idesc.x == T_P2_RET) {
                    isrc = P.WdTt + (((size_t)idesc.z * P.n_cg + (size_t)idesc.y) * (size_t)(KT >> 2) + (size_t)(w * GSL)) * SLOT + lane * 16;
                    istep = (KT >> 2) * SLOT;
                }
            }
            if (idesc.x == T_END) { iend = true; return false; }
            const u32 dst0 = ring0 + (u32)(iring * GSL * SLOT);
            const int b = idesc.z;
            if (idesc.x != T_P2_CAND) {
#pragma unroll
                for (int j = 0; j < GSL; ++j) cp16(dst0 + j * SLOT + lane * 16, isrc + j * SLOT);
                isrc += istep;
            } else {   // T_P2_CAND: 16 rows x CPR chunks, row r at chunk (r * CPR + c), swizzled when CPR == 8
                const int* rw = rows + (im % ND) * 32 + ig * 16;
#pragma unroll
                for (int j = 0; j < GSL; ++j) {
                    const int f = j * 32 + lane, r = f / CPR, c = f - r * CPR;
                    const int sc = rw[r];
                    const int cc = (CPR % 8 == 0) ? (c ^ (r & 7)) : c;
                    const u32 dst = dst0 + (u32)((r * CPR + cc) * 16);
                    if (sc >= 0)
                        cp16(dst, P.WdTc + (size_t)sc * (size_t)d * 2 + ((size_t)b * (d >> 2) + (size_t)(w * GSL * 16)) * 2 + c * 16);
                    else
                        cp16_zero(dst, P.WdTc);
                }
            }
            cmt[iring] = ncommit;                       // the copies just issued go into the next commit
            iring = iring + 1 == NG ? 0 : iring + 1;
            ++icount; ++ig;
            if (ig == idesc.w) { ihave = false; ++im; }
            return true;
        };

        // One pipeline step: top the ring up, commit, wait for group n.  Returns its base address.
        auto step = [&]() -> u32 {
            while (icount < n + NG && !iend) {
                if (!issue_one(icount <= n)) break;      // group n itself must be issued: block for it
            }
            cp_commit();
            ++ncommit;
            // group n is complete once at most (commits after its own) groups are pending: exact even when a
            // descriptor came late and the group was issued later than its regular turn
            const int after = ncommit - 1 - cmt[cring];
            cp_wait_pending(after < 7 ? after : 7);
            const u32 base = ring0 + (u32)(cring * GSL * SLOT);
            cring = cring + 1 == NG ? 0 : cring + 1;
            return base;
        };

        // The partial-sum buffer of phase-1 unit number p1seq must have been released by the reducer.
        auto part_buffer_free = [&]() -> bool {
            PopWaitClock sp;
            while (ctrl->reduced < p1seq - NPB + 1) {
                if (ctrl->abort) return false;
                if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_PART_FREE); return false; }
                __nanosleep(20);
            }
            return true;
        };
        // Hands the partial sums (and, for a candidate unit, the magnitudes) of this warp's k range of a
        // phase-1 unit to the reducer warp: [16 rows][BCAP columns] each.
        auto deposit = [&](int type, int unit, const float (&c)[4], const float (&cmx)[4]) -> bool {
            if (!part_buffer_free()) return false;
            const int buf = p1seq % NPB;
            float* pw = reinterpret_cast<float*>(smem + P.off_part) + ((size_t)buf * NCW + w) * PART_W;
            if (2 * t4 < BCAP) {
                pw[g8 * BCAP + 2 * t4] = c[0];
                pw[g8 * BCAP + 2 * t4 + 1] = c[1];
                pw[(g8 + 8) * BCAP + 2 * t4] = c[2];
                pw[(g8 + 8) * BCAP + 2 * t4 + 1] = c[3];
                if (type == T_P1_CAND) {
                    float* mw = pw + 16 * BCAP;
                    mw[g8 * BCAP + 2 * t4] = cmx[0];
                    mw[g8 * BCAP + 2 * t4 + 1] = cmx[1];
                    mw[(g8 + 8) * BCAP + 2 * t4] = cmx[2];
                    mw[(g8 + 8) * BCAP + 2 * t4 + 1] = cmx[3];
                }
            }
            if (tid == 0) ctrl->part_hdr[buf] = make_int2(type, unit);
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->bar_full[buf]));
            ++p1seq;
            return true;
        };

        // Fills the copy ring for the descriptor-driven units: NG - 1 commits, group i in commit i when its
        // descriptor is there.  block_first: the first group may wait for its descriptor; a later one never does:
        // a later unit's descriptor can depend on work this very CTA still has to do (a selected-candidate
        // unit waits for the selection, which waits for every candidate unit), so the consumer side never waits
        // for more than the group it is about to read.
        auto ring_prologue = [&](bool block_first) {
            for (int i = 0; i < NG - 1 && ok; ++i) {
                if (!iend && icount <= i) issue_one(block_first && i == 0);
                cp_commit();
                ++ncommit;
            }
        };

        {
            // ---- phase 1 on direct loads: unit i of this CTA is unit cta + i G; this warp's part of it is a
            // contiguous run of S 512-byte slots, each lane's 16 bytes being its mma A fragment.
            // Loads are issued in batches of BS slots into two register buffers that take turns: a batch is
            // consumed (BS mma) and its buffer refilled at once with the batch after next, so BS to 2 BS loads
            // per lane are in flight at any time.
            constexpr int BS = S % 16 == 0 ? 8 : 5;
            constexpr int NB = S / BS;
            static_assert(S % BS == 0 && NB % 2 == 0, "a unit must be an even number of batches");
            const int p1_count = cta < P.U1 ? (P.U1 - cta + G - 1) / G : 0;
            auto src_of = [&](int i) -> const unsigned char* {
                const int p = cta + i * G;
                const int tile = p < P.Uc ? P.n_rt + p : p - P.Uc;        // candidate tiles follow the retained ones
                return P.GUt + ((size_t)tile * KT + (size_t)(w * S)) * SLOT + lane * 16;
            };
            static_assert(BS == PRE_BS, "the loads issued before the dependency wait are the first two batches");
            uint4 bufA[BS], bufB[BS];
#pragma unroll
            for (int j = 0; j < BS; ++j) { bufA[j] = preA[j]; bufB[j] = preB[j]; }      // issued at the top of the kernel
#pragma unroll 1
            for (int i = 0; i < p1_count && ok; ++i) {
                if (w == 0 && lane == 0) ctrl->p1_started = i + 1;
                if (i == p1_count - 1) ring_prologue(false);       // phase 2's first copies fly during the last unit
                const int p = cta + i * G;
                const bool is_cand = p < P.Uc;
                const unsigned char* cur = src_of(i);
                const unsigned char* nxt = i + 1 < p1_count ? src_of(i + 1) : nullptr;
                float c[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
                float cmx[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    uint4 (&buf)[BS] = (b & 1) ? bufB : bufA;
#pragma unroll
                    for (int j = 0; j < BS; ++j) {
                        const int sl = b * BS + j;
                        if (sl & 1) mma_bf16(c2, buf[j], xf[sl][0], xf[sl][1]);
                        else mma_bf16(c, buf[j], xf[sl][0], xf[sl][1]);
                        if (is_cand) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) cmx[e] = fmaxf(cmx[e], fmaxf(fabsf(c[e]), fabsf(c2[e])));
                        }
                    }
                    // refill with the batch after next: of this unit, or of the next one
                    if (b + 2 < NB) {
#pragma unroll
                        for (int j = 0; j < BS; ++j) buf[j] = ldg_stream(cur + ((b + 2) * BS + j) * SLOT);
                    } else if (nxt) {
#pragma unroll
                        for (int j = 0; j < BS; ++j) buf[j] = ldg_stream(nxt + ((b + 2 - NB) * BS + j) * SLOT);
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) c[e] += c2[e];
                if (!deposit(is_cand ? T_P1_CAND : T_P1_RET, is_cand ? p : p - P.Uc, c, cmx)) { ok = false; break; }
            }
            if (p1_count == 0) ring_prologue(true);
        }

        // phase-2 accumulators: [m-tile][n-block][4]
        float acc[GSL][NBLK][4];
#pragma unroll
        for (int i = 0; i < GSL; ++i)
#pragma unroll
            for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][nb][e] = 0.f;
        int cq = -1;                                         // quarter the accumulators belong to

        // partial y of quarter q -> global fp32 accumulator
        auto flush = [&](int q) {
            float* ys = reinterpret_cast<float*>(smem + P.off_ystage) + w * (GSL * 16);
            for (int bb = 0; bb < B; ++bb) {
                const int nb = bb >> 2, tt = bb & 3;
#pragma unroll
                for (int nbs = 0; nbs < NBLK; ++nbs) {
                    if (nbs == nb && t4 == tt) {
#pragma unroll
                        for (int i = 0; i < GSL; ++i) {
                            ys[i * 16 + g8] = acc[i][nbs][0] + acc[i][nbs][1];
                            ys[i * 16 + g8 + 8] = acc[i][nbs][2] + acc[i][nbs][3];
                        }
                    }
                }
                __syncwarp();
                for (int l = lane; l < GSL * 4; l += 32) {
                    const float4 v = *reinterpret_cast<const float4*>(ys + l * 4);
                    red_add_v4(P.y_acc + (size_t)bb * d + (size_t)q * (d >> 2) + w * (GSL * 16) + l * 4, v.x, v.y, v.z, v.w);
                }
                __syncwarp();
            }
        };

        while (ok) {
            // descriptor of the unit to consume
            {
                PopWaitClock sp;
                while (ctrl->filled <= cm) {
                    if (ctrl->abort) { ok = false; break; }
                    if (sp.expired(P.wait_ns)) { POP_RAISE(ERR_DESC); ok = false; break; }
                    __nanosleep(20);
                }
                if (!ok) break;
                __threadfence_block();
            }
            const int4 cd = ctrl->desc[cm % ND];
            const int dslot = cm % ND;
            if (cd.x == T_END) break;
#ifdef POP_STREAM_TRACE
            if (w == 0 && cd.x == T_P2_RET && cq < 0) POP_TRACE(11);
            if (w == 0 && cd.x == T_P2_CAND && !g_trace[cta * TRACE_SLOTS + 12]) POP_TRACE(12);
            if (w == 0 && lane == 0) {
                g_trace[cta * TRACE_SLOTS + 21] = (unsigned long long)cd.x;                       // type of the last unit
                g_trace[cta * TRACE_SLOTS + (cd.x == T_P2_CAND ? 22 : 23)] += (unsigned long long)cd.w;   // groups by type
                g_trace[cta * TRACE_SLOTS + 24] = trace_now();                                    // start of the last unit
            }
#endif

            // ---- unit prologue
            if (cd.z != cq) {
                if (cq >= 0) {
                    flush(cq);
#pragma unroll
                    for (int i = 0; i < GSL; ++i)
#pragma unroll
                        for (int nb = 0; nb < NBLK; ++nb)
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[i][nb][e] = 0.f;
                }
                cq = cd.z;
            }
            const u32 hf0 = smem_u32(hfrag) + (u32)(dslot * MAXG * NBLK * 32 + lane) * 8u;

            // ---- the unit's copy groups: one pipeline step each (a single call site keeps the code small)
#pragma unroll 1
            for (int gi = 0; gi < cd.w; ++gi) {
                const u32 base = step();
                if (!ok) break;
                if (cd.x != T_P2_CAND) {
                    // all fragments of the group first (the loads pipeline), then the mma chains
                    uint4 av[GSL];
#pragma unroll
                    for (int j = 0; j < GSL; ++j) av[j] = lds128(base + lane * 16 + j * SLOT);
                    {
                        uint2 hb[NBLK];
#pragma unroll
                        for (int nb = 0; nb < NBLK; ++nb) hb[nb] = lds64(hf0 + (u32)((gi * NBLK + nb) * 32) * 8u);
#pragma unroll
                        for (int i = 0; i < GSL; ++i) {
#pragma unroll
                            for (int nb = 0; nb < NBLK; ++nb) mma_bf16(acc[i][nb], av[i], hb[nb].x, hb[nb].y);
                        }
                    }
                } else {
                    __syncwarp();                       // lanes read what other lanes copied
                    uint2 hb[NBLK];
#pragma unroll
                    for (int nb = 0; nb < NBLK; ++nb) hb[nb] = lds64(hf0 + (u32)((gi * NBLK + nb) * 32) * 8u);
                    const int mi = lane >> 3;
                    const int r = ((mi >> 1) << 3) + (lane & 7);
#pragma unroll
                    for (int i = 0; i < GSL; ++i) {
                        const int cch = 2 * i + (mi & 1);
                        const int cc = (CPR % 8 == 0) ? (cch ^ (r & 7)) : cch;
                        const uint4 av = ldmatrix_x4_trans(base + (u32)((r * CPR + cc) * 16));
#pragma unroll
                        for (int nb = 0; nb < NBLK; ++nb) mma_bf16(acc[i][nb], av, hb[nb].x, hb[nb].y);
                    }
                    __syncwarp();
                }
                ++n;
                if (lane == 0) ctrl->cons_g[w] = n;
            }
            if (!ok) break;

            ++cm;
            if (lane == 0) ctrl->cons_m[w] = cm;
        }
        if (w == 0) POP_TRACE(13);
        cp_wait<0>();
        if (ok && !ctrl->abort && cq >= 0) flush(cq);
        __threadfence();
    }

    // ========================================================================= finish
    __syncthreads();
    if (warp == 0) POP_TRACE(15);
    // The CTAs that finish last cast the accumulator: one of them at small batches; at large ones (NBLK = 2: up to
    // 8 d values, more than one SM moves in a microsecond) the last CAST_K share it, each waiting until every CTA has
    // added its partial sums (they are the last to arrive, so the wait is short; it is bounded like every other).
    constexpr int CAST_K_MAX = NBLK == 2 ? 8 : 1;
    const int cast_k = CAST_K_MAX < G ? CAST_K_MAX : G;
    if (tid == 0) {
        const u32 ticket = atomicAdd(P.sync + SYNC_TICKET, 1u);
        __threadfence();
        ctrl->last = (int)ticket - (G - cast_k) + 1;          // > 0: this CTA casts slice last - 1
    }
    __syncthreads();
    if (ctrl->last > 0) {
        const int slice = ctrl->last - 1;
        if (cast_k > 1) {
            if (tid == 0) {
                PopWaitClock sp;
                while (ld_acquire_gpu(P.sync + SYNC_TICKET) < (u32)G) {
                    if (sp.expired(P.wait_ns)) { atomicExch(gerr, (u32)ERR_THROTTLE); break; }
                    __nanosleep(50);
                }
            }
            __syncthreads();
        }
        // every CTA has added its partial sums: cast this CTA's part of the accumulator and clear it
        const int n4 = (B * d) >> 2;
        const int lo = (int)((long long)n4 * slice / cast_k), hi = (int)((long long)n4 * (slice + 1) / cast_k);
        cast_y<8 * NBLK>(P.y_acc, P.y, lo, hi, tid);
        bool rearm = cast_k == 1;
        if (cast_k > 1) {
            __threadfence();
            __syncthreads();
            if (tid == 0) rearm = atomicAdd(P.sync + SYNC_CAST_DONE, 1u) == (u32)cast_k - 1u;
        }
        if (tid == 0 && rearm) {
            // every CTA is past its last use of the counters: re-arm them and advance the epoch (plain stores: the
            // next launch on the stream starts only after this grid has completed)
            P.sync[SYNC_TICKET] = 0;
            P.sync[SYNC_CAST_DONE] = 0;
            P.sync[SYNC_CAND_DONE] = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) { P.sync[SYNC_Q0 + 32 * q] = 0; P.sync[SYNC_QC0 + 32 * q] = 0; }
            P.sync[SYNC_RF_DONE] = 0;
            P.sync[SYNC_EPOCH] = ctrl->epoch;
        }
        if (warp == 0) POP_TRACE(18);
    }
}

inline int align_up(int v, int a) { return (v + a - 1) / a * a; }

template <int GS, int NBLK, int KPL>
int launch_stream(StreamParams& P, const pop_partition* p, cudaStream_t st) {
    using Ctrl = CtrlT<KPL>;
    auto kern = pop_decode_stream_kernel<GS, NBLK, KPL>;
    // shared-memory layout: [ring][part][hfrag][rows][ystage][ctrl]
    const int GSL = GS * (16 / NCW);
    const int NPB = NBLK == 1 ? 3 : 2;
    const int sel_bytes = KPL * 32 * (4 + 4 + 8);              // selection warp: candidate keys, uncertain list, exact keys
    const int part_bytes = NPB * NCW * 2 * 16 * (4 * NBLK) * 4;
    const int hfrag_bytes = ND * MAXG * NBLK * 32 * 8;
    const int rows_bytes = ND * 32 * 4;
    const int ystage_bytes = NCW * GSL * 16 * 4;
    const int fixed = align_up(part_bytes, 128) + align_up(hfrag_bytes, 128) + align_up(rows_bytes, 128) +
                      align_up(ystage_bytes, 128) + align_up(sel_bytes, 128) + align_up((int)sizeof(Ctrl), 128);
    const int group_bytes = NCW * GSL * SLOT;
    int NG = (p->max_smem_optin - 1024 - fixed) / group_bytes;
    if (NG > 8) NG = 8;
    if (NG > RING_GROUPS) NG = RING_GROUPS;
    if (NG < 3) return POP_ERR_UNSUPPORTED;
    P.NG = NG;
    P.NPB = NPB;
    int off = NG * group_bytes;
    P.off_part = off; off += align_up(part_bytes, 128);
    P.off_hfrag = off; off += align_up(hfrag_bytes, 128);
    P.off_rows = off; off += align_up(rows_bytes, 128);
    P.off_ystage = off; off += align_up(ystage_bytes, 128);
    P.off_sel = off; off += align_up(sel_bytes, 128);
    P.off_ctrl = off; off += align_up((int)sizeof(Ctrl), 128);
    const size_t smem_bytes = (size_t)off;

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
    // CTAs wait on one another's results.  Launch mode (pop_set_config): POP_LAUNCH_PDL (default) = plain launch with
    // programmatic stream serialization, which lets this kernel's CTAs take the SMs the previous kernel of the stream
    // leaves, up to their griddepcontrol.wait, and so hides the launch latency between the steps of a decode loop;
    // POP_LAUNCH_COOPERATIVE = cooperative launch, which makes the driver place all CTAs at once even when other
    // streams keep SMs busy, at the price of that latency; POP_LAUNCH_PLAIN.  In the first and last mode a CTA that
    // could not be placed alongside the others makes the bounded waits of the others expire (POP_ERR_TIMEOUT from
    // pop_partition_check), not hang.
    const int mode = pop_config_snapshot().launch_mode;
    const int pdl_env = mode == POP_LAUNCH_PDL;
    const int coop_env = mode == POP_LAUNCH_COOPERATIVE;
    if (pdl_env) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(p->sm_count); cfg.blockDim = dim3(NTHREADS); cfg.dynamicSmemBytes = smem_bytes; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        POP_CUDA(cudaLaunchKernelEx(&cfg, kern, P));
    } else if (p->coop && coop_env) {
        void* args[] = {(void*)&P};
        POP_CUDA(cudaLaunchCooperativeKernel((const void*)kern, dim3(p->sm_count), dim3(NTHREADS), args, smem_bytes, st));
    } else {
        kern<<<p->sm_count, NTHREADS, smem_bytes, st>>>(P);
    }
    POP_LAUNCHED();
    return POP_OK;
}

}  // namespace

#ifdef POP_STREAM_TRACE
// Copies the event timestamps of the last launch to the host (trace builds only): [ctas][32].
extern "C" int pop_debug_stream_trace(unsigned long long* h_out, int ctas) {
    POP_CUDA(cudaDeviceSynchronize());
    POP_CUDA(cudaMemcpyFromSymbol(h_out, g_trace, sizeof(unsigned long long) * 32 * (size_t)ctas));
    return POP_OK;
}
#endif

int pop_stream_max_candidates() { return 32 * KPL_LARGE; }

bool pop_stream_layout_supported(int d, pop_dtype_t dt) {
    if (dt != POP_BF16 || d % 1024 != 0) return false;
    const int gs = d / 1024;
    return gs == 2 || gs == 4 || gs == 5;
}

int pop_launch_decode_stream(pop_partition* p, const void* x, int B, int k, void* y, uint8_t* mask_out,
                             int32_t* sel_out, cudaStream_t st) {
    if (p->layout != POP_LAYOUT_TILED) return POP_ERR_UNSUPPORTED;
    StreamParams P;
    memset(&P, 0, sizeof(P));
    const size_t row = (size_t)p->d * 2;
    P.GUt = (const unsigned char*)p->GU;
    P.GUc = P.GUt + (size_t)(p->n_rt + p->n_ct) * 16 * row;
    P.WdTt = (const unsigned char*)p->WdT;
    P.WdTc = P.WdTt + (size_t)p->n_ret_pad * row;
    P.x = (const __nv_bfloat16*)x; P.y = (__nv_bfloat16*)y;
    P.wmax_cand = p->wnorm_cand; P.km = reinterpret_cast<uint2*>(p->keys); P.rpart = p->rpart;
    // Error model of a warp's partial dot product (d/16/NCW mma steps, each adding 16 exact bf16 x bf16 products to
    // an fp32 accumulator).  Measured on B200 with addends placed around the accumulator's last place: the 17 addends
    // are aligned to the largest one and cut two bits below its last place (an addend below 2^-25 of the largest
    // vanishes), the aligned sum is exact and the result is truncated toward zero.  One step therefore errs by less
    // than 16 * 2^-25 * M + 2^-23 * |result| <= 5 * 2^-23 of the largest magnitude involved (accumulator before and
    // after, any single product), which the kernel tracks.  The GPU tests check the bound against the oracle's exact
    // scores (the observed error stays below a few percent of it).
    P.cstep = (double)(p->d / 16 / NCW) * 5.0 * (1.0 / 8388608.0);
    P.norm_cand = p->norm_cand; P.idx_cand = p->idx_cand; P.h = reinterpret_cast<u64*>(p->h); P.y_acc = p->y_acc;
    P.sync = p->sync; P.mask_out = mask_out; P.sel_out = sel_out;
    P.d = p->d; P.B = B; P.k = k; P.n_ret = p->n_ret; P.n_cand = p->n_cand; P.n_rt = p->n_rt; P.n_cg = p->n_cg;
    P.n_ret_pad = p->n_ret_pad; P.h_stride = p->h_stride;
    P.Uc = (p->n_cand + 7) / 8;
    P.U1 = P.Uc + p->n_rt;
    P.n_cu = k > 0 ? (p->n_cand + 31) / 32 : 0;
    P.p2_macro = P2_MACRO;
    // groups the scheduler may stage beyond the copy ring in phase 2: what is staged is committed to this CTA, so a
    // deep queue makes the CTAs finish unevenly, a shallow one lets the ring run dry
    P.window = P2_WINDOW;
    P.wait_ns = 1000ull * (unsigned long long)pop_config_snapshot().wait_budget_us;
    const int gs = p->d / 1024;
    const int nblk = B <= 4 ? 1 : 2;
#define POP_CASE(G_, N_) if (gs == G_ && nblk == N_) return p->n_cand <= 32 * KPL_SMALL ? launch_stream<G_, N_, KPL_SMALL>(P, p, st) : launch_stream<G_, N_, KPL_LARGE>(P, p, st);
    POP_CASE(2, 1) POP_CASE(2, 2) POP_CASE(4, 1) POP_CASE(4, 2) POP_CASE(5, 1) POP_CASE(5, 2)
#undef POP_CASE
    return POP_ERR_UNSUPPORTED;
}
