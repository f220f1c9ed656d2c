// Prefilling stage on the tensor cores (Sec. 3.3 "Prefilling Stage"; score of Sec. 3.4 Eq. 3), bf16.
//
//   H[t, i] = silu(Wg[i].X[t]) * (Wu[i].X[t]),   s2[i] = sum_t H[t, i]^2
//
// is a dense contraction over the hidden size (4 L d N flops), so it runs on the 5th-generation
// tensor cores: tcgen05.mma with the accumulators in tensor memory, operands brought into shared
// memory by the TMA engine (cp.async.bulk.tensor, 128-byte swizzle) through an mbarrier pipeline.
//
// What the partition needs from this pass is a RANKING, and the ranking has to be the one exact
// arithmetic gives.  So the pass also produces, per channel, a bound of the error of its energy;
// the few channels whose scores the bounds cannot separate from one of the two rank boundaries
// (Retained | Candidate, Candidate | Pruned) are then re-scored in fp64 (kernels further down) and
// the regions are taken on the mixed scores, which rank like exact ones (argument at
// select_uncertain_kernel).
//
// Unit of work: 128 channels (MMA M = tensor-memory lanes) x 128 tokens (MMA N).  With the channels
// on the lanes one epilogue thread owns one channel and sums over tokens in registers.  The hidden
// size is consumed in chunks of 64 (4 MMAs of K = 16 each for gate and for up); every chunk starts a
// fresh accumulator and the epilogue warps add the chunk results in fp32 registers.  That keeps
// the number of accumulation steps whose rounding is not observable at 4, which is what makes a
// useful error bound possible (see TC_* constants).  Two accumulator sets (2 x 256 columns) take turns,
// so the tensor cores work on chunk c + 1 while chunk c is read out.
//
// Warp roles (320 threads, one CTA per SM, persistent over units):
//   warp 0      TMA producer (one lane): Wg tile, Wu tile, X tile of a 64-wide K slab per stage
//   warp 1      allocates tensor memory; one lane issues the MMAs and the commits
//   warps 2..9  epilogue: warp w reads lanes 32 (w % 4) .. + 31, columns of token half (w - 2) / 4
// Every wait is bounded; a wait that runs out sets the status word and the CTA winds down.
#include <cuda.h>          // CUtensorMap and its enums (the encoder itself is looked up through the runtime)
#include <string.h>

#include "pop_common.cuh"
#include "pop_select.cuh"

namespace {

constexpr int TC_BM = 128;                 // channels per unit
constexpr int TC_BN = 128;                 // tokens per unit
constexpr int TC_BK = 64;                  // K slab of one pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr int TC_STAGES = 4;
constexpr int TC_CHUNK_SLABS = 1;          // accumulate-restart chunk = 64 hidden dimensions (4 MMAs)
constexpr int TC_TRACK = 8;                // the running sums' magnitudes are sampled every TC_TRACK chunks
constexpr int TC_TILE_BYTES = TC_BM * TC_BK * 2;          // 16 KB
constexpr int TC_STAGE_BYTES = 3 * TC_TILE_BYTES;         // Wg, Wu, X
constexpr int TC_THREADS = 320;
constexpr int TC_EPI_WARPS = 8;
constexpr int TC_TMEM_COLS = 512;
constexpr size_t TC_SMEM_BYTES = (size_t)TC_STAGES * TC_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

// Error model of one tcgen05.mma of kind::f16 with an fp32 accumulator (D = C + sum of 16 exact products), as
// measured on B200 with addends placed around the accumulator's last place: every addend is aligned to the
// largest one and cut two bits below that one's last place (an addend below 2^-25 of the largest vanishes), the
// aligned sum is exact, and the result is truncated toward zero to fp32.  Hence
//   |D - exact| < 16 * 2^-25 * M + 2^-23 * |D|  <=  TC_KAPPA * (sum of the magnitudes of the 17 addends),
// with M the largest addend and TC_KAPPA = 2^-21 + 2^-23.
// The sum of magnitudes over one chunk of K is at most |x_chunk|_2 |w_chunk|_2 (Cauchy-Schwarz), and the sum
// of those over the chunks at most |x|_2 |w|_2: the MMA steps of a dot product err by at most
// (steps per chunk) * TC_KAPPA * |x|_2 |w|_2 in all.
// Adding a chunk result to the running fp32 sum rounds by at most 2^-24 of the new sum.  The running sums are
// observed: every TC_TRACK chunks a thread takes the largest magnitude among its sums; between two samples a sum
// moves by at most the Cauchy-Schwarz bounds of the chunks in between, so the magnitudes of all n_chunks sums add up
// to at most TC_TRACK * (sum of the samples + |x|_2 |w|_2).
constexpr float TC_KAPPA = 5.9604644775390625e-07f;         // 2^-21 + 2^-23
constexpr float TC_ADD_ULP = 5.9604644775390625e-08f;      // 2^-24

constexpr unsigned long long TC_WAIT_BUDGET_NS = 200ull * 1000ull * 1000ull;   // per wait

enum { TC_ERR_PRODUCER = 101, TC_ERR_MMA_FULL = 102, TC_ERR_MMA_ACC = 103, TC_ERR_EPILOGUE = 104 };

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
__device__ __forceinline__ u32 mbar_try_wait(u32 bar, u32 parity) {
    u32 ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(2000u)      // the thread may stay suspended this long (ns) inside one try: fewer polls
        : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for the phase with the given parity to complete; gives up after TC_WAIT_BUDGET_NS or when another
// role of the CTA has given up.  Returns false in that case (the caller leaves its loop).
__device__ __forceinline__ bool mbar_wait(u32 bar, u32 parity, volatile int* abort_flag, u32* status, u32 code) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (u32 it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 31u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > TC_WAIT_BUDGET_NS) {
                *abort_flag = 1;
                atomicCAS(status, 0u, code);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(u32 dst, const CUtensorMap* map, int x, int y, u32 bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, fp32 accumulation.
__device__ __forceinline__ void umma_bf16(u32 d_tmem, u64 a_desc, u64 b_desc, u32 idesc, u32 accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(u32 bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(u32 taddr, float (&v)[32]) {
    u32 r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) in the 128-byte swizzle
// the TMA engine wrote: groups of 8 rows are 1024 bytes apart (stride byte offset), the leading offset is unused
// for swizzled K-major tiles (set to 1), descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ u64 smem_desc_sw128(u32 addr) {
    return (u64)((addr & 0x3ffffu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), both K-major
// (bits 15, 16 = 0), N / 8 at bit 17, M / 16 at bit 24.
constexpr u32 TC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((u32)(TC_BN >> 3) << 17) | ((u32)(TC_BM >> 4) << 24);

struct TcParams {
    int L, d, N;
    int n_ct, n_tt, n_pad;        // channel tiles, token tiles, n_ct * 128
    int nk;                       // K slabs of 64
    const float* xnorm;           // [n_tt * 128]  |X[t]|_2, rounded up; 0 past L
    const float* gnorm;           // [n_pad]       |Wg[i]|_2, rounded up; 0 past N
    const float* unorm;           // [n_pad]
    __nv_bfloat16* H;             // [2][n_tt * 128][n_pad] intermediate activations silu(g) u as a bf16 pair (nearest bf16, then
                                  // nearest bf16 of the remainder: 16 significant bits), or NULL when nobody needs them
    double* s2part;               // [2 n_tt][n_pad] partial energies (token half h of token tile tt at 2 tt + h)
    float* bpart;                 // [2 n_tt][n_pad] bounds of their errors
    u32* status;
#ifdef POP_TC_DUMP
    float* dump_g;                // [n_pad][n_tt * 128] raw gate / up sums (debug builds only)
    float* dump_u;
#endif
};

__global__ void __launch_bounds__(TC_THREADS, 1) prefill_tc_kernel(const __grid_constant__ CUtensorMap map_x,
                                                                   const __grid_constant__ CUtensorMap map_g,
                                                                   const __grid_constant__ CUtensorMap map_u,
                                                                   const TcParams P) {
    extern __shared__ unsigned char tc_smem_raw[];
    __shared__ u32 tmem_base_slot;
    __shared__ int abort_flag;

    const u32 raw = smem_u32(tc_smem_raw);
    const u32 tiles = (raw + 1023u) & ~1023u;                      // stage s at tiles + s * TC_STAGE_BYTES
    const u32 bars = tiles + TC_STAGES * TC_STAGE_BYTES;           // 8-byte mbarriers
    const u32 bar_full = bars, bar_empty = bars + 8 * TC_STAGES;
    const u32 bar_acc_full = bars + 16 * TC_STAGES, bar_acc_empty = bar_acc_full + 16, bar_drain = bar_acc_full + 32;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_acc_full + 8 * b, 1); mbar_init(bar_acc_empty + 8 * b, TC_EPI_WARPS); }
        mbar_init(bar_drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const u32 tmem_base = tmem_base_slot;

    const int n_units = P.n_ct * P.n_tt;
    const int n_chunks = (P.nk + TC_CHUNK_SLABS - 1) / TC_CHUNK_SLABS;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            u32 ph = 0;
            bool ok = true;
            int issued = 0;
            for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
                const int ct = unit / P.n_tt, tt = unit - ct * P.n_tt;
                for (int kb = 0; kb < P.nk; ++kb) {
                    ok = mbar_wait(bar_empty + 8 * s, ph ^ 1u, abortp, P.status, TC_ERR_PRODUCER);
                    if (!ok) break;
                    const u32 dst = tiles + (u32)s * TC_STAGE_BYTES, bar = bar_full + 8 * s;
                    mbar_expect_tx(bar, TC_STAGE_BYTES);
                    tma_load_2d(dst, &map_g, kb * TC_BK, ct * TC_BM, bar);
                    tma_load_2d(dst + TC_TILE_BYTES, &map_u, kb * TC_BK, ct * TC_BM, bar);
                    tma_load_2d(dst + 2 * TC_TILE_BYTES, &map_x, kb * TC_BK, tt * TC_BN, bar);
                    ++issued;
                    if (++s == TC_STAGES) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // copies already issued still land in this CTA's shared memory: wait for them (bounded) before leaving.
                // Stage s is the next to fill; the min(issued, STAGES) stages before it may still be in flight.
                const int back = issued < TC_STAGES ? issued : TC_STAGES;
                for (int j = 1; j <= back; ++j) {
                    int sj = s - j;
                    u32 pj = ph;
                    if (sj < 0) { sj += TC_STAGES; pj ^= 1u; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * sj, pj) && global_ns() - t0 < TC_WAIT_BUDGET_NS) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            int s = 0, buf = 0;
            u32 ph = 0, accph[2] = {0u, 0u};
            bool ok = true;
            for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
                for (int c = 0; c < n_chunks && ok; ++c) {
                    ok = mbar_wait(bar_acc_empty + 8 * buf, accph[buf] ^ 1u, abortp, P.status, TC_ERR_MMA_ACC);
                    if (!ok) break;
                    tc_fence_after();
                    const u32 d_g = tmem_base + (u32)buf * 256u, d_u = d_g + 128u;
                    const int kb_end = min(P.nk, (c + 1) * TC_CHUNK_SLABS);
                    for (int kb = c * TC_CHUNK_SLABS; kb < kb_end; ++kb) {
                        ok = mbar_wait(bar_full + 8 * s, ph, abortp, P.status, TC_ERR_MMA_FULL);
                        if (!ok) break;
                        tc_fence_after();
                        const u32 base = tiles + (u32)s * TC_STAGE_BYTES;
                        const u64 dg = smem_desc_sw128(base), du = smem_desc_sw128(base + TC_TILE_BYTES),
                                  dx = smem_desc_sw128(base + 2 * TC_TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < TC_BK / 16; ++k) {
                            const u32 acc = (kb > c * TC_CHUNK_SLABS || k > 0) ? 1u : 0u;
                            // one K = 16 step is 32 bytes along the swizzled row: + 2 in the descriptor's 16-byte units
                            umma_bf16(d_g, dg + 2ull * k, dx + 2ull * k, TC_IDESC, acc);
                            umma_bf16(d_u, du + 2ull * k, dx + 2ull * k, TC_IDESC, acc);
                        }
                        umma_commit(bar_empty + 8 * s);          // the stage is free once these MMAs have read it
                        if (++s == TC_STAGES) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit(bar_acc_full + 8 * buf);         // the chunk's accumulators are complete
                    accph[buf] ^= 1u;
                    buf ^= 1;
                }
            }
            // nothing of this CTA may still be executing on the tensor cores when tensor memory is given back
            umma_commit(bar_drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0u) && global_ns() - t0 < TC_WAIT_BUDGET_NS) {}
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - 2;
        const int quarter = warp & 3;                   // tensor-memory lanes this warp may read: 32 quarter .. + 31
        const int half = ew >> 2;                       // tokens 64 half .. 64 half + 63 of the unit
        const u32 lane_base = ((u32)(quarter * 32)) << 16;
        int buf = 0;
        u32 accph[2] = {0u, 0u};
        bool ok = true;
        // the MMA steps of a chunk, and the part of the chunk additions that the samples do not cover, as a
        // relative bound of |x|_2 |w|_2
        const float eps = (float)(TC_CHUNK_SLABS * (TC_BK / 16)) * TC_KAPPA + (float)TC_TRACK * TC_ADD_ULP;
        for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
            const int ct = unit / P.n_tt, tt = unit - ct * P.n_tt;
            // running sums in pairs: the chunk additions are packed fp32 additions (two round-to-nearest sums per
            // instruction), which halves what the read-out costs the issue slots it shares with everything else
            float2 g2[32], u2[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) { g2[j] = make_float2(0.f, 0.f); u2[j] = make_float2(0.f, 0.f); }
            float track_g = 0.f, track_u = 0.f;           // sums of the sampled largest |running sum|
            for (int c = 0; c < n_chunks; ++c) {
                ok = mbar_wait(bar_acc_full + 8 * buf, accph[buf], abortp, P.status, TC_ERR_EPILOGUE);
                if (!ok) break;
                tc_fence_after();
                const u32 t_g = tmem_base + lane_base + (u32)buf * 256u + (u32)half * 64u, t_u = t_g + 128u;
                // (two loads in flight at a time, the second under the additions of the first, measured no faster)
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    float v[32];
                    tmem_ld32(t_g + 32u * p, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) g2[16 * p + j] = __fadd2_rn(g2[16 * p + j], make_float2(v[2 * j], v[2 * j + 1]));
                    tmem_ld32(t_u + 32u * p, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) u2[16 * p + j] = __fadd2_rn(u2[16 * p + j], make_float2(v[2 * j], v[2 * j + 1]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
                accph[buf] ^= 1u;
                buf ^= 1;
                if ((c % TC_TRACK) == TC_TRACK - 1 || c == n_chunks - 1) {
                    float mg = 0.f, mu = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        mg = fmaxf(mg, fmaxf(fabsf(g2[j].x), fabsf(g2[j].y)));
                        mu = fmaxf(mu, fmaxf(fabsf(u2[j].x), fabsf(u2[j].y)));
                    }
                    track_g += mg;
                    track_u += mu;
                }
            }
            if (!ok) break;
            // h = silu(g) u in fp32, its square summed in fp64, and a bound of what the fp32 pipeline may have lost
            const int ch = ct * TC_BM + quarter * 32 + lane;
#ifdef POP_TC_DUMP
            if (P.dump_g) {
                const size_t o = (size_t)ch * (P.n_tt * TC_BN) + tt * TC_BN + half * 64;
#pragma unroll
                for (int j = 0; j < 64; ++j) { P.dump_g[o + j] = (j & 1) ? g2[j >> 1].y : g2[j >> 1].x; P.dump_u[o + j] = (j & 1) ? u2[j >> 1].y : u2[j >> 1].x; }
            }
#endif
            const float cg = eps * P.gnorm[ch], cu = eps * P.unorm[ch];
            // chunk additions: 2^-24 of every running sum's magnitude, TC_TRACK * (samples + |x| |w|) in all (the
            // second part is inside eps)
            const float ag = (float)TC_TRACK * TC_ADD_ULP * track_g * 1.0001f, au = (float)TC_TRACK * TC_ADD_ULP * track_u * 1.0001f;
            const float* xn = P.xnorm + tt * TC_BN + half * 64;
            double e2 = 0.0;
            float eb = 0.f;
            __nv_bfloat16* hrow = P.H ? P.H + (size_t)(tt * TC_BN + half * 64) * P.n_pad + ch : nullptr;
            const size_t h_lo_off = (size_t)P.n_tt * TC_BN * P.n_pad;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float at = __ldg(xn + j);
                const float dg = at * cg + ag, du = at * cu + au;       // |g - exact|, |u - exact| at most these
                const float gj = (j & 1) ? g2[j >> 1].y : g2[j >> 1].x, uj = (j & 1) ? u2[j >> 1].y : u2[j >> 1].x;
                const float e = __expf(-fmaxf(gj, -80.f));
                const float s = gj * __fdividef(1.f, 1.f + e);          // silu(g)
                const float h = s * uj;
                // |silu'| <= 1.1; the fast exponential and division err by a few ulp, growing with |g|;
                // past g = -80 the clamped exponential differs from the true one by less than |g| 2e-35
                const float rho = (8.f + 1.2f * fabsf(gj)) * 1.1920929e-07f;
                const float dh = 1.1f * dg * fabsf(uj) + (fabsf(s) + 1.1f * dg) * du + rho * fabsf(h) + 2e-35f * fabsf(gj * uj);
                eb += 2.f * fabsf(h) * dh + dh * dh;
                e2 = fma((double)h, (double)h, e2);
                if (hrow) {                                              // a warp writes 64 contiguous bytes per token and part
                    const __nv_bfloat16 hi = __float2bfloat16_rn(h);
                    hrow[(size_t)j * P.n_pad] = hi;
                    hrow[h_lo_off + (size_t)j * P.n_pad] = __float2bfloat16_rn(h - __bfloat162float(hi));
                }
            }
            const size_t slot = (size_t)(2 * tt + half) * P.n_pad + ch;
            P.s2part[slot] = e2;
            P.bpart[slot] = eb * 1.0001f;                               // covers the fp32 rounding of this sum itself
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Row norms |row|_2 of [rows, d] bf16 matrices, rounded up (they are used as bounds), zero for the padding rows
// up to rows_pad.  One warp per row; up to two matrices of the same shape per launch (M1 may be NULL).
// Thread 0 of the grid also clears the words in zero_a / zero_b when they are given.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rownorm_up_kernel(const __nv_bfloat16* __restrict__ M0, const __nv_bfloat16* __restrict__ M1,
                                                         int rows, int rows_pad, int d, float* __restrict__ out0,
                                                         float* __restrict__ out1, u64* zero_a, int* zero_b) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (zero_a) *zero_a = 0ull;
        if (zero_b) *zero_b = 0;
    }
    int r = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const __nv_bfloat16* M = M0;
    float* out = out0;
    if (r >= rows_pad) {
        if (!M1) return;
        r -= rows_pad; M = M1; out = out1;
        if (r >= rows_pad) return;
    }
    float acc = 0.f;
    if (r < rows) {
        const uint4* row = reinterpret_cast<const uint4*>(M + (size_t)r * d);
        const int nv = d >> 3;
        for (int v = lane; v < nv; v += 32) {
            float f[8];
            Elem<__nv_bfloat16>::unpack(__ldg(row + v), f);
#pragma unroll
            for (int j = 0; j < 8; ++j) acc = fmaf(f[j], f[j], acc);
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    // fp32 sum of non-negative terms, at most 1024 + 5 additions per chain (rows are at most 32768 elements):
    // relative error of the sum below 7e-5, of its root below 4e-5
    if (lane == 0) out[r] = sqrtf(acc) * 1.001f;
}

// ---------------------------------------------------------------------------------------------
// Sums the partial energies in a fixed order and forms, per channel, the score a_i = sqrt(s2_i) n_i (Eq. 3)
// with a bound m_i of |a_i - exact score|: |s2 - exact| <= E gives |sqrt(s2) - sqrt(exact)| <= min(sqrt(E), E / sqrt(s2)).
// The largest bound goes to *m_max (bit pattern of a non-negative double).
// ---------------------------------------------------------------------------------------------
__global__ void tc_finish_kernel(const double* __restrict__ s2part, const float* __restrict__ bpart, int n_parts, int n_pad,
                                 const double* __restrict__ norm, int N, double* __restrict__ scores,
                                 double* __restrict__ bounds, u64* __restrict__ m_max, int32_t* __restrict__ rank_to_zero) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    double m = 0.0;
    if (i < N) {
        rank_to_zero[i] = 0;                      // the ranking pass that follows adds into it
        double s2 = 0.0, E = 0.0;
        for (int p = 0; p < n_parts; ++p) {
            s2 += s2part[(size_t)p * n_pad + i];
            E += (double)bpart[(size_t)p * n_pad + i];
        }
        const double r = sqrt(s2);
        double dr = sqrt(E);
        if (r > 0.0) dr = fmin(dr, E / r);
        m = norm[i] * dr * (1.0 + 1e-9);
        scores[i] = r * norm[i];
        bounds[i] = m;
    }
    // block maximum, then one atomic
    __shared__ double red[32];
    for (int off = 16; off; off >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.0;
        for (int off = 16; off; off >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, off));
        if (threadIdx.x == 0) atomicMax(m_max, (u64)__double_as_longlong(m));
    }
}

// ---------------------------------------------------------------------------------------------
// Channels that the bounds cannot place.  Let a_i be the streamed scores, m the largest bound, and tau the
// n-th largest a_i (n = n_ret for the Retained | Candidate boundary, n_ret + n_cand for Candidate | Pruned).
//   a_i > tau + 2m  =>  exact score > tau + m; every channel whose exact score is at least that has a_j > tau,
//                       and fewer than n channels do: i is inside the exact top n.
//   a_i < tau - 2m  =>  exact score < tau - m, while the n channels with a_j >= tau all have exact scores
//                       >= tau - m: i is outside the exact top n.
// The channels in between, for either boundary, are listed (ascending) for exact re-scoring.  Ranking all
// channels by (exact score where re-scored, streamed score elsewhere) then gives the regions of exact
// arithmetic: a channel outside the window keeps its side whichever scores the others carry, by the same two
// counts, and inside the window the order is the exact one.
// When every bound is zero the streamed scores are exact and nothing is listed.
// ---------------------------------------------------------------------------------------------
constexpr int SEL_NT = 1024;

__global__ void __launch_bounds__(SEL_NT) select_uncertain_kernel(const double* __restrict__ scores,
                                                                  const double* __restrict__ bounds,
                                                                  const int32_t* __restrict__ rank, int N, int n_ret, int n_cand,
                                                                  int n_third, const u64* __restrict__ m_max,
                                                                  int32_t* __restrict__ list, int* __restrict__ n_list) {
    __shared__ u32 sm[POP_SELECT_SMEM_WORDS(SEL_NT)];
    __shared__ u64 mw_bits[3];
    __shared__ double tau_sm[3];
    const int tid = threadIdx.x;
    const double m = __longlong_as_double((long long)*m_max);
    if (!(m > 0.0)) { if (tid == 0) *n_list = 0; return; }
    // rank boundaries: Retained | Candidate, Candidate | Pruned and, when the caller wants the prompt's own output,
    // the boundary of its mask inside the Candidate region (n_third = n_ret + k; 0 = none)
    const int n1 = n_ret, n2 = n_ret + n_cand, n3 = n_third;
    const bool b1 = n1 > 0 && n1 < N, b2 = n2 > 0 && n2 < N && n2 != n1, b3 = n3 > 0 && n3 < N && n3 != n1 && n3 != n2;
    const int per = (N + SEL_NT - 1) / SEL_NT;
    const int lo = min(N, tid * per), hi = min(N, lo + per);
    if (tid < 3) { mw_bits[tid] = 0ull; tau_sm[tid] = 0.0; }
    __syncthreads();
    // tau = the streamed score of the channel at rank n - 1 (exactly one channel holds each rank)
    for (int i = tid; i < N; i += SEL_NT) {                  // (coalesced: which thread finds them does not matter)
        const int r = rank[i];
        if (b1 && r == n1 - 1) tau_sm[0] = scores[i];
        if (b2 && r == n2 - 1) tau_sm[1] = scores[i];
        if (b3 && r == n3 - 1) tau_sm[2] = scores[i];
    }
    __syncthreads();
    const double tau1 = tau_sm[0], tau2 = tau_sm[1], tau3 = tau_sm[2];
    // Outside tau +- 2m every channel is placed (argument above).  Inside, the test can use the channel's own bound:
    // with m_W the largest bound inside that window, at most n - 1 channels have a_j + m_j > tau + m_W and at least
    // n have a_j - m_j >= tau - m_W, so a_i - m_i > tau + m_W places i inside the top n and a_i + m_i < tau - m_W
    // outside, by the same two counts.
    const double w = 2.0 * m * (1.0 + 1e-9);
    double mw1 = 0.0, mw2 = 0.0, mw3 = 0.0;
    for (int i = tid; i < N; i += SEL_NT) {
        const double a = scores[i], mi = bounds[i];
        if (b1 && fabs(a - tau1) <= w) mw1 = fmax(mw1, mi);
        if (b2 && fabs(a - tau2) <= w) mw2 = fmax(mw2, mi);
        if (b3 && fabs(a - tau3) <= w) mw3 = fmax(mw3, mi);
    }
    if (mw1 > 0.0) atomicMax(&mw_bits[0], (u64)__double_as_longlong(mw1));
    if (mw2 > 0.0) atomicMax(&mw_bits[1], (u64)__double_as_longlong(mw2));
    if (mw3 > 0.0) atomicMax(&mw_bits[2], (u64)__double_as_longlong(mw3));
    __syncthreads();
    mw1 = __longlong_as_double((long long)mw_bits[0]) * (1.0 + 1e-9);
    mw2 = __longlong_as_double((long long)mw_bits[1]) * (1.0 + 1e-9);
    mw3 = __longlong_as_double((long long)mw_bits[2]) * (1.0 + 1e-9);
    auto open_at = [&](double a, double mi) -> bool {
        return (b1 && fabs(a - tau1) <= w && fabs(a - tau1) <= mi + mw1) || (b2 && fabs(a - tau2) <= w && fabs(a - tau2) <= mi + mw2) ||
               (b3 && fabs(a - tau3) <= w && fabs(a - tau3) <= mi + mw3);
    };
    // the list ascends: every thread a contiguous chunk of channels, read once (the open ones as a bit mask when the
    // chunk has at most 64 channels)
    int cnt = 0;
    u64 open_bits = 0ull;
    for (int i = lo; i < hi; ++i) {
        const bool o = open_at(scores[i], bounds[i]);
        cnt += o;
        if (o && i - lo < 64) open_bits |= 1ull << (i - lo);
    }
    int tot;
    int pos = group_excl_scan<SEL_NT>(cnt, sm, tid, 0, tot);
    if (per <= 64) {
        while (open_bits) {
            const int b = __ffsll((long long)open_bits) - 1;
            list[pos++] = lo + b;
            open_bits &= open_bits - 1ull;
        }
    } else {
        for (int i = lo; i < hi; ++i) {
            if (open_at(scores[i], bounds[i])) list[pos++] = i;
        }
    }
    if (tid == 0) *n_list = tot;
}

// ---------------------------------------------------------------------------------------------
// Exact (fp64) energies of the listed channels on the fp64 matrix path (mma.m8n8k4.f64: D[8x8] += A[8x4] B[4x8],
// every product and sum an IEEE fp64 fused multiply-add).  A warp owns 32 tokens (4 A fragments) x 8 listed
// channels (one B fragment each for their gate and up rows) over the whole hidden size.  Lane (r, c) =
// (lane / 4, lane % 4) holds row r, k slot c of each fragment; within a block of 32 hidden dimensions slot c is
// fed from dimensions 8c .. 8c+7, one per step (a dot product does not care in which order its terms are taken
// as long as both operands agree), so one 16-byte load per row and lane feeds 8 steps, straight from L2 with no
// shared memory: 6 conversions per 8 matrix instructions.
// The token sum of an item is taken in a fixed order and written to part[listed channel][token group];
// rescore_finish_kernel adds the groups in order.
// Does nothing when the list is empty or longer than max_list (then the full fp64 pass runs instead).
// ---------------------------------------------------------------------------------------------
constexpr int RS_CH = 8;
// The four warps of a block share an item: each takes a quarter of the hidden size, and warp 0 adds the four partial
// gate and up sums (in warp order) before the activation.  One warp per item was bound by the length of its dependent
// fp64 MMA chains (84 us whatever the number of items); a quarter of the chain and four times the warps keep the fp64
// tensor path busy.
constexpr int RS_WARPS = 4;
constexpr int RS_TOK_MIN = 16;             // token groups of the shortest items (part[] is sized for them)
constexpr int RS_SHORT_LIST = 256;         // lists up to this length use 16-token items (more, shorter items)

__device__ __forceinline__ void dmma_884(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}
// element s (0..7) of a vector of 8 bf16 values, exactly, as a double
__device__ __forceinline__ double bf16x8_elem(const uint4& v, int s) {
    const u32 w = (s >> 1) == 0 ? v.x : (s >> 1) == 1 ? v.y : (s >> 1) == 2 ? v.z : v.w;
    return (double)__uint_as_float((s & 1) ? (w & 0xffff0000u) : (w << 16));
}

// One warp item: NA A fragments (8 NA tokens from t0) x the 8 listed channels of group grp.
template <int NA>
__device__ __forceinline__ void rescore_item(const __nv_bfloat16* __restrict__ X, int L, int d,
                                             const __nv_bfloat16* __restrict__ Wg, const __nv_bfloat16* __restrict__ Wu,
                                             const int32_t* __restrict__ list, int n, int grp, int t0, int lane,
                                             int kb_lo, int kb_hi, double (&g)[NA][2], double (&u)[NA][2]) {
    const int r = lane >> 2, c = lane & 3;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    const __nv_bfloat16* xr[NA];
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        const int t = t0 + a * 8 + r;
        xr[a] = t < L ? X + (size_t)t * d + 8 * c : nullptr;
    }
    const int li = grp * RS_CH + r;
    const int ch = li < n ? list[li] : -1;
    const __nv_bfloat16* wg = ch >= 0 ? Wg + (size_t)ch * d + 8 * c : nullptr;
    const __nv_bfloat16* wu = ch >= 0 ? Wu + (size_t)ch * d + 8 * c : nullptr;
#pragma unroll
    for (int a = 0; a < NA; ++a) { g[a][0] = g[a][1] = u[a][0] = u[a][1] = 0.0; }
    uint4 vx[NA], vg, vu;
    auto fetch = [&](int kb) {
        const bool in = (kb << 5) + 8 * c < d;          // d is a multiple of 8: a vector is inside or outside
#pragma unroll
        for (int a = 0; a < NA; ++a) vx[a] = (xr[a] && in) ? __ldg(reinterpret_cast<const uint4*>(xr[a] + (kb << 5))) : zero;
        vg = (wg && in) ? __ldg(reinterpret_cast<const uint4*>(wg + (kb << 5))) : zero;
        vu = (wu && in) ? __ldg(reinterpret_cast<const uint4*>(wu + (kb << 5))) : zero;
    };
    if (kb_lo < kb_hi) fetch(kb_lo);
    for (int kb = kb_lo; kb < kb_hi; ++kb) {
        uint4 cx[NA];
#pragma unroll
        for (int a = 0; a < NA; ++a) cx[a] = vx[a];
        const uint4 cg = vg, cu = vu;
        if (kb + 1 < kb_hi) fetch(kb + 1);                // the next block's loads fly during this block's arithmetic
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const double gb = bf16x8_elem(cg, s), ub = bf16x8_elem(cu, s);
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                const double xa = bf16x8_elem(cx[a], s);
                dmma_884(g[a][0], g[a][1], xa, gb);
                dmma_884(u[a][0], u[a][1], xa, ub);
            }
        }
    }
}

// The item's token sum from the complete gate and up sums: lane (r, c) holds token row r of each fragment at listed
// channels 2c, 2c + 1 of the group (tokens past L gave 0); the fragments in the lane, then the 8 token rows (lanes
// r = 0..7 of the same c) by shuffles.
template <int NA>
__device__ __forceinline__ void rescore_item_energy(const double (&g)[NA][2], const double (&u)[NA][2], double& e0, double& e1) {
    e0 = 0.0; e1 = 0.0;
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        const double h0 = silu_f64(g[a][0]) * u[a][0], h1 = silu_f64(g[a][1]) * u[a][1];
        e0 = fma(h0, h0, e0);
        e1 = fma(h1, h1, e1);
    }
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        e0 += __shfl_xor_sync(0xffffffffu, e0, off);
        e1 += __shfl_xor_sync(0xffffffffu, e1, off);
    }
}

// One item by the block's RS_WARPS warps: partial sums over a share of the hidden size each, exchanged through shared
// memory and added by warp 0 in warp order.
template <int NA>
__device__ __forceinline__ void rescore_block_item(const __nv_bfloat16* __restrict__ X, int L, int d,
                                                   const __nv_bfloat16* __restrict__ Wg, const __nv_bfloat16* __restrict__ Wu,
                                                   const int32_t* __restrict__ list, int n, int grp, int t0, int warp, int lane,
                                                   double* xch, double& e0, double& e1) {
    const int nkb = (d + 31) >> 5, per = (nkb + RS_WARPS - 1) / RS_WARPS;
    double g[NA][2], u[NA][2];
    rescore_item<NA>(X, L, d, Wg, Wu, list, n, grp, t0, lane, min(nkb, warp * per), min(nkb, (warp + 1) * per), g, u);
    __syncthreads();                                   // the exchange buffer is free (the item before has been read)
    if (warp > 0) {
#pragma unroll
        for (int a = 0; a < NA; ++a)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                xch[(((warp - 1) * NA + a) * 4 + h) * 32 + lane] = g[a][h];
                xch[(((warp - 1) * NA + a) * 4 + 2 + h) * 32 + lane] = u[a][h];
            }
    }
    __syncthreads();
    e0 = 0.0; e1 = 0.0;
    if (warp == 0) {
#pragma unroll
        for (int w = 1; w < RS_WARPS; ++w)
#pragma unroll
            for (int a = 0; a < NA; ++a)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    g[a][h] += xch[(((w - 1) * NA + a) * 4 + h) * 32 + lane];
                    u[a][h] += xch[(((w - 1) * NA + a) * 4 + 2 + h) * 32 + lane];
                }
        rescore_item_energy<NA>(g, u, e0, e1);
    }
}

// part is [listed channel][n_tb] with n_tb = ceil(L / RS_TOK_MIN); items of 32 tokens fill every second entry and
// leave the other zero, so that rescore_finish_kernel adds n_tb entries either way.
__global__ void __launch_bounds__(32 * RS_WARPS) rescore_list_kernel(const __nv_bfloat16* __restrict__ X, int L, int d,
                                                                      const __nv_bfloat16* __restrict__ Wg,
                                                                      const __nv_bfloat16* __restrict__ Wu,
                                                                      const int32_t* __restrict__ list,
                                                                      const int* __restrict__ n_list, int max_list, int n_tb,
                                                                      double* __restrict__ part) {
    const int n = *n_list;
    if (n <= 0 || n > max_list) return;
    const int lane = threadIdx.x & 31, r = lane >> 2, c = lane & 3;
    const int n_grp = (n + RS_CH - 1) / RS_CH;
    const bool short_items = n <= RS_SHORT_LIST;
    const int n_tg = short_items ? n_tb : (n_tb + 1) / 2;
    const int items = n_grp * n_tg;
    __shared__ double xch[(RS_WARPS - 1) * 4 * 4 * 32];           // partial sums of warps 1.. for up to 4 fragments
    const int warp = threadIdx.x >> 5;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int grp = item / n_tg, tg = item - grp * n_tg;
        double e0, e1;
        if (short_items) rescore_block_item<2>(X, L, d, Wg, Wu, list, n, grp, tg * 16, warp, lane, xch, e0, e1);
        else rescore_block_item<4>(X, L, d, Wg, Wu, list, n, grp, tg * 32, warp, lane, xch, e0, e1);
        if (warp != 0) continue;
        if (r == 0) {
            const int l0 = grp * RS_CH + 2 * c;
            const int slot = short_items ? tg : 2 * tg;
            if (l0 < n) part[(size_t)l0 * n_tb + slot] = e0;
            if (l0 + 1 < n) part[(size_t)(l0 + 1) * n_tb + slot] = e1;
            if (!short_items && slot + 1 < n_tb) {
                if (l0 < n) part[(size_t)l0 * n_tb + slot + 1] = 0.0;
                if (l0 + 1 < n) part[(size_t)(l0 + 1) * n_tb + slot + 1] = 0.0;
            }
        }
    }
}

// Scores of the re-scored channels: exact energy = sum of the token groups in order, I_i = sqrt(s2_i) n_i, bound 0.
// With a list longer than max_list every channel was re-scored by the full fp64 pass, whose token ranges
// (s2part_full [n_split][N]) are added here in order.  Also clears the rank entries that the ranking pass that
// follows recomputes: those of the listed channels, or all of them when every score was replaced.
__global__ void rescore_finish_kernel(const int32_t* __restrict__ list, const int* __restrict__ n_list, int max_list,
                                      const double* __restrict__ part, int n_tb, const double* __restrict__ s2part_full,
                                      int n_split, const double* __restrict__ norm, int N, double* __restrict__ scores,
                                      double* __restrict__ bounds, int32_t* __restrict__ rank_to_zero) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int n = *n_list;
    if (n > max_list) {
        if (i < N) {
            rank_to_zero[i] = 0;
            double s = 0.0;
            for (int y = 0; y < n_split; ++y) s += s2part_full[(size_t)y * N + i];
            scores[i] = sqrt(s) * norm[i];
            bounds[i] = 0.0;
        }
        return;
    }
    if (i >= n) return;
    const int ch = list[i];
    double s = 0.0;
    for (int tb = 0; tb < n_tb; ++tb) s += part[(size_t)i * n_tb + tb];
    scores[ch] = sqrt(s) * norm[ch];
    bounds[ch] = 0.0;
    rank_to_zero[ch] = 0;
}

// ---------------------------------------------------------------------------------------------
// The prompt's own output under the pruned structure (Sec. 3.4: "the prefilling pass is then completed under the
// resulting pruning structure"): Y[t, :] = sum over the active channels i of Wd[:, i] H[t, i], the active channels
// being Retained plus the k best Candidates by prefill score.  H comes from the scoring pass as a bf16 pair
// (high part + low part: a single bf16 would leave 2^-9 of every term, too much for outputs that nearly cancel); the
// channels outside the mask are cleared in H (mask_h_kernel), so that the contraction can run over all N channels on
// plain K-major operands: A = H_hi and H_lo [tokens, N], B = Wd [d, N], all as they lie in memory, no gather.  Both
// parts of a K slab are multiplied with the same Wd tile.
// Unit: 128 tokens x 128 outputs over all channels; accumulator in tensor memory (two sets take turns over the
// units); warp 0 TMA producer, warp 1 MMA issue, warps 2..5 epilogue (warp w reads lanes 32 (w % 4) ..).
// ---------------------------------------------------------------------------------------------
constexpr int DN_STAGES = 4;
constexpr int DN_STAGE_BYTES = 3 * TC_TILE_BYTES;        // H_hi, H_lo, Wd
constexpr int DN_THREADS = 192;
constexpr size_t DN_SMEM_BYTES = (size_t)DN_STAGES * DN_STAGE_BYTES + 1024 + 256;
enum { DN_ERR_PRODUCER = 111, DN_ERR_MMA_FULL = 112, DN_ERR_MMA_ACC = 113, DN_ERR_EPILOGUE = 114 };

struct DownParams {
    int L, d, n_tt, n_jt, nk;
    int lo_row;                   // first row of the low parts in the H tensor map
    __nv_bfloat16* Y;             // [L, d]
    u32* status;
};

__global__ void __launch_bounds__(DN_THREADS, 1) prefill_down_kernel(const __grid_constant__ CUtensorMap map_h,
                                                                     const __grid_constant__ CUtensorMap map_d,
                                                                     const DownParams P) {
    extern __shared__ unsigned char dn_smem_raw[];
    __shared__ u32 tmem_base_slot;
    __shared__ int abort_flag;
    const u32 raw = smem_u32(dn_smem_raw);
    const u32 tiles = (raw + 1023u) & ~1023u;
    const u32 bars = tiles + DN_STAGES * DN_STAGE_BYTES;
    const u32 bar_full = bars, bar_empty = bars + 8 * DN_STAGES;
    const u32 bar_acc_full = bars + 16 * DN_STAGES, bar_acc_empty = bar_acc_full + 16, bar_drain = bar_acc_full + 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abortp = &abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < DN_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_acc_full + 8 * b, 1); mbar_init(bar_acc_empty + 8 * b, 4); }
        mbar_init(bar_drain, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const u32 tmem_base = tmem_base_slot;
    const int n_units = P.n_tt * P.n_jt;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0, issued = 0;
            u32 ph = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
                const int tt = unit / P.n_jt, jt = unit - tt * P.n_jt;
                for (int kb = 0; kb < P.nk; ++kb) {
                    ok = mbar_wait(bar_empty + 8 * s, ph ^ 1u, abortp, P.status, DN_ERR_PRODUCER);
                    if (!ok) break;
                    const u32 dst = tiles + (u32)s * DN_STAGE_BYTES, bar = bar_full + 8 * s;
                    mbar_expect_tx(bar, DN_STAGE_BYTES);
                    tma_load_2d(dst, &map_h, kb * TC_BK, tt * 128, bar);
                    tma_load_2d(dst + TC_TILE_BYTES, &map_h, kb * TC_BK, P.lo_row + tt * 128, bar);
                    tma_load_2d(dst + 2 * TC_TILE_BYTES, &map_d, kb * TC_BK, jt * 128, bar);
                    ++issued;
                    if (++s == DN_STAGES) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                const int back = issued < DN_STAGES ? issued : DN_STAGES;
                for (int j = 1; j <= back; ++j) {
                    int sj = s - j;
                    u32 pj = ph;
                    if (sj < 0) { sj += DN_STAGES; pj ^= 1u; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(bar_full + 8 * sj, pj) && global_ns() - t0 < TC_WAIT_BUDGET_NS) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0, buf = 0;
            u32 ph = 0, accph[2] = {0u, 0u};
            bool ok = true;
            for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
                ok = mbar_wait(bar_acc_empty + 8 * buf, accph[buf] ^ 1u, abortp, P.status, DN_ERR_MMA_ACC);
                if (!ok) break;
                tc_fence_after();
                const u32 dacc = tmem_base + (u32)buf * 128u;
                for (int kb = 0; kb < P.nk; ++kb) {
                    ok = mbar_wait(bar_full + 8 * s, ph, abortp, P.status, DN_ERR_MMA_FULL);
                    if (!ok) break;
                    tc_fence_after();
                    const u32 base = tiles + (u32)s * DN_STAGE_BYTES;
                    const u64 da = smem_desc_sw128(base), dl = smem_desc_sw128(base + TC_TILE_BYTES),
                              db = smem_desc_sw128(base + 2 * TC_TILE_BYTES);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {
                        umma_bf16(dacc, da + 2ull * k, db + 2ull * k, TC_IDESC, (kb > 0 || k > 0) ? 1u : 0u);
                        umma_bf16(dacc, dl + 2ull * k, db + 2ull * k, TC_IDESC, 1u);
                    }
                    umma_commit(bar_empty + 8 * s);
                    if (++s == DN_STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                umma_commit(bar_acc_full + 8 * buf);
                accph[buf] ^= 1u;
                buf ^= 1;
            }
            umma_commit(bar_drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar_drain, 0u) && global_ns() - t0 < TC_WAIT_BUDGET_NS) {}
        }
    } else {
        const int quarter = warp & 3;
        const u32 lane_base = ((u32)(quarter * 32)) << 16;
        int buf = 0;
        u32 accph[2] = {0u, 0u};
        bool ok = true;
        for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
            const int tt = unit / P.n_jt, jt = unit - tt * P.n_jt;
            ok = mbar_wait(bar_acc_full + 8 * buf, accph[buf], abortp, P.status, DN_ERR_EPILOGUE);
            if (!ok) break;
            tc_fence_after();
            const int t = tt * 128 + quarter * 32 + lane;
            const int j0 = jt * 128;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                float v[32];
                tmem_ld32(tmem_base + lane_base + (u32)buf * 128u + 32u * p, v);
                if (t < P.L) {
                    uint4* dst = reinterpret_cast<uint4*>(P.Y + (size_t)t * P.d + j0 + 32 * p);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (j0 + 32 * p + 8 * q < P.d) {                    // d is a multiple of 8
                            uint4 o;
                            o.x = (u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 0])) | ((u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 1])) << 16);
                            o.y = (u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 2])) | ((u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 3])) << 16);
                            o.z = (u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 4])) | ((u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 5])) << 16);
                            o.w = (u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 6])) | ((u32)__bfloat16_as_ushort(__float2bfloat16_rn(v[8 * q + 7])) << 16);
                            dst[q] = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
            accph[buf] ^= 1u;
            buf ^= 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256) : "memory");
    }
}

// Clears, in H [rows][n_pad], the columns of the channels outside the prompt's mask: rank[i] >= n_active.
__global__ void mask_h_kernel(__nv_bfloat16* __restrict__ H, int rows, int n_pad, int N, const int32_t* __restrict__ rank, int n_active) {
    const int vec_per_row = n_pad >> 3;
    const size_t total = (size_t)rows * vec_per_row;
    for (size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (size_t)gridDim.x * blockDim.x) {
        const int c0 = (int)(o % vec_per_row) * 8;
        u32 keep = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) keep |= (c0 + e < N && rank[c0 + e] < n_active) ? (1u << e) : 0u;
        if (keep == 0xffu) continue;
        uint4* p = reinterpret_cast<uint4*>(H) + o;
        uint4 v = *p;
        u32* w = reinterpret_cast<u32*>(&v);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (!((keep >> e) & 1u)) w[e >> 1] &= (e & 1) ? 0x0000ffffu : 0xffff0000u;
        *p = v;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        (void)cudaGetLastError();
        return (EncodeTiledFn)f;
    }();
    return fn;
}

// [rows, d] bf16 row-major (row pitch `pitch` elements); box = 64 columns (128 bytes, the swizzle span) x 128 rows;
// out-of-range elements read as zero
int make_map(CUtensorMap* map, const void* base, int rows, int d, int pitch = 0) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) { pop_set_cuda_error(cudaErrorNotSupported, "cuTensorMapEncodeTiled is not available from this driver"); return POP_ERR_CUDA; }
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)(pitch ? pitch : d) * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)TC_BM};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        pop_set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled rejected the tensor (base must be 16-byte aligned, row pitch a multiple of 16 bytes)");
        return POP_ERR_CUDA;
    }
    return POP_OK;
}

}  // namespace

#ifdef POP_TC_DUMP
// Debug builds: the next tensor-core passes also write their raw gate / up sums ([n_pad][n_tt * 128] floats each).
static float *g_tc_dump_g = nullptr, *g_tc_dump_u = nullptr;
extern "C" void pop_debug_tc_dump(float* g, float* u) { g_tc_dump_g = g; g_tc_dump_u = u; }
#endif

bool pop_prefill_tc_supported(int d, pop_dtype_t dt) { return dt == POP_BF16 && d >= TC_BK && d % 8 == 0; }

void pop_prefill_tc_plan(int L, int d, int N, PrefillTcPlan* plan) {
    plan->n_ct = (N + TC_BM - 1) / TC_BM;
    plan->n_tt = (L + TC_BN - 1) / TC_BN;
    plan->n_pad = plan->n_ct * TC_BM;
    plan->l_pad = plan->n_tt * TC_BN;
    plan->n_parts = 2 * plan->n_tt;
    plan->n_tb = (L + RS_TOK_MIN - 1) / RS_TOK_MIN;   // token groups of the list re-scoring kernel
    // without the blocked fp64 pass (hidden sizes that are not a multiple of 16) the list kernel takes any length
    plan->max_list = pop_prefill_s2_gemm_supported(d) ? (N < POP_PREFILL_MAX_LIST ? N : POP_PREFILL_MAX_LIST) : N;
}

int pop_launch_weight_rownorms(const void* Wg, const void* Wu, int N, int n_pad, int d, float* gnorm, float* unorm, cudaStream_t st) {
    rownorm_up_kernel<<<(2 * n_pad + 7) / 8, 256, 0, st>>>((const __nv_bfloat16*)Wg, (const __nv_bfloat16*)Wu, N, n_pad, d, gnorm,
                                                           unorm, nullptr, nullptr);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_prefill_tc_encode_weight_maps(const void* Wg, const void* Wu, int N, int d, void* map_g, void* map_u) {
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    int rc = make_map(reinterpret_cast<CUtensorMap*>(map_g), Wg, N, d);
    if (rc == POP_OK) rc = make_map(reinterpret_cast<CUtensorMap*>(map_u), Wu, N, d);
    return rc;
}

int pop_launch_prefill_tc(const void* X, int L, int d, const void* Wg, const void* Wu, int N, const WeightStats& ws,
                          const PrefillTcScratch& s, double* scores, double* bounds, u32* status, int sm_count,
                          cudaStream_t st) {
    PrefillTcPlan plan;
    pop_prefill_tc_plan(L, d, N, &plan);
    CUtensorMap mx, mg, mu;
    int rc = make_map(&mx, X, L, d);
    if (rc != POP_OK) return rc;
    if (ws.map_g && ws.map_u) {
        memcpy(&mg, ws.map_g, sizeof(CUtensorMap));
        memcpy(&mu, ws.map_u, sizeof(CUtensorMap));
    } else {
        rc = make_map(&mg, Wg, N, d);
        if (rc == POP_OK) rc = make_map(&mu, Wu, N, d);
        if (rc != POP_OK) return rc;
    }
    // token norms; the same launch clears the largest-bound word and the list length
    rownorm_up_kernel<<<(plan.l_pad + 7) / 8, 256, 0, st>>>((const __nv_bfloat16*)X, nullptr, L, plan.l_pad, d, s.xnorm, nullptr,
                                                            s.m_max, s.n_list);
    POP_LAUNCHED();

    static thread_local int cfg_dev = -1;
    int dev = 0;
    POP_CUDA(cudaGetDevice(&dev));
    if (cfg_dev != dev) {
        POP_CUDA(cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_BYTES));
        cfg_dev = dev;
    }
    TcParams P;
    P.L = L; P.d = d; P.N = N;
    P.n_ct = plan.n_ct; P.n_tt = plan.n_tt; P.n_pad = plan.n_pad;
    P.nk = (d + TC_BK - 1) / TC_BK;
    P.xnorm = s.xnorm; P.gnorm = ws.gnorm; P.unorm = ws.unorm;
    P.s2part = s.s2part; P.bpart = s.bpart; P.status = status;
    P.H = (__nv_bfloat16*)s.H;
#ifdef POP_TC_DUMP
    P.dump_g = g_tc_dump_g; P.dump_u = g_tc_dump_u;
#endif
    const int units = plan.n_ct * plan.n_tt;
    const int grid = units < sm_count ? units : sm_count;
    prefill_tc_kernel<<<grid, TC_THREADS, TC_SMEM_BYTES, st>>>(mx, mg, mu, P);
    POP_LAUNCHED();

    tc_finish_kernel<<<(N + 255) / 256, 256, 0, st>>>(s.s2part, s.bpart, plan.n_parts, plan.n_pad, ws.norm, N, scores, bounds,
                                                      s.m_max, s.rank);
    POP_LAUNCHED();
    return POP_OK;
}

int pop_launch_prefill_rescore(const void* X, int L, int d, const void* Wg, const void* Wu, int N, const double* norm,
                               int n_ret, int n_cand, int n_third, const PrefillTcScratch& s, double* scores, double* bounds,
                               int sm_count, cudaStream_t st) {
    PrefillTcPlan plan;
    pop_prefill_tc_plan(L, d, N, &plan);
    const int rc0 = pop_launch_ranks(scores, N, s.rank, sm_count, st);          // s.rank was cleared by tc_finish_kernel
    if (rc0 != POP_OK) return rc0;
    select_uncertain_kernel<<<1, SEL_NT, 0, st>>>(scores, bounds, s.rank, N, n_ret, n_cand, n_third, s.m_max, s.list, s.n_list);
    POP_LAUNCHED();
    rescore_list_kernel<<<sm_count * 8, 32 * RS_WARPS, 0, st>>>((const __nv_bfloat16*)X, L, d, (const __nv_bfloat16*)Wg,
                                                        (const __nv_bfloat16*)Wu, s.list, s.n_list, plan.max_list,
                                                        plan.n_tb, s.part);
    POP_LAUNCHED();
    // the full fp64 pass runs only when the list is longer than max_list (its blocks return at once otherwise)
    if (plan.max_list < N) {
        const int rc = pop_launch_prefill_s2_gemm_parts_if(X, L, d, Wg, Wu, N, POP_BF16, s.s2part_full, s.n_list, plan.max_list, st);
        if (rc != POP_OK) return rc;
    }
    rescore_finish_kernel<<<(N + 255) / 256, 256, 0, st>>>(s.list, s.n_list, plan.max_list, s.part, plan.n_tb, s.s2part_full,
                                                           pop_prefill_s2_gemm_splits(L), norm, N, scores, bounds, s.rank);
    POP_LAUNCHED();
    return POP_OK;
}

bool pop_prefill_output_supported(int d, int N, pop_dtype_t dt) { return pop_prefill_tc_supported(d, dt) && N % 8 == 0; }

int pop_launch_prefill_output(void* H, int L, int d, const void* Wd, int N, const int32_t* rank, int n_active, void* Y,
                              u32* status, int sm_count, cudaStream_t st) {
    PrefillTcPlan plan;
    pop_prefill_tc_plan(L, d, N, &plan);
    mask_h_kernel<<<sm_count * 8, 256, 0, st>>>((__nv_bfloat16*)H, 2 * plan.l_pad, plan.n_pad, N, rank, n_active);
    POP_LAUNCHED();
    CUtensorMap mh, md;
    int rc = make_map(&mh, H, 2 * plan.l_pad, plan.n_pad);
    if (rc == POP_OK) rc = make_map(&md, Wd, d, N);
    if (rc != POP_OK) return rc;
    static thread_local int cfg_dev = -1;
    int dev = 0;
    POP_CUDA(cudaGetDevice(&dev));
    if (cfg_dev != dev) {
        POP_CUDA(cudaFuncSetAttribute(prefill_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DN_SMEM_BYTES));
        cfg_dev = dev;
    }
    DownParams P;
    P.L = L; P.d = d; P.n_tt = plan.n_tt; P.n_jt = (d + 127) / 128; P.nk = plan.n_pad / TC_BK;
    P.lo_row = plan.l_pad;
    P.Y = (__nv_bfloat16*)Y; P.status = status;
    const int units = P.n_tt * P.n_jt;
    prefill_down_kernel<<<units < sm_count ? units : sm_count, DN_THREADS, DN_SMEM_BYTES, st>>>(mh, md, P);
    POP_LAUNCHED();
    return POP_OK;
}
