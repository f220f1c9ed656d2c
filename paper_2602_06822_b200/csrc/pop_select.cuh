// Exact top-k selection on 64-bit keys by a group of NT threads (NT a multiple of 32).
//
// Order: larger key first; equal keys by lower index first.  This is the total order
// (score descending, channel id ascending) used for the regions of Sec. 3.3 and for the
// per-step choice among the candidates: index order equals channel order because every index
// list in the library is ascending by channel id.
//
// The group synchronises with the named barrier `bar` (bar.sync bar, NT); bar 0 with
// NT == blockDim.x is __syncthreads().
#pragma once
#include "pop_common.cuh"

#define POP_SELECT_SMEM_WORDS(NT) (256 + 4)

template <int NT>
__device__ __forceinline__ void group_sync(int bar) {
    asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(NT) : "memory");
}

// Exclusive prefix sum of one int per thread over the group; `total` gets the group sum.
// sm: NT/32 + 1 words.  Contains two group barriers.
template <int NT>
__device__ __forceinline__ int group_excl_scan(int v, u32* sm, int tid, int bar, int& total) {
    const int lane = tid & 31, w = tid >> 5;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    group_sync<NT>(bar);                       // previous users of sm are done
    if (lane == 31) sm[w] = (u32)incl;
    group_sync<NT>(bar);
    int base = 0, tot = 0;
#pragma unroll
    for (int j = 0; j < NT / 32; ++j) {
        int t = (int)sm[j];
        if (j < w) base += t;
        tot += t;
    }
    total = tot;
    return base + incl - v;
}

// Finds thr = the k-th largest of keys[0..n) (1 <= k <= n) and need_eq = how many of the keys
// equal to thr are inside the top k.  Keys may live in shared or global memory.
// sm: POP_SELECT_SMEM_WORDS(NT) words.  All NT threads must call it with the same arguments.
template <int NT>
__device__ void radix_select_kth(const u64* keys, int n, int k, u32* sm, int tid, int bar,
                                 u64& thr, int& need_eq) {
    const int lane = tid & 31;
    // Bits on which the keys differ: passes above the highest differing bit are skipped.
    u64 k0 = keys[0], diff = 0;
    for (int i = tid; i < n; i += NT) diff |= keys[i] ^ k0;
#pragma unroll
    for (int off = 16; off; off >>= 1) diff |= __shfl_xor_sync(0xffffffffu, diff, off);
    group_sync<NT>(bar);
    if (tid == 0) { sm[256] = 0; sm[257] = 0; }
    group_sync<NT>(bar);
    if (lane == 0) {                                        // OR across warps, two 32-bit halves
        atomicOr(&sm[256], (u32)(diff & 0xffffffffu));
        atomicOr(&sm[257], (u32)(diff >> 32));
    }
    group_sync<NT>(bar);
    diff = ((u64)sm[257] << 32) | (u64)sm[256];
    group_sync<NT>(bar);
    int top = diff ? (63 - __clzll((long long)diff)) : -1;  // highest differing bit
    u64 prefix, mhi;
    int shift;
    if (top < 0) {                                          // all keys equal
        thr = k0; need_eq = k; return;
    }
    shift = (top / 8) * 8;
    mhi = (shift + 8 >= 64) ? 0ull : (~0ull << (shift + 8));
    prefix = k0 & mhi;
    int rem = k;
    for (; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) sm[i] = 0;
        group_sync<NT>(bar);
        for (int i = tid; i < n; i += NT) {
            u64 key = keys[i];
            if ((key & mhi) == prefix) atomicAdd(&sm[(u32)(key >> shift) & 255u], 1u);
        }
        group_sync<NT>(bar);
        if (tid < 32) {
            u32 c[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = sm[8 * lane + j]; tot += c[j]; }
            u32 incl = tot;                                 // inclusive suffix sum over lanes
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                u32 t = __shfl_down_sync(0xffffffffu, incl, off);
                if (lane + off < 32) incl += t;
            }
            u32 above = incl - tot;                         // keys in bins of higher lanes
            if (above < (u32)rem && (u32)rem <= above + tot) {
                u32 cum = above;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (cum + c[j] >= (u32)rem) { sm[256] = 8 * lane + j; sm[257] = cum; break; }
                    cum += c[j];
                }
            }
        }
        group_sync<NT>(bar);
        u32 b = sm[256];
        rem -= (int)sm[257];
        prefix |= (u64)b << shift;
        mhi |= 0xffull << shift;
        group_sync<NT>(bar);
    }
    thr = prefix;
    need_eq = rem;
}

// Membership in the top k given (thr, need_eq) from radix_select_kth: key > thr, or key == thr
// and fewer than need_eq equal keys precede it.  The walk below gives every thread a
// contiguous chunk of indices so that "precede" is a prefix count.
//
// Calls emit(i, selected, pos) for every index i in [0, n) in ascending order per thread, where
// pos is the rank of i among the selected indices (ascending index order) when selected.
// sm: NT/32 + 1 words.
template <int NT, typename Emit>
__device__ void select_walk(const u64* keys, int n, u64 thr, int need_eq, u32* sm, int tid, int bar,
                            Emit emit) {
    const int per = (n + NT - 1) / NT;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    int eq = 0;
    for (int i = lo; i < hi; ++i) eq += (keys[i] == thr);
    int tot;
    int eq_before = group_excl_scan<NT>(eq, sm, tid, bar, tot);
    int cnt = 0, e = eq_before;
    for (int i = lo; i < hi; ++i) {
        u64 key = keys[i];
        bool s = key > thr;
        if (key == thr) { s = e < need_eq; ++e; }
        cnt += s;
    }
    int pos = group_excl_scan<NT>(cnt, sm, tid, bar, tot);
    e = eq_before;
    for (int i = lo; i < hi; ++i) {
        u64 key = keys[i];
        bool s = key > thr;
        if (key == thr) { s = e < need_eq; ++e; }
        emit(i, s, pos);
        pos += s;
    }
}
