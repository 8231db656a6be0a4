// Block-wide Eq. 3 selection shared by the stand-alone select kernel and the
// fused layer-step kernel.  Each row of the previous region gets the 64-bit key
//   (order-preserving image of the float score) << 32 | position,
// so "score ascending, then position ascending" is plain unsigned order and all
// keys are distinct.  The K lowest keys are found without sorting:
//   K >= p      keep all;   K == 0  drop all;
//   K == p - 1  (steady state of Section 4.2, one eviction per step) drop the maximum key;
//   otherwise   most-significant-digit-first radix select, 8 bits per pass,
//               stopping as soon as the bin of the K-th key is taken whole.
// The result is a threshold on a masked key: keep iff (key & mask) <= thr.
#pragma once

#include "adsa_dev.cuh"

namespace adsa {

constexpr int kSelThreads = 256;   // the block size both callers use (one histogram bin per thread)
constexpr int kSelWarps = kSelThreads / 32;
constexpr uint8_t kCandNextBit = 4;  // region byte, bit 2: the row is in the previous region at cur_pos + 1

__device__ __forceinline__ uint32_t orderable(float s)
{
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelScratch {                 // static shared memory of the calling kernel
    int cnt[3];                     // row counts indexed by region id (prefix, previous, local)
    int hist[256];
    unsigned long long max_key;
    int digit, krem, bin;
};

struct SelResult {
    int n_pre, n_loc, p, K;
    unsigned long long mask, thr;
    bool drop_all;
    __device__ __forceinline__ bool keeps(uint8_t region, unsigned long long key) const
    {
        int reg = region & 3;
        if (reg != kRegionPrevious) return true;   // prefix, local; invalid rows are flagged, never silently dropped
        return !drop_all && (key & mask) <= thr;
    }
};

// Barrier the selecting threads meet at: the whole block, or (persistent kernel) the 256 consumer
// threads alone on a named barrier while the copy-issuing warp runs on.
struct BlockSync { static __device__ __forceinline__ void sync() { __syncthreads(); } };
struct ConsumerSync { static __device__ __forceinline__ void sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); } };

// Fills sm_keys[0..n) and region[0..n) (region id in bits 0-1, kCandNextBit) and returns the
// threshold.  Must be called by kSelThreads threads with threadIdx.x = 0 .. kSelThreads-1.
template <class Sync = BlockSync>
__device__ inline SelResult block_select(const DevCtx &c, const int32_t *__restrict__ pos,
                                         const float *__restrict__ scores, int n, int cur_pos, int budget_rows,
                                         unsigned long long *sm_keys, uint8_t *region, SelScratch &s)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < 3) s.cnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) s.max_key = 0ull;
    Sync::sync();

    unsigned long long my_max = 0ull;
    for (int base = 0; base < n; base += kSelThreads) {
        int slot = base + threadIdx.x;
        int reg = kRegionInvalid;
        if (slot < n) {
            int ps = pos[slot];
            reg = region_of(c, ps, cur_pos);
            uint8_t rb = (uint8_t)reg;
            if (reg != kRegionInvalid && region_of(c, ps, cur_pos + 1) == kRegionPrevious) rb |= kCandNextBit;
            region[slot] = rb;
            unsigned long long key = ~0ull;
            if (reg == kRegionPrevious) {
                // the K lowest keys are kept: the score itself (Eq. 3), or its complement when the highest are wanted
                // (attention mass); the position breaks ties either way, lower first
                const uint32_t hi = c.score_mode == 1 ? ~orderable(scores[slot]) : orderable(scores[slot]);
                key = ((unsigned long long)hi << 32) | (uint32_t)ps;
                my_max = key > my_max ? key : my_max;
            }
            sm_keys[slot] = key;
        }
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            unsigned b = __ballot_sync(0xffffffffu, reg == r);
            if (lane == 0 && b) atomicAdd(&s.cnt[r], __popc(b));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, my_max, o);
        my_max = other > my_max ? other : my_max;
    }
    if (lane == 0) atomicMax(&s.max_key, my_max);
    Sync::sync();

    SelResult r;
    r.n_pre = s.cnt[kRegionPrefix]; r.n_loc = s.cnt[kRegionLocal]; r.p = s.cnt[kRegionPrevious];
    int K = budget_rows - r.n_pre - r.n_loc - 1;
    K = K < 0 ? 0 : (K > r.p ? r.p : K);
    r.K = K;
    r.mask = 0ull; r.thr = 0ull; r.drop_all = false;   // every key passes
    if (K >= r.p) {
    } else if (K == 0) {
        r.drop_all = true;
    } else if (K == r.p - 1) {
        r.mask = ~0ull; r.thr = s.max_key - 1ull;      // keys are distinct: everything below the maximum
    } else {
        unsigned long long mask = 0ull, thr = 0ull;
        int k_rem = K;
        for (int shift = 56; shift >= 0; shift -= 8) {
            s.hist[threadIdx.x] = 0;
            Sync::sync();
            for (int slot = threadIdx.x; slot < n; slot += kSelThreads) {
                unsigned long long key = sm_keys[slot];
                if ((region[slot] & 3) == kRegionPrevious && (key & mask) == thr)
                    atomicAdd(&s.hist[(int)((key >> shift) & 255ull)], 1);
            }
            Sync::sync();
            if (warp == 0) {                     // find the bin holding the k_rem-th key of the current prefix
                int h[8], tot = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { h[i] = s.hist[lane * 8 + i]; tot += h[i]; }
                int incl = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    int t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                int excl = incl - tot;
                if (excl < k_rem && k_rem <= incl) {
                    int cum = excl;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (cum < k_rem && k_rem <= cum + h[i]) { s.digit = lane * 8 + i; s.krem = k_rem - cum; s.bin = h[i]; }
                        cum += h[i];
                    }
                }
            }
            Sync::sync();
            thr |= (unsigned long long)s.digit << shift;
            mask |= 255ull << shift;
            k_rem = s.krem;
            int bin = s.bin;
            Sync::sync();
            if (k_rem == bin) break;             // the whole bin is kept: masked compare decides
        }
        r.mask = mask; r.thr = thr;
    }
    return r;
}

// Section 4.1 partition without a division per row: for a given current position the local window
// is "pos >= lo", lo = first position of grid row (current row - rows_back), so a row's region is
// two comparisons.  Equivalent to region_of.
struct RegionCut {
    int cur, lo;   // lo = INT_MAX when the current position is still inside the text condition
};
__device__ __forceinline__ RegionCut region_cut(const DevCtx &c, int cur_pos)
{
    RegionCut r;
    r.cur = cur_pos;
    r.lo = 0x7fffffff;
    if (cur_pos >= c.n_text) {
        int row = (cur_pos - c.n_text) / c.grid_w - c.rows_back;
        r.lo = c.n_text + (row > 0 ? row : 0) * c.grid_w;
    }
    return r;
}
__device__ __forceinline__ int region_by_cut(const DevCtx &c, const RegionCut &k, int pos)
{
    if (pos < 0 || pos >= k.cur) return kRegionInvalid;
    if (pos < c.n_prefix) return kRegionPrefix;
    return pos >= k.lo ? kRegionLocal : kRegionPrevious;
}

// The same selection done by ONE warp (the warp-per-stream kernel): no block barrier, only
// __syncwarp.  hist is 256 ints of the warp's own shared memory.  All 32 lanes must call it.
__device__ inline SelResult warp_select(const DevCtx &c, const int32_t *pos, const float *scores, int n, int cur_pos,
                                        int budget_rows, unsigned long long *sm_keys, uint8_t *region, int *hist)
{
    const int lane = threadIdx.x & 31;
    int cnt[3] = {0, 0, 0};
    unsigned long long my_max = 0ull;
    const RegionCut cut_now = region_cut(c, cur_pos), cut_next = region_cut(c, cur_pos + 1);
    for (int base = 0; base < n; base += 32) {
        int slot = base + lane;
        int reg = kRegionInvalid;
        if (slot < n) {
            int ps = pos[slot];
            reg = region_by_cut(c, cut_now, ps);
            uint8_t rb = (uint8_t)reg;
            if (reg != kRegionInvalid && region_by_cut(c, cut_next, ps) == kRegionPrevious) rb |= kCandNextBit;
            region[slot] = rb;
            unsigned long long key = ~0ull;
            if (reg == kRegionPrevious) {
                key = ((unsigned long long)orderable(scores[slot]) << 32) | (uint32_t)ps;
                my_max = key > my_max ? key : my_max;
            }
            sm_keys[slot] = key;
        }
#pragma unroll
        for (int r = 0; r < 3; ++r) cnt[r] += __popc(__ballot_sync(0xffffffffu, reg == r));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, my_max, o);
        my_max = other > my_max ? other : my_max;
    }
    __syncwarp();
    SelResult r;
    r.n_pre = cnt[kRegionPrefix]; r.n_loc = cnt[kRegionLocal]; r.p = cnt[kRegionPrevious];
    int K = budget_rows - r.n_pre - r.n_loc - 1;
    K = K < 0 ? 0 : (K > r.p ? r.p : K);
    r.K = K;
    r.mask = 0ull; r.thr = 0ull; r.drop_all = false;
    if (K >= r.p) {
    } else if (K == 0) {
        r.drop_all = true;
    } else if (K == r.p - 1) {
        r.mask = ~0ull; r.thr = my_max - 1ull;
    } else {
        unsigned long long mask = 0ull, thr = 0ull;
        int k_rem = K;
        for (int shift = 56; shift >= 0; shift -= 8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) hist[lane * 8 + i] = 0;
            __syncwarp();
            for (int slot = lane; slot < n; slot += 32) {
                unsigned long long key = sm_keys[slot];
                if ((region[slot] & 3) == kRegionPrevious && (key & mask) == thr)
                    atomicAdd(&hist[(int)((key >> shift) & 255ull)], 1);
            }
            __syncwarp();
            int h[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { h[i] = hist[lane * 8 + i]; tot += h[i]; }
            int incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            int excl = incl - tot;
            int digit = 0, krem = 0, bin = 0;
            const bool mine = excl < k_rem && k_rem <= incl;   // exactly one lane holds the bin of the k_rem-th key
            if (mine) {
                int cum = excl;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (cum < k_rem && k_rem <= cum + h[i]) { digit = lane * 8 + i; krem = k_rem - cum; bin = h[i]; }
                    cum += h[i];
                }
            }
            const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
            digit = __shfl_sync(0xffffffffu, digit, src);
            krem = __shfl_sync(0xffffffffu, krem, src);
            bin = __shfl_sync(0xffffffffu, bin, src);
            thr |= (unsigned long long)digit << shift;
            mask |= 255ull << shift;
            k_rem = krem;
            __syncwarp();
            if (k_rem == bin) break;
        }
        r.mask = mask; r.thr = thr;
    }
    return r;
}

}  // namespace adsa
