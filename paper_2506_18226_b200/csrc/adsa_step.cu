// The staged stream kernel: one thread-block cluster per stream, the stream's
// K and V rows brought into shared memory once by bulk asynchronous copies and
// used there by everything that needs them.
//
//   step_kernel<LPR, false>   adsa_sparse_decode_attn: Eq. 4 + the attention of Fig. 3
//                             over the rows adsa_select retained (keep mask in the workspace).
//   step_kernel<LPR, true>    the whole layer-step in one pass over the cache:
//                             Eq. 3 selection from the scores carried in from the previous
//                             step, attention, the Eq. 1-2 scores of the NEXT step (every row
//                             the next step can score is among the rows read now), and the
//                             Section 4.2 update.  K and V cross HBM once per step.
//
// Work split.  A stream's live rows [0, n) are cut into gridDim.x equal chunks,
// one per CTA of the cluster (blockIdx.x = rank).  Each CTA issues, right at its
// start, bulk copies (cp.async.bulk, mbarrier completion) of its whole chunk,
// page piece by page piece, in groups of group_rows rows with one mbarrier per
// group; nearly every cached row is retained (one eviction per step), so the
// copies do not wait for the selection, which runs while they are in flight.
// Warps then sweep the groups as they land: LPR lanes share a row, 16 bytes
// each, online softmax per lane group.  Partial states are merged through warp
// shuffles, shared memory, and across the cluster through distributed shared
// memory in rank order, so results do not depend on scheduling.
//
// Every wait on a copy is bounded: if it runs out the block raises
// ADSA_DEV_COPY_TIMEOUT, carries on to the end of the kernel (all accesses stay
// in bounds) and waits once more, bounded, before it leaves.
#include <cooperative_groups.h>
#include <float.h>
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"
#include "adsa_select.cuh"
#include "adsa_async.cuh"

namespace cg = cooperative_groups;

namespace adsa {

constexpr int kStepThreads = kSelThreads;
constexpr int kStepWarps = kStepThreads / 32;
constexpr int kStepUnroll = 2;

// ---- shared-memory layout (same function on host and device) ---------------
struct StepLayout {
    uint32_t bars, xchg, wred, svec, mask, inv, keys, region, kbuf, vbuf, total;
};

__host__ __device__ inline uint32_t step_align(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline StepLayout step_layout(int max_rows, int mask_words, int chunk_rows, int row_stride, bool fused)
{
    StepLayout L;
    uint32_t off = 0;
    L.bars = off;   off += kStepMaxGroups * 8;
    L.xchg = off;   off += (2 * row_stride + 4) * 4;                     // acc[stride] | s_next[stride] | m, l
    L.wred = off;   off += kStepWarps * (2 * row_stride + 2) * 4;        // per warp: acc | s_next | m, l
    L.svec = off;   off += row_stride * 4;
    L.mask = off;   off += step_align(mask_words * 4, 16);
    L.inv = off;    off += fused ? step_align(chunk_rows * 4, 16) : 0;
    L.keys = off;   off += fused ? step_align((max_rows + 2) * 8, 16) : 0;   // later reused: holes[max_rows+1], survivors[max_rows]
    L.region = off; off += fused ? step_align(max_rows, 16) : 0;
    off = step_align(off, 128);
    L.kbuf = off;   off += chunk_rows * row_stride * 2;
    off = step_align(off, 128);
    L.vbuf = off;   off += chunk_rows * row_stride * 2;
    L.total = off;
    return L;
}

struct StepArgs {
    int layer, cur_pos, budget_rows;
    int chunk_rows;   // rows per CTA of the cluster (multiple of 8)
    int group_rows;   // rows per copy group / mbarrier
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out_bf16;
    float *out_f32;
};

template <int LPR, bool FUSED>
__global__ void __launch_bounds__(kStepThreads)
step_kernel(DevCtx c, StepArgs a)
{
    constexpr int RPW = 32 / LPR;             // rows a warp covers per load
    constexpr int STEP = kStepWarps * RPW;    // rows the block covers per load
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ SelScratch s_sel;
    __shared__ int s_wcnt[2][kStepWarps], s_nholes, s_nsurv, s_pnext, s_ok, s_timeout;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = blockIdx.x, CS = gridDim.x;
    const int local = blockIdx.y, sid = a.layer * c.S + local;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < c.row_stride;
    const StepLayout L = step_layout(c.max_rows, c.mask_words, a.chunk_rows, c.row_stride, FUSED);
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + L.bars);
    float *xchg = reinterpret_cast<float *>(smem + L.xchg);
    float *wred = reinterpret_cast<float *>(smem + L.wred);
    float *svec = reinterpret_cast<float *>(smem + L.svec);
    uint32_t *kmask = reinterpret_cast<uint32_t *>(smem + L.mask);
    float *inv_s = reinterpret_cast<float *>(smem + L.inv);
    unsigned long long *sm_keys = reinterpret_cast<unsigned long long *>(smem + L.keys);
    uint8_t *region = smem + L.region;
    const __nv_bfloat16 *kbuf = reinterpret_cast<const __nv_bfloat16 *>(smem + L.kbuf);
    const __nv_bfloat16 *vbuf = reinterpret_cast<const __nv_bfloat16 *>(smem + L.vbuf);

    int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    int32_t *pos = c.pos + (size_t)sid * c.max_rows;
    float *inv_norm = c.inv_norm + (size_t)sid * c.max_rows;
    float *scores = c.scores + (size_t)sid * c.max_rows;
    const int n = c.n_live[sid];
    // the same decision in every CTA of the cluster, taken before any barrier exists
    if (n < 0 || n > c.max_rows || n > CS * a.chunk_rows) {
        if (tid == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW);
        return;
    }
    const int c0 = min(n, rank * a.chunk_rows), c1 = min(n, c0 + a.chunk_rows);
    const int n_groups = (c1 - c0 + a.group_rows - 1) / a.group_rows;
    const int row_bytes = c.row_stride * 2;

    if (tid == 0) {
        for (int g = 0; g < n_groups; ++g) mbar_init(smem_u32(bars + g), 1);
        mbar_init_fence();
        s_timeout = 0;
    }
    __syncthreads();

    // ---- copies of the whole chunk, one lane per group ----------------------------------------
    if (warp == 0) {
        for (int g = lane; g < n_groups; g += 32) {
            const int r0 = c0 + g * a.group_rows, r1 = min(c1, r0 + a.group_rows);
            const uint32_t bar = smem_u32(bars + g);
            mbar_expect_tx(bar, (uint32_t)(r1 - r0) * row_bytes * 2u);
            int r = r0;
            while (r < r1) {
                uint32_t pg = __umulhi((uint32_t)r, c.pr_magic);
                int in = r - (int)pg * c.page_rows;
                int cnt = min(r1 - r, c.page_rows - in);
                size_t src = ((size_t)pt[pg] * c.page_rows + in) * (size_t)c.row_stride;
                uint32_t dst = (uint32_t)(r - c0) * row_bytes, bytes = (uint32_t)cnt * row_bytes;
                bulk_g2s(smem_u32(smem + L.kbuf) + dst, c.k_pool + src, bytes, bar);
                bulk_g2s(smem_u32(smem + L.vbuf) + dst, c.v_pool + src, bytes, bar);
                r += cnt;
            }
        }
    }

    // ---- which rows are attended ---------------------------------------------------------------
    int n2 = n, p_next = 0;
    // With a window of the current grid row only, the new row itself is a candidate of the next step
    // when that step starts a new grid row.
    const bool new_cand = FUSED && region_of(c, a.cur_pos, a.cur_pos + 1) == kRegionPrevious;
    if constexpr (FUSED) {
        for (int r = c0 + tid; r < c1; r += kStepThreads) inv_s[r - c0] = inv_norm[r];
        const SelResult sel = block_select(c, pos, scores, n, a.cur_pos, a.budget_rows, sm_keys, region, s_sel);
        n2 = n - (sel.p - sel.K) + 1;
        if (tid == 0) { s_pnext = 0; s_nholes = 0; s_nsurv = 0; }
        __syncthreads();
        // keep mask of the whole stream (every CTA of the cluster builds the same one)
        int my_pn = 0;
        for (int base = 0; base < n; base += kStepThreads) {
            int slot = base + tid;
            bool kept = slot < n && sel.keeps(region[slot], sm_keys[slot]);
            if (slot < n && (region[slot] & 3) == kRegionInvalid && rank == 0) set_status(c, ADSA_DEV_BAD_POSITION);
            unsigned bk = __ballot_sync(0xffffffffu, kept);
            if (lane == 0 && base + warp * 32 < n) kmask[(base >> 5) + warp] = bk;
            if (kept && (region[slot] & kCandNextBit)) ++my_pn;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) my_pn += __shfl_xor_sync(0xffffffffu, my_pn, o);
        if (lane == 0 && my_pn) atomicAdd(&s_pnext, my_pn);
        __syncthreads();
        p_next = s_pnext + (new_cand ? 1 : 0);
    } else {
        const uint32_t *gmask = c.keep_mask + (size_t)sid * c.mask_words;
        for (int w = tid; w * 32 < n; w += kStepThreads) kmask[w] = gmask[w];
        __syncthreads();
    }

    // ---- sweep ---------------------------------------------------------------------------------
    float qf[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int x = sub * 8 + e;
        qf[e] = x < c.d ? __bfloat162float(a.q[(size_t)local * c.d + x]) * c.scale_log2e : 0.f;
    }
    float m = -FLT_MAX, l = 0.f, acc[8], sn[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { acc[e] = 0.f; sn[e] = 0.f; }

    if (rank == 0 && warp == 0) {   // the new row, always attended
        float s = 0.f, vf[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int x = sub * 8 + e;
            float kf = x < c.d ? __bfloat162float(a.k_new[(size_t)local * c.d + x]) : 0.f;
            vf[e] = x < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + x]) : 0.f;
            s = fmaf(qf[e], kf, s);
        }
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        float inv_new = 0.f;
        if (new_cand) {
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(vf[e], vf[e], ss);
#pragma unroll
            for (int o = 1; o < LPR; o <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
            inv_new = 1.0f / fmaxf(sqrtf(ss), kNormEps);
        }
        if (grp == 0) {
            m = s; l = 1.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) { acc[e] = vf[e]; sn[e] = inv_new * vf[e]; }
        }
    }

    int spin_limit = kCopySpinLimit;
    for (int g = 0; g < n_groups; ++g) {
        if (!mbar_wait_bounded(smem_u32(bars + g), 0, spin_limit)) {
            if (lane == 0) { set_status(c, ADSA_DEV_COPY_TIMEOUT); s_timeout = 1; }
            spin_limit = kCopySpinAfterTimeout;
        }
        const int r0 = c0 + g * a.group_rows, r1 = min(c1, r0 + a.group_rows);
        // loop bounds are warp-uniform: every lane takes part in the shuffles of every iteration
        for (int it0 = r0 + warp * RPW; it0 < r1; it0 += STEP * kStepUnroll) {
            uint4 kr[kStepUnroll], vr[kStepUnroll];
            bool ok[kStepUnroll];
            float wn[kStepUnroll];
#pragma unroll
            for (int u = 0; u < kStepUnroll; ++u) {
                int row = it0 + u * STEP + grp;
                ok[u] = row < r1 && ((kmask[row >> 5] >> (row & 31)) & 1u);
                kr[u] = make_uint4(0u, 0u, 0u, 0u);
                vr[u] = make_uint4(0u, 0u, 0u, 0u);
                wn[u] = 0.f;
                if (ok[u] && piece_ok) {
                    size_t off = (size_t)(row - c0) * c.row_stride + sub * 8;
                    kr[u] = lds128(kbuf + off);
                    vr[u] = lds128(vbuf + off);
                }
                if constexpr (FUSED) {
                    if (ok[u] && (region[row] & kCandNextBit)) wn[u] = inv_s[row - c0];
                }
            }
            float s[kStepUnroll], m_new = m;
#pragma unroll
            for (int u = 0; u < kStepUnroll; ++u) {
                float kf[8];
                unpack8(kr[u], kf);
                float t = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) t = fmaf(qf[e], kf[e], t);
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                s[u] = ok[u] ? t : -INFINITY;
                m_new = fmaxf(m_new, s[u]);
            }
            float corr = exp2f(m - m_new);
            l *= corr;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= corr;
#pragma unroll
            for (int u = 0; u < kStepUnroll; ++u) {
                float pw = exp2f(s[u] - m_new), vf[8];
                unpack8(vr[u], vf);
                l += pw;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(pw, vf[e], acc[e]);
                if constexpr (FUSED) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) sn[e] = fmaf(wn[u], vf[e], sn[e]);
                }
            }
            m = m_new;
        }
    }

    // ---- lane groups -> warp -> block ----------------------------------------------------------
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o), a2[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a2[e] = __shfl_xor_sync(0xffffffffu, acc[e], o);
        merge2(m, l, acc, m2, l2, a2);
        if constexpr (FUSED) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sn[e] += __shfl_xor_sync(0xffffffffu, sn[e], o);
        }
    }
    const int wstride = 2 * c.row_stride + 2;
    if (grp == 0) {
        float *w = wred + warp * wstride;
        if (piece_ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e) { w[sub * 8 + e] = acc[e]; w[c.row_stride + sub * 8 + e] = sn[e]; }
        }
        if (sub == 0) { w[2 * c.row_stride] = m; w[2 * c.row_stride + 1] = l; }
    }
    __syncthreads();
    if (tid < c.row_stride) {
        float M = -FLT_MAX, Lb = 0.f, A = 0.f, SN = 0.f;
#pragma unroll
        for (int w = 0; w < kStepWarps; ++w) M = fmaxf(M, wred[w * wstride + 2 * c.row_stride]);
#pragma unroll
        for (int w = 0; w < kStepWarps; ++w) {
            const float *ws = wred + w * wstride;
            float wgt = exp2f(ws[2 * c.row_stride] - M);
            Lb = fmaf(ws[2 * c.row_stride + 1], wgt, Lb);
            A = fmaf(ws[tid], wgt, A);
            SN += ws[c.row_stride + tid];
        }
        xchg[tid] = A;
        xchg[c.row_stride + tid] = SN;
        if (tid == 0) { xchg[2 * c.row_stride] = M; xchg[2 * c.row_stride + 1] = Lb; }
    }

    // ---- across the cluster, in rank order -----------------------------------------------------
    cluster.sync();
    if (tid < c.row_stride) {
        float SN = 0.f;
        if (rank == 0) {
            float M = -FLT_MAX;
            for (int r = 0; r < CS; ++r) M = fmaxf(M, cluster.map_shared_rank(xchg, r)[2 * c.row_stride]);
            float Lx = 0.f, Ax = 0.f;
            for (int r = 0; r < CS; ++r) {
                const float *xr = cluster.map_shared_rank(xchg, r);
                float wgt = exp2f(xr[2 * c.row_stride] - M);
                Lx = fmaf(xr[2 * c.row_stride + 1], wgt, Lx);
                Ax = fmaf(xr[tid], wgt, Ax);
                SN += xr[c.row_stride + tid];
            }
            if (tid < c.d) {
                float o = Ax / Lx;
                if (a.out_f32) a.out_f32[(size_t)local * c.d + tid] = o;
                if (a.out_bf16) a.out_bf16[(size_t)local * c.d + tid] = __float2bfloat16_rn(o);
            }
        } else if (FUSED) {
            for (int r = 0; r < CS; ++r) SN += cluster.map_shared_rank(xchg, r)[c.row_stride + tid];
        }
        svec[tid] = SN;
    }
    cluster.barrier_arrive();   // nobody reads this CTA's exchange buffer after the matching wait
    __syncthreads();

    if constexpr (FUSED) {
        // ---- Eq. 1-2 for the next step: S_i = (u_i . s - u_i . u_i) / (p' - 1), u = v * inv_norm ----
        // ---- and the Section 4.2 update: hole / survivor pairing as in kv_update_kernel ------------
        int32_t *holes = reinterpret_cast<int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;   // keys are dead now
        const int top = max(n, n2);
        for (int base = 0; base < top; base += kStepThreads) {
            int s = base + tid;
            bool kept = s < n && ((kmask[s >> 5] >> (s & 31)) & 1u);
            bool is_hole = s < n2 && !kept, is_surv = s >= n2 && s < n && kept;
            unsigned bh = __ballot_sync(0xffffffffu, is_hole), bs = __ballot_sync(0xffffffffu, is_surv);
            if (lane == 0) { s_wcnt[0][warp] = __popc(bh); s_wcnt[1][warp] = __popc(bs); }
            __syncthreads();
            int oh = s_nholes, os = s_nsurv;
            for (int w = 0; w < warp; ++w) { oh += s_wcnt[0][w]; os += s_wcnt[1][w]; }
            unsigned below = (1u << lane) - 1u;
            if (is_hole) holes[oh + __popc(bh & below)] = s;
            if (is_surv) surv[os + __popc(bs & below)] = s;
            __syncthreads();
            if (tid == 0) {
                for (int w = 0; w < kStepWarps; ++w) { s_nholes += s_wcnt[0][w]; s_nsurv += s_wcnt[1][w]; }
            }
            __syncthreads();
        }
        const int nh = s_nholes, ns = s_nsurv;
        const int have = (n + c.page_rows - 1) / c.page_rows, need = (n2 + c.page_rows - 1) / c.page_rows;
        if (tid == 0) {
            s_ok = 1;
            if (nh != ns + 1) { set_status(c, ADSA_DEV_BAD_EVICT); s_ok = 0; }
            else if (n2 > c.max_rows) { set_status(c, ADSA_DEV_ROW_OVERFLOW); s_ok = 0; }
            else if (rank == 0 && need > have && !resize_pages(c, pt, have, need)) s_ok = 0;
        }
        __syncthreads();
        if (s_ok) {
            float sv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) sv[e] = piece_ok ? svec[sub * 8 + e] : 0.f;
            const float denom = (float)(p_next - 1);
            // rows that stay where they are (warp-uniform bounds: all lanes join the shuffles)
            const int stay_end = min(c1, n2);
            for (int rb = c0 + warp * RPW; rb < stay_end; rb += STEP) {
                const int row = rb + grp;
                bool want = row < stay_end && ((kmask[row >> 5] >> (row & 31)) & 1u) && (region[row] & kCandNextBit);
                float dot = 0.f, self = 0.f;
                if (want && piece_ok) {
                    float f[8];
                    unpack8(lds128(vbuf + (size_t)(row - c0) * c.row_stride + sub * 8), f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], sv[e], dot); self = fmaf(f[e], f[e], self); }
                }
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) {
                    dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    self += __shfl_xor_sync(0xffffffffu, self, o);
                }
                if (want && sub == 0) {
                    float inv = inv_s[row - c0];
                    scores[row] = p_next > 1 ? (inv * dot - inv * inv * self) / denom + 0.0f : 0.0f;
                }
            }
            // survivors above the new length move into the holes below it, payload from shared memory
            for (int ib = warp * RPW; ib < ns; ib += STEP) {
                const int i = ib + grp;
                const int row = i < ns ? surv[i] : -1, dst = i < ns ? holes[i] : 0;
                const bool mine = row >= c0 && row < c1;
                const bool want = mine && (region[row] & kCandNextBit);
                float dot = 0.f, self = 0.f;
                if (mine && piece_ok) {
                    size_t so = (size_t)(row - c0) * c.row_stride + sub * 8;
                    uint4 kq = lds128(kbuf + so), vq = lds128(vbuf + so);
                    size_t go = row_offset(c, pt, dst) + sub * 8;
                    *reinterpret_cast<uint4 *>(c.k_pool + go) = kq;
                    *reinterpret_cast<uint4 *>(c.v_pool + go) = vq;
                    float f[8];
                    unpack8(vq, f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], sv[e], dot); self = fmaf(f[e], f[e], self); }
                }
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) {
                    dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    self += __shfl_xor_sync(0xffffffffu, self, o);
                }
                if (mine && sub == 0) {
                    float inv = inv_s[row - c0];
                    pos[dst] = pos[row];
                    inv_norm[dst] = inv;
                    if (want) scores[dst] = p_next > 1 ? (inv * dot - inv * inv * self) / denom + 0.0f : 0.0f;
                }
            }
            if (rank == 0) {
                if (warp == 0 && new_cand) {   // the new row's own score for the next step
                    float vf[8], dot = 0.f, ss = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        int x = sub * 8 + e;
                        vf[e] = x < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + x]) : 0.f;
                        dot = fmaf(vf[e], sv[e], dot);
                        ss = fmaf(vf[e], vf[e], ss);
                    }
#pragma unroll
                    for (int o = 1; o < LPR; o <<= 1) {
                        dot += __shfl_xor_sync(0xffffffffu, dot, o);
                        ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    }
                    float inv = 1.0f / fmaxf(sqrtf(ss), kNormEps);
                    if (lane == 0) scores[holes[ns]] = p_next > 1 ? (inv * dot - inv * inv * ss) / denom + 0.0f : 0.0f;
                }
                if (warp == 0)
                    write_row(c, pt, sid, holes[ns], a.k_new + (size_t)local * c.d, a.v_new + (size_t)local * c.d, a.cur_pos);
                if (tid == 32) {
                    if (need < have) resize_pages(c, pt, have, need);
                    c.n_live[sid] = n2;
                }
            }
        }
    }

    if (s_timeout) {   // a copy may still be in flight into this CTA's shared memory: give it one more bounded wait
        for (int g = 0; g < n_groups; ++g) mbar_wait_bounded(smem_u32(bars + g), 0, kCopySpinLimit >> 4);
    }
    cluster.barrier_wait();
}

// ---- host side ------------------------------------------------------------
namespace {

template <int LPR, bool FUSED>
cudaError_t launch_one(const DevCtx &c, const StepArgs &a, int cluster_size, size_t smem, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster_size, c.S, 1);
    cfg.blockDim = dim3(kStepThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, step_kernel<LPR, FUSED>, c, a);
}

template <int LPR>
cudaError_t configure_lpr()
{
    cudaError_t e = cudaFuncSetAttribute(step_kernel<LPR, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kStepSmemLimit);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(step_kernel<LPR, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kStepSmemLimit);
}

int step_lanes(int row_stride)
{
    int pieces = row_stride / 8;
    return pieces <= 4 ? 4 : pieces <= 8 ? 8 : pieces <= 16 ? 16 : 32;
}

}  // namespace

cudaError_t configure_step_kernel(const DevCtx &c)
{
    switch (step_lanes(c.row_stride)) {
    case 4: return configure_lpr<4>();
    case 8: return configure_lpr<8>();
    case 16: return configure_lpr<16>();
    default: return configure_lpr<32>();
    }
}

// Cluster size and chunk for streams of up to n_rows rows; cluster_size 0 when no cluster of at
// most 8 CTAs can hold such a stream in shared memory.
StepPlan plan_step(const DevCtx &c, int n_rows, bool fused, int sm_count, int chunk_target)
{
    StepPlan p = {};
    const int lanes = step_lanes(c.row_stride), step = kStepWarps * (32 / lanes);
    int rows = n_rows < 1 ? 1 : n_rows;
    const bool automatic = chunk_target <= 0;
    if (automatic) {
        chunk_target = (40 * 1024) / (c.row_stride * 4);           // about 40 KB of K+V per CTA
        if (chunk_target < step * kStepUnroll) chunk_target = step * kStepUnroll;
    }
    int cs = 1;
    while (cs < 8 && (rows + cs - 1) / cs > chunk_target) cs *= 2;
    while (automatic && cs < 8 && (long long)c.S * cs < 2ll * sm_count && (rows + cs - 1) / cs > step * kStepUnroll) cs *= 2;
    for (;; cs *= 2) {
        int chunk = ((rows + cs - 1) / cs + 7) / 8 * 8;
        int unit = step * kStepUnroll;
        int group = ((chunk + kStepMaxGroups - 1) / kStepMaxGroups + unit - 1) / unit * unit;
        StepLayout L = step_layout(c.max_rows, c.mask_words, chunk, c.row_stride, fused);
        if (L.total + 4096 <= (uint32_t)kStepSmemLimit && (size_t)group * c.row_stride * 4 < (1u << 20)) {
            p.cluster_size = cs; p.chunk_rows = chunk; p.group_rows = group; p.smem_bytes = L.total;
            return p;
        }
        if (cs >= 8) break;
    }
    return p;
}

cudaError_t launch_step(const DevCtx &c, const StepPlan &plan, bool fused, int layer, int cur_pos, int budget_rows,
                        const void *q, const void *k_new, const void *v_new, void *out_bf16, float *out_f32,
                        cudaStream_t st)
{
    StepArgs a;
    a.layer = layer; a.cur_pos = cur_pos; a.budget_rows = budget_rows;
    a.chunk_rows = plan.chunk_rows; a.group_rows = plan.group_rows;
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    const int cs = plan.cluster_size;
    const size_t sm = plan.smem_bytes;
#define ADSA_STEP_CASE(LPR)                                                              \
    return fused ? launch_one<LPR, true>(c, a, cs, sm, st) : launch_one<LPR, false>(c, a, cs, sm, st)
    switch (step_lanes(c.row_stride)) {
    case 4: ADSA_STEP_CASE(4);
    case 8: ADSA_STEP_CASE(8);
    case 16: ADSA_STEP_CASE(16);
    default: ADSA_STEP_CASE(32);
    }
#undef ADSA_STEP_CASE
}

}  // namespace adsa
