// The persistent, pipelined stream kernel.  One CTA per SM stays resident and
// walks over the streams of a layer (stream = blockIdx.x, += gridDim.x).  A
// producer warp keeps a ring of shared-memory stages full with tiles of K and
// V rows (cp.async.bulk + mbarrier), running ahead of the eight consumer warps
// across stream boundaries, so HBM requests stay in flight the whole time the
// kernel runs, whatever the consumers are doing at the moment.
//
//   pstep_kernel<LPR, false>  adsa_sparse_decode_attn (keep mask from adsa_select).
//   pstep_kernel<LPR, true>   the whole layer-step: Eq. 3 selection from the scores
//       carried in from the previous step, attention (Eq. 4, Fig. 3), the Eq. 1-2
//       scores of the NEXT step, and the Section 4.2 update.
//
// Per stream the producer sends: the per-row metadata (positions, carried
// scores, inverse norms; or the keep mask) into one of two metadata buffers;
// pass 1, tiles of K and V rows in slot order; and (fused) pass 2, the V tiles
// once more.  Pass 2 computes S_i = (u_i.s - u_i.u_i)/(p-1) for the rows the next
// step can score, which needs s = sum of the normalised retained rows, complete
// only after pass 1; its tiles come out of L2 (the stream's V was read a few
// microseconds earlier), so K and V still cross HBM once per step.
// All rows of a stream are copied, retained or not (one row per step is not).
//
// Every wait is bounded.  A wait that runs out raises ADSA_DEV_COPY_TIMEOUT,
// shortens all later waits of the CTA and lets the kernel run to its end (all
// accesses stay in bounds); before leaving, the producer waits, bounded, for
// the copies it still has in flight.
#include <float.h>
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"
#include "adsa_select.cuh"
#include "adsa_async.cuh"

namespace adsa {

constexpr int kPConsumers = kSelThreads;          // 256 consumer threads (8 warps) ...
constexpr int kPWarps = kPConsumers / 32;
constexpr int kPThreads = kPConsumers + 32;       // ... and one producer warp
constexpr int kPUnroll = 2;                       // a tile is kPUnroll block-wide row groups

struct PLayout {
    uint32_t bars, hdr, meta[2], pt[2], keys, region, kmask, wred, svec, stages;
    uint32_t meta_words;     // words per metadata array (room for the alignment lead)
    uint32_t tile_bytes;     // one K (or V) tile
    uint32_t total;
};

__host__ __device__ inline uint32_t p_align(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline PLayout p_layout(int max_rows, int max_pages, int mask_words, int row_stride, int tile_rows,
                                            int n_stages, bool fused)
{
    PLayout L;
    uint32_t off = 0;
    L.bars = off;   off += (2 * kPMaxStages + 4) * 8;
    L.hdr = off;    off += 2 * 16;                                       // per metadata buffer: n
    L.meta_words = p_align(max_rows + 8, 4);
    const uint32_t meta_bytes = fused ? 3 * L.meta_words * 4 : p_align(mask_words * 4, 16);
    L.meta[0] = off; off += meta_bytes;
    L.meta[1] = off; off += meta_bytes;
    L.pt[0] = off;  off += p_align(max_pages * 4, 16);
    L.pt[1] = off;  off += p_align(max_pages * 4, 16);
    L.keys = off;   off += fused ? p_align((max_rows + 2) * 8, 16) : 0;  // later reused: holes, survivors
    L.region = off; off += fused ? p_align(max_rows, 16) : 0;
    L.kmask = off;  off += p_align(mask_words * 4, 16);
    L.wred = off;   off += kPWarps * (2 * row_stride + 2) * 4;
    L.svec = off;   off += row_stride * 4;
    off = p_align(off, 128);
    L.tile_bytes = tile_rows * row_stride * 2;
    L.stages = off; off += n_stages * 2 * L.tile_bytes;
    L.total = off;
    return L;
}

struct PStepArgs {
    int layer, cur_pos, budget_rows, n_stages;
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out_bf16;
    float *out_f32;
};

// CTA-wide state of the bounded waits
struct PWaitState {
    int limit;
};

template <int LPR, bool FUSED>
__global__ void __launch_bounds__(kPThreads, 1)
pstep_kernel(DevCtx c, PStepArgs a)
{
    constexpr int RPW = 32 / LPR;
    constexpr int STEP = kPWarps * RPW;           // rows the consumers cover per load
    constexpr int TILE = STEP * kPUnroll;         // rows per tile
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ SelScratch s_sel;
    __shared__ int s_wcnt[2][kPWarps], s_nholes, s_nsurv, s_pnext, s_ok;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NST = a.n_stages;
    const PLayout L = p_layout(c.max_rows, c.max_pages, c.mask_words, c.row_stride, TILE, NST, FUSED);
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + L.bars);
    // barrier indices: full[s] = s, empty[s] = kPMaxStages + s, meta_full[b] = 2*kPMaxStages + b, meta_empty[b] = +2 + b
    auto bar_full = [&](int s) { return smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return smem_u32(bars + kPMaxStages + s); };
    auto bar_mfull = [&](int b) { return smem_u32(bars + 2 * kPMaxStages + b); };
    auto bar_mempty = [&](int b) { return smem_u32(bars + 2 * kPMaxStages + 2 + b); };
    const int row_bytes = c.row_stride * 2;

    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), kPWarps); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_mfull(b), 1); mbar_init(bar_mempty(b), 1); }
        mbar_init_fence();
        s_abort = 0;
    }
    __syncthreads();

    auto wait = [&](uint32_t bar, uint32_t parity) {   // bounded; after the first failure every wait is short
        int limit = s_abort ? kCopySpinAfterTimeout : kCopySpinLimit;
        if (!mbar_wait_sleepy(bar, parity, limit)) {
            if (lane == 0) set_status(c, ADSA_DEV_COPY_TIMEOUT);
            s_abort = 1;
        }
    };

    if (warp == kPWarps) {
        // =============================== producer warp ===============================
        uint32_t it = 0;   // tiles issued so far by this CTA
        int j = 0;
        for (int local = blockIdx.x; local < c.S; local += gridDim.x, ++j) {
            const int sid = a.layer * c.S + local, mb = j & 1;
            const int32_t *pt_g = c.page_table + (size_t)sid * c.max_pages;
            int32_t *pt_s = reinterpret_cast<int32_t *>(smem + L.pt[mb]);
            wait(bar_mempty(mb), ((j >> 1) & 1) ^ 1);   // the consumers are done with this buffer's previous stream
            int n = c.n_live[sid];
            if (n < 0 || n > c.max_rows) { if (lane == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW); n = 0; }
            const int np = (n + c.page_rows - 1) / c.page_rows;
            for (int pg = lane; pg < np; pg += 32) pt_s[pg] = pt_g[pg];
            // ---- metadata of the stream ----
            unsigned char *meta = smem + L.meta[mb];
            uint32_t meta_tx = 0;
            if constexpr (FUSED) {
                const void *src[3] = {c.pos + (size_t)sid * c.max_rows, c.scores + (size_t)sid * c.max_rows,
                                      c.inv_norm + (size_t)sid * c.max_rows};
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    // word i of the array lands at word (lead + i) of its buffer, so that the 16-byte aligned
                    // interior can go by bulk copy; the ragged ends (< 4 words each) go by plain loads
                    const uint32_t *g = reinterpret_cast<const uint32_t *>(src[k]);
                    uint32_t *d = reinterpret_cast<uint32_t *>(meta) + k * L.meta_words;
                    const int lead = (int)(((uintptr_t)g >> 2) & 3);
                    const int head = min(n, (4 - lead) & 3);
                    const int body = (n - head) & ~3;
                    if (lane < head) d[lead + lane] = g[lane];
                    if (lane < n - head - body) d[lead + head + body + lane] = g[head + body + lane];
                    if (lane == 0 && body > 0) {
                        bulk_g2s(smem_u32(d + lead + head), g + head, (uint32_t)body * 4u, bar_mfull(mb));
                        meta_tx += (uint32_t)body * 4u;
                    }
                }
            } else {
                const uint32_t *g = c.keep_mask + (size_t)sid * c.mask_words;
                uint32_t *d = reinterpret_cast<uint32_t *>(meta);
                for (int w = lane; w * 32 < n; w += 32) d[w] = g[w];
            }
            if (lane == 0) reinterpret_cast<int *>(smem + L.hdr)[mb * 4] = n;
            __syncwarp();
            if (lane == 0) mbar_expect_tx(bar_mfull(mb), meta_tx);   // release: the plain stores above are visible to the waiters
            // ---- tiles ----
            if (lane == 0) {
                const int n_tiles = (n + TILE - 1) / TILE;
                for (int pass = 0; pass < (FUSED ? 2 : 1); ++pass) {
                    for (int t = 0; t < n_tiles; ++t, ++it) {
                        const int stage = it % NST;
                        wait(bar_empty(stage), ((it / NST) & 1) ^ 1);
                        const int r0 = t * TILE, r1 = min(n, r0 + TILE);
                        const uint32_t kdst = smem_u32(smem + L.stages) + stage * 2 * L.tile_bytes;
                        const uint32_t vdst = kdst + L.tile_bytes, bar = bar_full(stage);
                        mbar_expect_tx(bar, (uint32_t)(r1 - r0) * row_bytes * (pass == 0 ? 2u : 1u));
                        int r = r0;
                        while (r < r1) {
                            uint32_t pg = __umulhi((uint32_t)r, c.pr_magic);
                            int in = r - (int)pg * c.page_rows;
                            int cnt = min(r1 - r, c.page_rows - in);
                            size_t src = ((size_t)pt_s[pg] * c.page_rows + in) * (size_t)c.row_stride;
                            uint32_t dst = (uint32_t)(r - r0) * row_bytes, bytes = (uint32_t)cnt * row_bytes;
                            if (pass == 0) bulk_g2s(kdst + dst, c.k_pool + src, bytes, bar);
                            bulk_g2s(vdst + dst, c.v_pool + src, bytes, bar);
                            r += cnt;
                        }
                    }
                }
            }
            __syncwarp();
        }
        // nothing of this CTA's may still be in flight when it leaves: the last round of every stage has landed
        if (lane == 0) {
            for (uint32_t back = 0; back < (uint32_t)NST && back < it; ++back) {
                uint32_t i = it - 1 - back;
                mbar_wait_sleepy(bar_full(i % NST), (i / NST) & 1, s_abort ? kCopySpinAfterTimeout : kCopySpinLimit);
            }
        }
        return;
    }

    // ================================= consumer warps =================================
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < c.row_stride;
    unsigned long long *sm_keys = reinterpret_cast<unsigned long long *>(smem + L.keys);
    uint8_t *region = smem + L.region;
    uint32_t *kmask = reinterpret_cast<uint32_t *>(smem + L.kmask);
    float *wred = reinterpret_cast<float *>(smem + L.wred);
    float *svec = reinterpret_cast<float *>(smem + L.svec);
    const int wstride = 2 * c.row_stride + 2;
    const bool new_cand = FUSED && region_of(c, a.cur_pos, a.cur_pos + 1) == kRegionPrevious;

    uint32_t it = 0;
    int j = 0;
    for (int local = blockIdx.x; local < c.S; local += gridDim.x, ++j) {
        const int sid = a.layer * c.S + local, mb = j & 1;
        int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
        wait(bar_mfull(mb), (j >> 1) & 1);
        const int n = reinterpret_cast<const int *>(smem + L.hdr)[mb * 4];
        const int n_tiles = (n + TILE - 1) / TILE;
        const unsigned char *meta = smem + L.meta[mb];
        const int32_t *pos_s = nullptr;
        const float *inv_s = nullptr;
        int n2 = n, p_next = 0;

        // ---- which rows are attended ---------------------------------------------------------
        if constexpr (FUSED) {
            const int lead = (int)((((uintptr_t)(c.pos + (size_t)sid * c.max_rows)) >> 2) & 3);
            const int lead_sc = (int)((((uintptr_t)(c.scores + (size_t)sid * c.max_rows)) >> 2) & 3);
            const int lead_in = (int)((((uintptr_t)(c.inv_norm + (size_t)sid * c.max_rows)) >> 2) & 3);
            pos_s = reinterpret_cast<const int32_t *>(meta) + lead;
            const float *scores_s = reinterpret_cast<const float *>(meta) + L.meta_words + lead_sc;
            inv_s = reinterpret_cast<const float *>(meta) + 2 * L.meta_words + lead_in;
            const SelResult sel = block_select<ConsumerSync>(c, pos_s, scores_s, n, a.cur_pos, a.budget_rows, sm_keys,
                                                             region, s_sel);
            n2 = n - (sel.p - sel.K) + 1;
            if (tid == 0) { s_pnext = 0; s_nholes = 0; s_nsurv = 0; }
            ConsumerSync::sync();
            int my_pn = 0;
            for (int base = 0; base < n; base += kPConsumers) {
                int slot = base + tid;
                bool kept = slot < n && sel.keeps(region[slot], sm_keys[slot]);
                if (slot < n && (region[slot] & 3) == kRegionInvalid) set_status(c, ADSA_DEV_BAD_POSITION);
                unsigned bk = __ballot_sync(0xffffffffu, kept);
                if (lane == 0 && base + warp * 32 < n) kmask[(base >> 5) + warp] = bk;
                if (kept && (region[slot] & kCandNextBit)) ++my_pn;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) my_pn += __shfl_xor_sync(0xffffffffu, my_pn, o);
            if (lane == 0 && my_pn) atomicAdd(&s_pnext, my_pn);
            ConsumerSync::sync();
            p_next = s_pnext + (new_cand ? 1 : 0);
        } else {
            const uint32_t *m = reinterpret_cast<const uint32_t *>(meta);
            for (int w = tid; w * 32 < n; w += kPConsumers) kmask[w] = m[w];
            ConsumerSync::sync();
        }

        // ---- pass 1: attention, and the sum of the normalised rows the next step scores -------
        float qf[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int x = sub * 8 + e;
            qf[e] = x < c.d ? __bfloat162float(a.q[(size_t)local * c.d + x]) * c.scale_log2e : 0.f;
        }
        float m = -FLT_MAX, l = 0.f, acc[8], sn[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) { acc[e] = 0.f; sn[e] = 0.f; }
        if (warp == 0) {   // the new row, always attended
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

        for (int t = 0; t < n_tiles; ++t, ++it) {
            const int stage = it % NST;
            wait(bar_full(stage), (it / NST) & 1);
            const __nv_bfloat16 *kbuf = reinterpret_cast<const __nv_bfloat16 *>(smem + L.stages + stage * 2 * L.tile_bytes);
            const __nv_bfloat16 *vbuf = reinterpret_cast<const __nv_bfloat16 *>(smem + L.stages + stage * 2 * L.tile_bytes + L.tile_bytes);
            const int r0 = t * TILE, r1 = min(n, r0 + TILE);
            uint4 kr[kPUnroll], vr[kPUnroll];
            bool ok[kPUnroll];
            float wn[kPUnroll];
#pragma unroll
            for (int u = 0; u < kPUnroll; ++u) {
                int row = r0 + u * STEP + warp * RPW + grp;
                ok[u] = row < r1 && ((kmask[row >> 5] >> (row & 31)) & 1u);
                kr[u] = make_uint4(0u, 0u, 0u, 0u);
                vr[u] = make_uint4(0u, 0u, 0u, 0u);
                wn[u] = 0.f;
                if (ok[u] && piece_ok) {
                    size_t off = (size_t)(row - r0) * c.row_stride + sub * 8;
                    kr[u] = lds128(kbuf + off);
                    vr[u] = lds128(vbuf + off);
                }
                if constexpr (FUSED) {
                    if (ok[u] && (region[row] & kCandNextBit)) wn[u] = inv_s[row];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(stage));   // the tile is in registers: the stage may be refilled
            float s[kPUnroll], m_new = m;
#pragma unroll
            for (int u = 0; u < kPUnroll; ++u) {
                float kf[8];
                unpack8(kr[u], kf);
                float tt = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) tt = fmaf(qf[e], kf[e], tt);
#pragma unroll
                for (int o = 1; o < LPR; o <<= 1) tt += __shfl_xor_sync(0xffffffffu, tt, o);
                s[u] = ok[u] ? tt : -INFINITY;
                m_new = fmaxf(m_new, s[u]);
            }
            float corr = exp2f(m - m_new);
            l *= corr;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= corr;
#pragma unroll
            for (int u = 0; u < kPUnroll; ++u) {
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

        // ---- lane groups -> warp -> block: the output row and s --------------------------------
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
        if (grp == 0) {
            float *w = wred + warp * wstride;
            if (piece_ok) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { w[sub * 8 + e] = acc[e]; w[c.row_stride + sub * 8 + e] = sn[e]; }
            }
            if (sub == 0) { w[2 * c.row_stride] = m; w[2 * c.row_stride + 1] = l; }
        }
        ConsumerSync::sync();
        if (tid < c.row_stride) {
            float M = -FLT_MAX, Lb = 0.f, A = 0.f, SN = 0.f;
#pragma unroll
            for (int w = 0; w < kPWarps; ++w) M = fmaxf(M, wred[w * wstride + 2 * c.row_stride]);
#pragma unroll
            for (int w = 0; w < kPWarps; ++w) {
                const float *ws = wred + w * wstride;
                float wgt = exp2f(ws[2 * c.row_stride] - M);
                Lb = fmaf(ws[2 * c.row_stride + 1], wgt, Lb);
                A = fmaf(ws[tid], wgt, A);
                SN += ws[c.row_stride + tid];
            }
            if (tid < c.d) {
                float o = A / Lb;
                if (a.out_f32) a.out_f32[(size_t)local * c.d + tid] = o;
                if (a.out_bf16) a.out_bf16[(size_t)local * c.d + tid] = __float2bfloat16_rn(o);
            }
            svec[tid] = SN;
        }

        if constexpr (FUSED) {
            // ---- Section 4.2 bookkeeping: holes below the new length, survivors above it --------
            int32_t *holes = reinterpret_cast<int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;   // keys are dead now
            const int top = max(n, n2);
            for (int base = 0; base < top; base += kPConsumers) {
                int s = base + tid;
                bool kept = s < n && ((kmask[s >> 5] >> (s & 31)) & 1u);
                bool is_hole = s < n2 && !kept, is_surv = s >= n2 && s < n && kept;
                unsigned bh = __ballot_sync(0xffffffffu, is_hole), bs = __ballot_sync(0xffffffffu, is_surv);
                if (lane == 0) { s_wcnt[0][warp] = __popc(bh); s_wcnt[1][warp] = __popc(bs); }
                ConsumerSync::sync();
                int oh = s_nholes, os = s_nsurv;
                for (int w = 0; w < warp; ++w) { oh += s_wcnt[0][w]; os += s_wcnt[1][w]; }
                unsigned below = (1u << lane) - 1u;
                if (is_hole) holes[oh + __popc(bh & below)] = s;
                if (is_surv) surv[os + __popc(bs & below)] = s;
                ConsumerSync::sync();
                if (tid == 0) {
                    for (int w = 0; w < kPWarps; ++w) { s_nholes += s_wcnt[0][w]; s_nsurv += s_wcnt[1][w]; }
                }
                ConsumerSync::sync();
            }
            const int nh = s_nholes, ns = s_nsurv;
            const int have = (n + c.page_rows - 1) / c.page_rows, need = (n2 + c.page_rows - 1) / c.page_rows;
            if (tid == 0) {
                s_ok = 1;
                if (nh != ns + 1) { set_status(c, ADSA_DEV_BAD_EVICT); s_ok = 0; }
                else if (n2 > c.max_rows) { set_status(c, ADSA_DEV_ROW_OVERFLOW); s_ok = 0; }
                else if (need > have && !resize_pages(c, pt, have, need)) s_ok = 0;
            }
            ConsumerSync::sync();   // also: svec is complete
            const bool okay = s_ok != 0;
            float sv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) sv[e] = piece_ok ? svec[sub * 8 + e] : 0.f;
            const float denom = (float)(p_next - 1);
            float *scores = c.scores + (size_t)sid * c.max_rows;

            // ---- pass 2: Eq. 1-2 of the next step, S_i = (u_i.s - u_i.u_i)/(p'-1), written at the row's new slot ----
            for (int t = 0; t < n_tiles; ++t, ++it) {
                const int stage = it % NST;
                wait(bar_full(stage), (it / NST) & 1);
                const __nv_bfloat16 *vbuf = reinterpret_cast<const __nv_bfloat16 *>(smem + L.stages + stage * 2 * L.tile_bytes + L.tile_bytes);
                const int r0 = t * TILE, r1 = min(n, r0 + TILE);
#pragma unroll
                for (int u = 0; u < kPUnroll; ++u) {
                    const int row = r0 + u * STEP + warp * RPW + grp;
                    const bool want = okay && row < r1 && ((kmask[row >> 5] >> (row & 31)) & 1u) && (region[row] & kCandNextBit);
                    float dot = 0.f, self = 0.f;
                    if (want && piece_ok) {
                        float f[8];
                        unpack8(lds128(vbuf + (size_t)(row - r0) * c.row_stride + sub * 8), f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], sv[e], dot); self = fmaf(f[e], f[e], self); }
                    }
#pragma unroll
                    for (int o = 1; o < LPR; o <<= 1) {
                        dot += __shfl_xor_sync(0xffffffffu, dot, o);
                        self += __shfl_xor_sync(0xffffffffu, self, o);
                    }
                    if (want && sub == 0) {
                        int dst = row;
                        if (row >= n2) {   // a survivor: it moves into the hole of the same rank
                            int lo = 0, hi = ns - 1;
                            while (lo < hi) { int mid = (lo + hi) >> 1; if (surv[mid] < row) lo = mid + 1; else hi = mid; }
                            dst = holes[lo];
                        }
                        float inv = inv_s[row];
                        scores[dst] = p_next > 1 ? (inv * dot - inv * inv * self) / denom + 0.0f : 0.0f;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty(stage));
            }

            // ---- the update itself -------------------------------------------------------------
            if (okay) {
                const int pieces = c.row_stride >> 3;
                for (int i = warp; i < ns; i += kPWarps) {   // survivors move down, 16-byte pieces of K and of V
                    const int row = surv[i], dst = holes[i];
                    size_t so = row_offset(c, pt, row), go = row_offset(c, pt, dst);
                    for (int x = lane; x < 2 * pieces; x += 32) {
                        __nv_bfloat16 *pool = x < pieces ? c.k_pool : c.v_pool;
                        int pc = x < pieces ? x : x - pieces;
                        reinterpret_cast<uint4 *>(pool + go)[pc] = reinterpret_cast<const uint4 *>(pool + so)[pc];
                    }
                    if (lane == 0) {
                        c.pos[(size_t)sid * c.max_rows + dst] = pos_s[row];
                        c.inv_norm[(size_t)sid * c.max_rows + dst] = inv_s[row];
                    }
                }
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
        ConsumerSync::sync();   // everyone is done with this stream's metadata, lists and reduction buffers
        if (tid == 0) mbar_arrive(bar_mempty(mb));
    }
}

// ---- host side ------------------------------------------------------------
namespace {

int p_lanes(int row_stride)
{
    int pieces = row_stride / 8;
    return pieces <= 4 ? 4 : pieces <= 8 ? 8 : pieces <= 16 ? 16 : 32;
}

template <int LPR>
cudaError_t p_configure()
{
    cudaError_t e = cudaFuncSetAttribute(pstep_kernel<LPR, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(pstep_kernel<LPR, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
}

}  // namespace

cudaError_t configure_pstep_kernel(const DevCtx &c)
{
    switch (p_lanes(c.row_stride)) {
    case 4: return p_configure<4>();
    case 8: return p_configure<8>();
    case 16: return p_configure<16>();
    default: return p_configure<32>();
    }
}

// Number of ring stages that fit (0: the configuration does not fit at all).
PStepPlan plan_pstep(const DevCtx &c, bool fused, int sm_count, int max_stages)
{
    PStepPlan p = {};
    const int tile_rows = kPWarps * (32 / p_lanes(c.row_stride)) * kPUnroll;
    int cap = max_stages > 0 && max_stages < kPMaxStages ? max_stages : kPMaxStages;
    for (int ns = cap; ns >= 3; --ns) {
        PLayout L = p_layout(c.max_rows, c.max_pages, c.mask_words, c.row_stride, tile_rows, ns, fused);
        if (L.total + 2048 <= (uint32_t)kPSmemLimit) {
            p.n_stages = ns; p.smem_bytes = L.total; p.grid = c.S < sm_count ? c.S : sm_count; p.tile_rows = tile_rows;
            return p;
        }
    }
    return p;
}

cudaError_t launch_pstep(const DevCtx &c, const PStepPlan &plan, bool fused, int layer, int cur_pos, int budget_rows,
                         const void *q, const void *k_new, const void *v_new, void *out_bf16, float *out_f32,
                         cudaStream_t st)
{
    PStepArgs a;
    a.layer = layer; a.cur_pos = cur_pos; a.budget_rows = budget_rows; a.n_stages = plan.n_stages;
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    const dim3 grid(plan.grid), block(kPThreads);
    const size_t sm = plan.smem_bytes;
#define ADSA_PSTEP_CASE(LPR)                                                                 \
    if (fused) pstep_kernel<LPR, true><<<grid, block, sm, st>>>(c, a);                        \
    else pstep_kernel<LPR, false><<<grid, block, sm, st>>>(c, a);                             \
    break
    switch (p_lanes(c.row_stride)) {
    case 4: ADSA_PSTEP_CASE(4);
    case 8: ADSA_PSTEP_CASE(8);
    case 16: ADSA_PSTEP_CASE(16);
    default: ADSA_PSTEP_CASE(32);
    }
#undef ADSA_PSTEP_CASE
    return cudaGetLastError();
}

}  // namespace adsa
