// The persistent pipelined stream kernel with tensor-core arithmetic, for pools
// whose rows are 64 elements (128 bytes) wide.
//
// Why tensor cores for a matrix-vector product.  One query per private KV stream
// gives 1 flop per byte, so the arithmetic is nowhere near a limit, but the
// INSTRUCTIONS are: a B200 issues about 1.1e12 warp instructions per second
// against 6.5e12 bytes per second of HBM, i.e. one warp instruction per 6 bytes
// of K/V.  Unpacking bf16 and running fp32 FMAs on the CUDA cores costs about 38
// warp instructions per 256-byte K+V row (measured), which caps attention alone at
// roughly half the HBM rate before any stall.  mma.sync.m16n8k16 consumes the
// bf16 rows as they lie in shared memory: about 6 warp instructions per row for
// attention and the next step's score sums together.  The M dimension of the MMAs
// is mostly padding; what is bought is issue slots, not flops.
//
// Structure (as in the CUDA-core persistent kernel): one CTA per SM slot walks
// over streams; a producer warp keeps a ring of stages full, each stage a tile of
// 32 K rows and 32 V rows, written by TMA tensor copies with the 128-byte swizzle
// so that ldmatrix reads them without bank conflicts.  Tiles are dealt to the
// eight consumer warps round-robin; each warp keeps its own online-softmax state
// per stream, merged through shared memory at the end of a stream.
//
// Pass 1, per tile:  S = q.K^T  (A = q in rows 0-7, B = K rows via ldmatrix);
//   P = exp2(S*scale - m), split into bf16 hi + lo so the product keeps fp32-like
//   accuracy;  O_tile = A'.V with A' rows {P_hi, P_lo, w_hi, w_mid, w_lo}, where
//   w_j = 1/|v_j| for the rows the next step will score and 0 otherwise: rows 0-1 of
//   the result accumulate softmax.V, rows 2-4 accumulate s = sum of normalised rows.
//   Each tile's product starts from zero and is folded into fp32 running sums with
//   round-to-nearest FMAs, so tensor-core accumulation rounding never compounds
//   beyond 32 rows.
// Pass 2 (fused), per tile of V rows again (from L2):  dot_i = v_i . s with s split
//   into three bf16 parts as B columns 0-2;  S_i = (dot_i/|v_i| - 1) / (p' - 1), Eq. 1-2
//   for the next step (u_i.u_i = 1 unless |v_i| was clamped, in which case it is
//   computed from the row).
//
// Rows of a partial last tile that were not copied hold older (finite) data and are
// masked; the ring is zeroed once at kernel start so no NaN pattern can meet a zero
// weight.  Every wait is bounded (see adsa_pstep.cu).
#include <cuda.h>
#include <float.h>
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"
#include "adsa_select.cuh"
#include "adsa_async.cuh"

namespace adsa {

constexpr int kMConsumers = kSelThreads;          // 256 consumer threads (8 warps) ...
constexpr int kMWarps = kMConsumers / 32;
constexpr int kMThreads = kMConsumers + 32;       // ... and one producer warp
constexpr int kMTile = 32;                        // rows per tile
constexpr int kMRowBytes = 128;                   // 64 bf16
constexpr int kMTileBytes = kMTile * kMRowBytes;  // one K (or V) tile
constexpr int kMStageBytes = 2 * kMTileBytes;

struct MLayout {
    uint32_t bars, hdr, meta[2], pt[2], keys, region, kmask, wsplit, wred, svec, stages;
    uint32_t meta_words, w_rows;
    uint32_t total;
};

__host__ __device__ inline uint32_t m_align(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline MLayout m_layout(int max_rows, int max_pages, int mask_words, int n_stages, bool fused)
{
    MLayout L;
    uint32_t off = 0;
    L.bars = off;   off += (2 * kPMaxStages + 4) * 8;
    L.hdr = off;    off += 2 * 16;
    L.meta_words = m_align(max_rows + 8, 4);
    const uint32_t meta_bytes = fused ? 3 * L.meta_words * 4 : m_align(mask_words * 4, 16);
    L.meta[0] = off; off += meta_bytes;
    L.meta[1] = off; off += meta_bytes;
    L.pt[0] = off;  off += m_align(max_pages * 4, 16);
    L.pt[1] = off;  off += m_align(max_pages * 4, 16);
    L.keys = off;   off += fused ? m_align((max_rows + 2) * 8, 16) : 0;
    L.region = off; off += fused ? m_align(max_rows + kMTile, 16) : 0;
    L.kmask = off;  off += m_align((mask_words + 1) * 4, 16);
    L.w_rows = m_align(max_rows + kMTile, 32);
    L.wsplit = off; off += fused ? 3 * L.w_rows * 2 : 0;               // bf16 hi | mid | lo of the row weights
    L.wred = off;   off += (kMWarps + 1) * (2 * 64 + 2) * 4;           // per warp (+ the new row): acc | s | m, l
    L.svec = off;   off += 64 * 4;
    off = m_align(off, 1024);                                          // the swizzle pattern repeats every 1024 bytes
    L.stages = off; off += n_stages * kMStageBytes;
    L.total = off;
    return L;
}

struct MStepArgs {
    int layer, cur_pos, budget_rows, n_stages;
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out_bf16;
    float *out_f32;
};

// ---- PTX wrappers ---------------------------------------------------------
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A(16x16, row) * B(16x8, col), bf16 in, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two floats -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }
// byte offset of 16-byte chunk c of row r inside a tile written with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * kMRowBytes + ((c ^ (r & 7)) << 4)); }

template <bool FUSED>
__global__ void __launch_bounds__(kMThreads, 1)
mstep_kernel(DevCtx c, MStepArgs a, const __grid_constant__ MStepMaps maps)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ SelScratch s_sel;
    __shared__ int s_wcnt[2][kMWarps], s_nholes, s_nsurv, s_pnext, s_ok;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NST = a.n_stages;
    const MLayout L = m_layout(c.max_rows, c.max_pages, c.mask_words, NST, FUSED);
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + L.bars);
    auto bar_full = [&](int s) { return smem_u32(bars + s); };
    auto bar_empty = [&](int s) { return smem_u32(bars + kPMaxStages + s); };
    auto bar_mfull = [&](int b) { return smem_u32(bars + 2 * kPMaxStages + b); };
    auto bar_mempty = [&](int b) { return smem_u32(bars + 2 * kPMaxStages + 2 + b); };
    const uint32_t stages_u32 = smem_u32(smem + L.stages);

    if (tid == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_mfull(b), 1); mbar_init(bar_mempty(b), 1); }
        mbar_init_fence();
        s_abort = 0;
    }
    {   // zero the ring once: rows a partial tile never receives must hold finite numbers
        uint4 *z = reinterpret_cast<uint4 *>(smem + L.stages);
        for (int i = tid; i < NST * kMStageBytes / 16; i += kMThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    auto wait = [&](uint32_t bar, uint32_t parity) {
        int limit = s_abort ? kCopySpinAfterTimeout : kCopySpinLimit;
        if (!mbar_wait_sleepy(bar, parity, limit)) {
            if (lane == 0) set_status(c, ADSA_DEV_COPY_TIMEOUT);
            s_abort = 1;
        }
    };

    if (warp == kMWarps) {
        // =============================== producer warp ===============================
        uint32_t it = 0;
        int j = 0;
        for (int local = blockIdx.x; local < c.S; local += gridDim.x, ++j) {
            const int sid = a.layer * c.S + local, mb = j & 1;
            const int32_t *pt_g = c.page_table + (size_t)sid * c.max_pages;
            int32_t *pt_s = reinterpret_cast<int32_t *>(smem + L.pt[mb]);
            wait(bar_mempty(mb), ((j >> 1) & 1) ^ 1);
            int n = c.n_live[sid];
            if (n < 0 || n > c.max_rows) { if (lane == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW); n = 0; }
            const int np = (n + c.page_rows - 1) / c.page_rows;
            for (int pg = lane; pg < np; pg += 32) pt_s[pg] = pt_g[pg];
            unsigned char *meta = smem + L.meta[mb];
            uint32_t meta_tx = 0;
            if constexpr (FUSED) {
                const void *src[3] = {c.pos + (size_t)sid * c.max_rows, c.scores + (size_t)sid * c.max_rows,
                                      c.inv_norm + (size_t)sid * c.max_rows};
#pragma unroll
                for (int k = 0; k < 3; ++k) {   // aligned interior by bulk copy, ragged ends by plain loads
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
                const uint32_t *g = c.keep_mask + (size_t)local * c.mask_words;
                uint32_t *d = reinterpret_cast<uint32_t *>(meta);
                for (int w = lane; w * 32 < n; w += 32) d[w] = g[w];
            }
            if (lane == 0) reinterpret_cast<int *>(smem + L.hdr)[mb * 4] = n;
            __syncwarp();
            if (lane == 0) mbar_expect_tx(bar_mfull(mb), meta_tx);
            if (lane == 0) {
                const int n_tiles = (n + kMTile - 1) / kMTile;
                for (int pass = 0; pass < (FUSED ? 2 : 1); ++pass) {
                    for (int t = 0; t < n_tiles; ++t, ++it) {
                        const int stage = it % NST;
                        wait(bar_empty(stage), ((it / NST) & 1) ^ 1);
                        const int r0 = t * kMTile, r1 = min(n, r0 + kMTile);
                        const uint32_t kdst = stages_u32 + stage * kMStageBytes, vdst = kdst + kMTileBytes;
                        const uint32_t bar = bar_full(stage);
                        mbar_expect_tx(bar, (uint32_t)(r1 - r0) * kMRowBytes * (pass == 0 ? 2u : 1u));
                        int r = r0;
                        while (r < r1) {   // page pieces, each cut into boxes of 32, 16, 8, 4, 2 or 1 rows
                            uint32_t pg = __umulhi((uint32_t)r, c.pr_magic);
                            int in = r - (int)pg * c.page_rows;
                            int cnt = min(r1 - r, c.page_rows - in);
                            int y = pt_s[pg] * c.page_rows + in;
                            uint32_t off = (uint32_t)(r - r0) * kMRowBytes;
                            r += cnt;
                            while (cnt > 0) {
                                int hb = 31 - __clz(cnt);
                                hb = hb > 5 ? 5 : hb;
                                if (pass == 0) tma_2d(kdst + off, &maps.k[hb], 0, y, bar);
                                tma_2d(vdst + off, &maps.v[hb], 0, y, bar);
                                y += 1 << hb; off += (uint32_t)kMRowBytes << hb; cnt -= 1 << hb;
                            }
                        }
                    }
                }
            }
            __syncwarp();
        }
        if (lane == 0) {   // the last round of every stage has landed before the CTA leaves
            for (uint32_t back = 0; back < (uint32_t)NST && back < it; ++back) {
                uint32_t i = it - 1 - back;
                mbar_wait_sleepy(bar_full(i % NST), (i / NST) & 1, s_abort ? kCopySpinAfterTimeout : kCopySpinLimit);
            }
        }
        return;
    }

    // ================================= consumer warps =================================
    const int g = lane >> 2, t = lane & 3;          // MMA fragment coordinates
    const int mi = lane >> 3, lr = lane & 7;        // ldmatrix: matrix index, row within the matrix
    unsigned long long *sm_keys = reinterpret_cast<unsigned long long *>(smem + L.keys);
    uint8_t *region = smem + L.region;
    uint32_t *kmask = reinterpret_cast<uint32_t *>(smem + L.kmask);
    __nv_bfloat16 *wsplit = reinterpret_cast<__nv_bfloat16 *>(smem + L.wsplit);
    float *wred = reinterpret_cast<float *>(smem + L.wred);
    float *svec = reinterpret_cast<float *>(smem + L.svec);
    constexpr int wstride = 2 * 64 + 2;
    const bool new_cand = FUSED && region_of(c, a.cur_pos, a.cur_pos + 1) == kRegionPrevious;
    // which row of A' this lane group feeds in the P.V product
    const uint32_t *w_role = reinterpret_cast<const uint32_t *>(wsplit + (size_t)(g >= 2 && g <= 4 ? g - 2 : 0) * L.w_rows);

    uint32_t it = 0;
    int j = 0;
    for (int local = blockIdx.x; local < c.S; local += gridDim.x, ++j) {
        const int sid = a.layer * c.S + local, mb = j & 1;
        int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
        wait(bar_mfull(mb), (j >> 1) & 1);
        const int n = reinterpret_cast<const int *>(smem + L.hdr)[mb * 4];
        const int n_tiles = (n + kMTile - 1) / kMTile;
        const unsigned char *meta = smem + L.meta[mb];
        const int32_t *pos_s = nullptr;
        const float *inv_s = nullptr;
        int n2 = n, p_next = 0;

        // ---- which rows are attended, and the weights of the rows the next step scores -----------
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
            const int n_pad = n_tiles * kMTile;
            for (int base = 0; base < n_pad; base += kMConsumers) {
                int slot = base + tid;
                bool kept = slot < n && sel.keeps(region[slot], sm_keys[slot]);
                if (slot < n && (region[slot] & 3) == kRegionInvalid) set_status(c, ADSA_DEV_BAD_POSITION);
                unsigned bk = __ballot_sync(0xffffffffu, kept);
                if (lane == 0 && base + warp * 32 < n_pad) kmask[(base >> 5) + warp] = bk;
                const bool cand = kept && (region[slot] & kCandNextBit);
                if (cand) ++my_pn;
                if (slot < n_pad) {   // w = 1/|v| for the rows the next step scores, as three bf16 parts (24 bits)
                    float w = cand ? inv_s[slot] : 0.f;
                    __nv_bfloat16 h = __float2bfloat16_rn(w);
                    float r1 = w - __bfloat162float(h);
                    __nv_bfloat16 md = __float2bfloat16_rn(r1);
                    __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(md));
                    wsplit[slot] = h; wsplit[L.w_rows + slot] = md; wsplit[2 * L.w_rows + slot] = lo;
                    if (slot >= n) region[slot] = 0;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) my_pn += __shfl_xor_sync(0xffffffffu, my_pn, o);
            if (lane == 0 && my_pn) atomicAdd(&s_pnext, my_pn);
            ConsumerSync::sync();
            p_next = s_pnext + (new_cand ? 1 : 0);
        } else {
            const uint32_t *m = reinterpret_cast<const uint32_t *>(meta);
            for (int w = tid; w < n_tiles; w += kMConsumers) {
                uint32_t bits = m[w];
                int valid = n - w * 32;
                kmask[w] = valid >= 32 ? bits : (bits & ((1u << valid) - 1u));
            }
            ConsumerSync::sync();
        }

        // ---- q as the A operand (rows 0-7 = q, rows 8-15 = 0), four k-steps of 16 elements ------
        uint32_t qa0[4], qa2[4];
        {
            const uint32_t *q2 = reinterpret_cast<const uint32_t *>(a.q + (size_t)local * c.d);   // c.d is even
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                int e0 = 16 * ks + 2 * t, e1 = e0 + 8;
                qa0[ks] = e0 + 1 < c.d ? q2[e0 >> 1] : (e0 < c.d ? (q2[e0 >> 1] & 0xffffu) : 0u);
                qa2[ks] = e1 + 1 < c.d ? q2[e1 >> 1] : (e1 < c.d ? (q2[e1 >> 1] & 0xffffu) : 0u);
            }
        }

        // ---- pass 1 ---------------------------------------------------------------------------
        float m_run = -FLT_MAX, l_run = 0.f, o_run[8][2];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) { o_run[nb][0] = 0.f; o_run[nb][1] = 0.f; }

        for (int tl = 0; tl < n_tiles; ++tl, ++it) {
            if ((int)(it % kMWarps) != warp) continue;
            const int stage = it % NST;
            wait(bar_full(stage), (it / NST) & 1);
            const uint32_t kb = stages_u32 + stage * kMStageBytes, vb = kb + kMTileBytes;
            const int r0 = tl * kMTile;
            const uint32_t kw = kmask[tl];
            // S = q.K^T: four blocks of 8 rows
            float sc[4][4];
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
                sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
                uint32_t kf0[4], kf1[4];
                const int row = 8 * nb + lr;
                ldsm_x4(kb + swz(row, mi), kf0);         // elements 0-31 of the 8 rows
                ldsm_x4(kb + swz(row, 4 + mi), kf1);     // elements 32-63
                mma_bf16(sc[nb], qa0[0], 0u, qa2[0], 0u, kf0[0], kf0[1]);
                mma_bf16(sc[nb], qa0[1], 0u, qa2[1], 0u, kf0[2], kf0[3]);
                mma_bf16(sc[nb], qa0[2], 0u, qa2[2], 0u, kf1[0], kf1[1]);
                mma_bf16(sc[nb], qa0[3], 0u, qa2[3], 0u, kf1[2], kf1[3]);
            }
            // this lane's 8 logits: rows 8*nb + 2t, 8*nb + 2t + 1 (the same in every lane group)
            float x[4][2], mx = -INFINITY;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    bool kept = (kw >> (8 * nb + 2 * t + e)) & 1u;
                    x[nb][e] = kept ? sc[nb][e] * c.scale_log2e : -INFINITY;
                    mx = fmaxf(mx, x[nb][e]);
                }
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run, mx);
            const float corr = exp2f(m_run - m_new);
            m_run = m_new;
            float psum = 0.f;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) { x[nb][e] = exp2f(x[nb][e] - m_new); psum += x[nb][e]; }
            }
            l_run = fmaf(l_run, corr, psum);
            // A' fragments for the two 16-row k-steps: row g of A' is P_hi, P_lo, w_hi, w_mid, w_lo, 0, 0, 0
            uint32_t pa0[2], pa2[2];
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                uint32_t h0 = pack_bf16(x[2 * ks][0], x[2 * ks][1]), h2 = pack_bf16(x[2 * ks + 1][0], x[2 * ks + 1][1]);
                uint32_t l0 = pack_bf16(x[2 * ks][0] - bf16_lo(h0), x[2 * ks][1] - bf16_hi(h0));
                uint32_t l2 = pack_bf16(x[2 * ks + 1][0] - bf16_lo(h2), x[2 * ks + 1][1] - bf16_hi(h2));
                uint32_t w0 = 0u, w2 = 0u;
                if constexpr (FUSED) {
                    w0 = w_role[(r0 + 16 * ks + 2 * t) >> 1];
                    w2 = w_role[(r0 + 16 * ks + 8 + 2 * t) >> 1];
                }
                pa0[ks] = g == 0 ? h0 : g == 1 ? l0 : g <= 4 ? w0 : 0u;
                pa2[ks] = g == 0 ? h2 : g == 1 ? l2 : g <= 4 ? w2 : 0u;
            }
            // O_tile = A'.V from zero, then folded into the running sums
            float ot[8][4];
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) ot[nb][0] = ot[nb][1] = ot[nb][2] = ot[nb][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
                for (int nbp = 0; nbp < 4; ++nbp) {
                    uint32_t vf[4];
                    ldsm_x4_t(vb + swz(16 * ks + 8 * (mi & 1) + lr, 2 * nbp + (mi >> 1)), vf);
                    mma_bf16(ot[2 * nbp], pa0[ks], 0u, pa2[ks], 0u, vf[0], vf[1]);
                    mma_bf16(ot[2 * nbp + 1], pa0[ks], 0u, pa2[ks], 0u, vf[2], vf[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(stage));   // everything of the tile is in registers
            const float corr_row = g < 2 ? corr : 1.0f;     // the weight sums are not softmax-scaled
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
                o_run[nb][0] = fmaf(o_run[nb][0], corr_row, ot[nb][0]);
                o_run[nb][1] = fmaf(o_run[nb][1], corr_row, ot[nb][1]);
            }
        }

        // ---- per warp: softmax.V = rows 0 + 1, s = rows 2 + 3 + 4; then warps -> block -------------
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        {
            float *w = wred + warp * wstride;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float v = o_run[nb][e];
                    float up1 = __shfl_down_sync(0xffffffffu, v, 4), up2 = __shfl_down_sync(0xffffffffu, v, 8);
                    if (g == 0) w[8 * nb + 2 * t + e] = v + up1;
                    if (g == 2) w[64 + 8 * nb + 2 * t + e] = (v + up1) + up2;
                }
            }
            if (lane == 0) { w[128] = m_run; w[129] = l_run; }
        }
        if (warp == 0) {   // the new row, always attended: one more partial state
            float *w = wred + kMWarps * wstride;
            float s = 0.f, ss = 0.f, vf[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int xx = 2 * lane + e;
                float qf = xx < c.d ? __bfloat162float(a.q[(size_t)local * c.d + xx]) : 0.f;
                float kf = xx < c.d ? __bfloat162float(a.k_new[(size_t)local * c.d + xx]) : 0.f;
                vf[e] = xx < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + xx]) : 0.f;
                s = fmaf(qf, kf, s);
                ss = fmaf(vf[e], vf[e], ss);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, o);
                ss += __shfl_xor_sync(0xffffffffu, ss, o);
            }
            const float inv_new = new_cand ? 1.0f / fmaxf(sqrtf(ss), kNormEps) : 0.f;
#pragma unroll
            for (int e = 0; e < 2; ++e) { w[2 * lane + e] = vf[e]; w[64 + 2 * lane + e] = inv_new * vf[e]; }
            if (lane == 0) { w[128] = s * c.scale_log2e; w[129] = 1.f; }
        }
        ConsumerSync::sync();
        if (tid < 64) {
            float M = -FLT_MAX, Lb = 0.f, A = 0.f, SN = 0.f;
#pragma unroll
            for (int w = 0; w <= kMWarps; ++w) M = fmaxf(M, wred[w * wstride + 128]);
#pragma unroll
            for (int w = 0; w <= kMWarps; ++w) {
                const float *ws = wred + w * wstride;
                float wgt = exp2f(ws[128] - M);
                Lb = fmaf(ws[129], wgt, Lb);
                A = fmaf(ws[tid], wgt, A);
                SN += ws[64 + tid];
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
            int32_t *holes = reinterpret_cast<int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;
            const int top = max(n, n2);
            for (int base = 0; base < top; base += kMConsumers) {
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
                    for (int w = 0; w < kMWarps; ++w) { s_nholes += s_wcnt[0][w]; s_nsurv += s_wcnt[1][w]; }
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
            const float denom = (float)(p_next - 1);
            float *scores = c.scores + (size_t)sid * c.max_rows;

            // s as the B operand: columns 0, 1, 2 = its bf16 hi, mid, lo parts
            uint32_t sb0[4], sb1[4];
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                float v[4] = {svec[16 * ks + 2 * t], svec[16 * ks + 2 * t + 1], svec[16 * ks + 2 * t + 8], svec[16 * ks + 2 * t + 9]};
                float part[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float h = __bfloat162float(__float2bfloat16_rn(v[i]));
                    float md = __bfloat162float(__float2bfloat16_rn(v[i] - h));
                    float lo = __bfloat162float(__float2bfloat16_rn(v[i] - h - md));
                    part[i] = g == 0 ? h : g == 1 ? md : g == 2 ? lo : 0.f;
                }
                sb0[ks] = pack_bf16(part[0], part[1]);
                sb1[ks] = pack_bf16(part[2], part[3]);
            }

            // ---- pass 2: dot_i = v_i . s, S_i = (dot_i/|v_i| - u_i.u_i) / (p' - 1), written at the row's new slot ----
            for (int tl = 0; tl < n_tiles; ++tl, ++it) {
                if ((int)(it % kMWarps) != warp) continue;
                const int stage = it % NST;
                wait(bar_full(stage), (it / NST) & 1);
                const uint32_t vb = stages_u32 + stage * kMStageBytes + kMTileBytes;
                const int r0 = tl * kMTile;
                float dt[2][4];
#pragma unroll
                for (int mbk = 0; mbk < 2; ++mbk) {
                    dt[mbk][0] = dt[mbk][1] = dt[mbk][2] = dt[mbk][3] = 0.f;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        uint32_t af[4];
                        ldsm_x4(vb + swz(16 * mbk + 8 * (mi & 1) + lr, 2 * ks + (mi >> 1)), af);
                        mma_bf16(dt[mbk], af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                    }
                }
#pragma unroll
                for (int mbk = 0; mbk < 2; ++mbk) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {   // rows 16*mbk + g and + 8: columns 0, 1 in lane t = 0, column 2 in t = 1
                        float lo = __shfl_down_sync(0xffffffffu, dt[mbk][2 * hh], 1);
                        const int row = r0 + 16 * mbk + 8 * hh + g;
                        const bool want = okay && t == 0 && ((kmask[tl] >> (16 * mbk + 8 * hh + g)) & 1u) &&
                                          (region[row] & kCandNextBit);
                        if (want) {
                            float dot = (dt[mbk][2 * hh] + dt[mbk][2 * hh + 1]) + lo;
                            float inv = inv_s[row], self = 1.0f;
                            if (inv >= 1.0f / kNormEps) {   // |v| was clamped: u.u is not 1, take it from the row
                                float ss = 0.f;
                                for (int ch = 0; ch < 8; ++ch) {
                                    float f[8];
                                    unpack8(*reinterpret_cast<const uint4 *>(smem + L.stages + stage * kMStageBytes + kMTileBytes +
                                                                           swz(row - r0, ch)), f);
                                    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
                                }
                                self = inv * inv * ss;
                            }
                            int dst = row;
                            if (row >= n2) {
                                int lo_i = 0, hi_i = ns - 1;
                                while (lo_i < hi_i) { int mid = (lo_i + hi_i) >> 1; if (surv[mid] < row) lo_i = mid + 1; else hi_i = mid; }
                                dst = holes[lo_i];
                            }
                            scores[dst] = p_next > 1 ? (inv * dot - self) / denom + 0.0f : 0.0f;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty(stage));
            }

            // ---- the update itself -------------------------------------------------------------
            if (okay) {
                for (int i = warp; i < ns; i += kMWarps) {   // survivors move down: 8 + 8 pieces of 16 bytes
                    const int row = surv[i], dst = holes[i];
                    size_t so = row_offset(c, pt, row), go = row_offset(c, pt, dst);
                    if (lane < 16) {
                        __nv_bfloat16 *pool = lane < 8 ? c.k_pool : c.v_pool;
                        reinterpret_cast<uint4 *>(pool + go)[lane & 7] = reinterpret_cast<const uint4 *>(pool + so)[lane & 7];
                    }
                    if (lane == 0) {
                        c.pos[(size_t)sid * c.max_rows + dst] = pos_s[row];
                        c.inv_norm[(size_t)sid * c.max_rows + dst] = inv_s[row];
                    }
                }
                if (warp == 0 && new_cand) {   // the new row's own score for the next step
                    float dot = 0.f, ss = 0.f;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        int xx = 2 * lane + e;
                        float vf = xx < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + xx]) : 0.f;
                        dot = fmaf(vf, svec[xx], dot);
                        ss = fmaf(vf, vf, ss);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
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
        ConsumerSync::sync();
        if (tid == 0) mbar_arrive(bar_mempty(mb));
    }
}

// ---- host side ------------------------------------------------------------
bool mstep_supported(const DevCtx &c) { return c.row_stride == 64 && c.d % 2 == 0; }

// Tensor maps of both pools for boxes of 1, 2, 4, .. 32 rows (128-byte swizzle).  encode is
// cuTensorMapEncodeTiled, looked up at run time so that the library links cudart only.
int build_mstep_maps(const DevCtx &c, MStepMaps *out)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return -1;
    }
    typedef CUresult (*encode_t)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    encode_t encode = (encode_t)fn;
    const cuuint64_t dims[2] = {64, (cuuint64_t)c.n_pages * (cuuint64_t)c.page_rows};
    if (dims[1] > (1ull << 32)) return -1;
    const cuuint64_t strides[1] = {kMRowBytes};
    const cuuint32_t estr[2] = {1, 1};
    for (int pool = 0; pool < 2; ++pool) {
        for (int hb = 0; hb < 6; ++hb) {
            const cuuint32_t box[2] = {64, 1u << hb};
            CUtensorMap *m = pool == 0 ? &out->k[hb] : &out->v[hb];
            CUresult r = encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pool == 0 ? (void *)c.k_pool : (void *)c.v_pool,
                                dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return -1;
        }
    }
    return 0;
}

cudaError_t configure_mstep_kernel(const DevCtx &c)
{
    (void)c;
    cudaError_t e = cudaFuncSetAttribute(mstep_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(mstep_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
}

PStepPlan plan_mstep(const DevCtx &c, bool fused, int sm_count, int max_stages)
{
    PStepPlan p = {};
    if (!mstep_supported(c)) return p;
    int cap = max_stages > 0 && max_stages < kPMaxStages ? max_stages : kPMaxStages;
    for (int ns = cap; ns >= 3; --ns) {
        MLayout L = m_layout(c.max_rows, c.max_pages, c.mask_words, ns, fused);
        if (L.total + 2048 <= (uint32_t)kPSmemLimit) {
            p.n_stages = ns; p.smem_bytes = L.total; p.grid = c.S < sm_count ? c.S : sm_count; p.tile_rows = kMTile;
            return p;
        }
    }
    return p;
}

cudaError_t launch_mstep(const DevCtx &c, const PStepPlan &plan, const MStepMaps &maps, bool fused, int layer, int cur_pos,
                         int budget_rows, const void *q, const void *k_new, const void *v_new, void *out_bf16,
                         float *out_f32, cudaStream_t st)
{
    MStepArgs a;
    a.layer = layer; a.cur_pos = cur_pos; a.budget_rows = budget_rows; a.n_stages = plan.n_stages;
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    if (fused) mstep_kernel<true><<<plan.grid, kMThreads, plan.smem_bytes, st>>>(c, a, maps);
    else mstep_kernel<false><<<plan.grid, kMThreads, plan.smem_bytes, st>>>(c, a, maps);
    return cudaGetLastError();
}

}  // namespace adsa
