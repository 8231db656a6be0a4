// The warp-per-stream kernel with tensor-core arithmetic, for pools whose rows are
// 64 elements (128 bytes) wide.  This is the kernel the benchmark's layer-step runs.
//
// Why one warp per stream.  A layer-step of one stream is a chain of short,
// dependent phases (selection, attention sweep, reduction, score sweep, update).
// Spread over a whole CTA each phase ends in a barrier and the SM idles on latency;
// measured, a CTA-wide version spent 27 us per stream.  Here every warp is a
// self-contained worker: it owns a stream from start to finish, keeps its own
// metadata and its own small ring of tiles in shared memory, issues its own TMA
// copies, and never waits for another warp.  Latency is hidden the way GPUs hide
// it best, by the other warps of the SM being in different places of their chains.
//
// Why tensor cores for a matrix-vector product.  One query per private KV stream is
// 1 flop per byte, so arithmetic is no limit, but INSTRUCTIONS are: a B200 issues
// about 1.1e12 warp instructions per second against 6.5e12 bytes per second of HBM,
// one warp instruction per 6 bytes of K/V.  Unpacking bf16 and running fp32 FMAs on
// the CUDA cores costs about 38 warp instructions per 256-byte K+V row (measured),
// which caps attention alone near half the HBM rate.  mma.sync.m16n8k16 consumes the
// bf16 rows as they lie in shared memory: about 6 warp instructions per row for
// attention and the next step's score sums together.  The M dimension of the MMAs is
// mostly padding; what is bought is issue slots, not flops.
//
// Data path.  A tile is 32 K rows + 32 V rows (4 KB each), written by TMA tensor
// copies with the 128-byte swizzle so that ldmatrix reads it without bank conflicts
// (page pieces are cut into boxes of 32, 16, .. 1 rows: one tensor map per height).
// The warp's lane 0 issues tile u + depth as soon as tile u has been read.
//
// Pass 1, per tile:  S = q.K^T  (A = q in rows 0-7, B = K rows via ldmatrix);
//   P = exp2(S*scale - m), split into bf16 hi + lo so the product keeps fp32-like
//   accuracy;  O_tile = A'.V with A' rows {P_hi, P_lo, w_hi, w_mid, w_lo}, where
//   w_j = 1/|v_j| for the rows the next step will score and 0 otherwise: rows 0-1 of
//   the result accumulate softmax.V, rows 2-4 accumulate s = sum of normalised rows.
//   Each tile's product starts from zero and is folded into fp32 running sums with
//   round-to-nearest FMAs, so tensor-core accumulation rounding never compounds
//   beyond 32 rows.
// Pass 2 (fused), per tile of V rows again (they come out of L2):  dot_i = v_i . s
//   with s split into three bf16 parts as B columns 0-2;
//   S_i = (dot_i/|v_i| - u_i.u_i) / (p' - 1), Eq. 1-2 for the next step (u_i.u_i = 1
//   unless |v_i| was clamped, in which case it is computed from the row).
// Then the Section 4.2 update.  All rows of a stream are copied, retained or not
// (one row per step is not); rows of a partial last tile that were not copied hold
// older finite data and are masked; the ring is zeroed once at kernel start.
//
// Every wait on a copy is bounded: if it runs out the warp raises
// ADSA_DEV_COPY_TIMEOUT, shortens its later waits and runs to the end (all accesses
// stay in bounds).  A warp leaves only after every copy it issued has been waited for.
#include <cuda.h>
#include <float.h>
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"
#include "adsa_select.cuh"
#include "adsa_async.cuh"

namespace adsa {

constexpr int kWTile = 32;                        // rows per tile
constexpr int kWRowBytes = 128;                   // 64 bf16
constexpr int kWTileBytes = kWTile * kWRowBytes;  // one K (or V) tile
constexpr int kWStageBytes = 2 * kWTileBytes;
constexpr int kWMaxDepth = 8;                     // stages per warp

// Per-warp shared memory (offsets from the warp's base)
struct WLayout {
    uint32_t bars, hdr, pt, meta, keys, region, kmask, cmask, wsplit, hist, svec, stages;
    uint32_t meta_words, w_rows;
    uint32_t per_warp;
};

__host__ __device__ inline uint32_t w_align(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline WLayout w_layout(int max_rows, int max_pages, int mask_words, int depth, bool fused)
{
    WLayout L;
    uint32_t off = 0;
    L.bars = off;   off += (kWMaxDepth + 2) * 8;
    L.hdr = off;    off += 16;
    L.pt = off;     off += w_align(max_pages * 4, 16);
    L.meta_words = w_align(max_rows + 8, 4);
    L.meta = off;   off += fused ? 3 * L.meta_words * 4 : 0;            // pos | carried scores | inverse norms
    L.keys = off;   off += fused ? w_align((max_rows + 2) * 8, 16) : 0; // later reused: holes, survivors
    L.region = off; off += fused ? w_align(max_rows + kWTile, 16) : 0;
    L.kmask = off;  off += w_align((mask_words + 1) * 4, 16);
    L.cmask = off;  off += fused ? w_align((mask_words + 1) * 4, 16) : 0;   // retained rows the next step scores
    L.w_rows = w_align(max_rows + kWTile, 32);
    L.wsplit = off; off += fused ? 3 * L.w_rows * 2 : 0;               // bf16 hi | mid | lo of the row weights
    L.hist = off;   off += fused ? 256 * 4 : 0;
    L.svec = off;   off += 64 * 4;
    off = w_align(off, 1024);                                          // the swizzle pattern repeats every 1024 bytes
    L.stages = off; off += depth * kWStageBytes;
    L.per_warp = w_align(off, 1024);
    return L;
}

struct WStepArgs {
    int layer, cur_pos, budget_rows, depth, n_workers;   // n_workers = warps per CTA
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
// D = A * B (accumulator starts at zero)
__device__ __forceinline__ void mma_bf16_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ float ex2(float x)   // 2^x, x <= 0 or -inf here
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * kWRowBytes + ((c ^ (r & 7)) << 4)); }

template <bool FUSED>
__global__ void __launch_bounds__(256, 1)
wstep_kernel(DevCtx c, WStepArgs a, const __grid_constant__ WStepMaps maps)
{
    extern __shared__ __align__(1024) unsigned char smem_all[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int D = a.depth;
    const WLayout L = w_layout(c.max_rows, c.max_pages, c.mask_words, D, FUSED);
    unsigned char *smem = smem_all + (size_t)warp * L.per_warp;
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + L.bars);   // [0..D) tiles, [kWMaxDepth] metadata
    const uint32_t bar_meta = smem_u32(bars + kWMaxDepth);
    const uint32_t stages_u32 = smem_u32(smem + L.stages);
    int32_t *pt_s = reinterpret_cast<int32_t *>(smem + L.pt);
    unsigned long long *sm_keys = reinterpret_cast<unsigned long long *>(smem + L.keys);
    uint8_t *region = smem + L.region;
    uint32_t *kmask = reinterpret_cast<uint32_t *>(smem + L.kmask);
    uint32_t *cmask = reinterpret_cast<uint32_t *>(smem + L.cmask);
    __nv_bfloat16 *wsplit = reinterpret_cast<__nv_bfloat16 *>(smem + L.wsplit);
    int *hist = reinterpret_cast<int *>(smem + L.hist);
    float *svec = reinterpret_cast<float *>(smem + L.svec);
    if (warp >= a.n_workers) return;

    if (lane == 0) {
        for (int s = 0; s < D; ++s) mbar_init(smem_u32(bars + s), 1);
        mbar_init(bar_meta, 1);
        mbar_init_fence();
    }
    {   // zero the ring once: rows a partial tile never receives must hold finite numbers
        uint4 *z = reinterpret_cast<uint4 *>(smem + L.stages);
        for (int i = lane; i < D * kWStageBytes / 16; i += 32) z[i] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const int g = lane >> 2, t = lane & 3;          // MMA fragment coordinates
    const int mi = lane >> 3, lr = lane & 7;        // ldmatrix: matrix index, row within the matrix
    const bool new_cand = FUSED && region_of(c, a.cur_pos, a.cur_pos + 1) == kRegionPrevious;
    // ldmatrix row addresses inside a tile.  Tile rows used by a lane are (multiple of 8) + lr, so the
    // swizzle term is (chunk ^ lr) << 4 and every address is a per-lane base xor a small constant:
    //   K, block nb, elements 0-31:   nb*1024 + k_off        (chunks mi);  elements 32-63: the same ^ 64
    //   V / pass 2, rows 16*a + 8*(mi&1) + lr, chunk 2*b + (mi>>1):   a*2048 + (v_off ^ (b << 5))
    const uint32_t k_off = (uint32_t)(lr * kWRowBytes + ((mi ^ lr) << 4));
    const uint32_t v_off = (uint32_t)((8 * (mi & 1) + lr) * kWRowBytes + (((mi >> 1) ^ lr) << 4));
    const uint32_t *w_role = reinterpret_cast<const uint32_t *>(wsplit + (size_t)(g >= 2 && g <= 4 ? g - 2 : 0) * L.w_rows);
    int spin_limit = kCopySpinLimit;
    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (!mbar_wait_sleepy(bar, parity, spin_limit)) {
            if (lane == 0) set_status(c, ADSA_DEV_COPY_TIMEOUT);
            spin_limit = kCopySpinAfterTimeout;
        }
    };

    uint32_t issued = 0, consumed = 0;   // tiles of this warp since kernel start (stage = count % D)
    int streams_done = 0;
    const int stride = gridDim.x * a.n_workers;
    for (int local = warp * gridDim.x + blockIdx.x; local < c.S; local += stride, ++streams_done) {
        const int sid = a.layer * c.S + local;
        int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
        int n = c.n_live[sid];
        if (n < 0 || n > c.max_rows) { if (lane == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW); n = 0; }
        const int np = (n + c.page_rows - 1) / c.page_rows;
        for (int pg = lane; pg < np; pg += 32) pt_s[pg] = pt[pg];
        const int n_tiles = (n + kWTile - 1) / kWTile;
        const int total = FUSED ? 2 * n_tiles : n_tiles;   // pass 1 tiles, then pass 2 tiles (V only)

        // ---- metadata: aligned interior by bulk copy, ragged ends by plain loads -------------------
        const int32_t *pos_s = nullptr;
        const float *scores_s = nullptr, *inv_s = nullptr;
        if constexpr (FUSED) {
            const void *src[3] = {c.pos + (size_t)sid * c.max_rows, c.scores + (size_t)sid * c.max_rows,
                                  c.inv_norm + (size_t)sid * c.max_rows};
            uint32_t meta_tx = 0;
            const uint32_t *base[3];
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const uint32_t *gp = reinterpret_cast<const uint32_t *>(src[k]);
                uint32_t *d = reinterpret_cast<uint32_t *>(smem + L.meta) + k * L.meta_words;
                const int lead = (int)(((uintptr_t)gp >> 2) & 3);
                const int head = min(n, (4 - lead) & 3);
                const int body = (n - head) & ~3;
                if (lane < head) d[lead + lane] = gp[lane];
                if (lane < n - head - body) d[lead + head + body + lane] = gp[head + body + lane];
                if (lane == 0 && body > 0) {
                    bulk_g2s(smem_u32(d + lead + head), gp + head, (uint32_t)body * 4u, bar_meta);
                    meta_tx += (uint32_t)body * 4u;
                }
                base[k] = d + lead;
            }
            if (lane == 0) mbar_expect_tx(bar_meta, meta_tx);
            pos_s = reinterpret_cast<const int32_t *>(base[0]);
            scores_s = reinterpret_cast<const float *>(base[1]);
            inv_s = reinterpret_cast<const float *>(base[2]);
        }
        __syncwarp();

        // ---- the warp's own copy pipeline ----------------------------------------------------------
        auto issue = [&](int u) {   // lane 0 only: tile u of this stream into the next free stage
            const int stage = issued % D;
            const int pass = u >= n_tiles ? 1 : 0, tl = pass ? u - n_tiles : u;
            const int r0 = tl * kWTile, r1 = min(n, r0 + kWTile);
            const uint32_t kdst = stages_u32 + stage * kWStageBytes, vdst = kdst + kWTileBytes;
            const uint32_t bar = smem_u32(bars + stage);
            mbar_expect_tx(bar, (uint32_t)(r1 - r0) * kWRowBytes * (pass == 0 ? 2u : 1u));
            int r = r0;
            {   // the common case: a whole tile inside one page is one box per pool
                uint32_t pg = __umulhi((uint32_t)r0, c.pr_magic);
                int in = r0 - (int)pg * c.page_rows;
                if (r1 - r0 == kWTile && in + kWTile <= c.page_rows) {
                    int y = pt_s[pg] * c.page_rows + in;
                    if (pass == 0) tma_2d(kdst, &maps.k[5], 0, y, bar);
                    tma_2d(vdst, &maps.v[5], 0, y, bar);
                    r = r1;
                }
            }
            while (r < r1) {   // page pieces, each cut into boxes of 32, 16, 8, 4, 2 or 1 rows
                uint32_t pg = __umulhi((uint32_t)r, c.pr_magic);
                int in = r - (int)pg * c.page_rows;
                int cnt = min(r1 - r, c.page_rows - in);
                int y = pt_s[pg] * c.page_rows + in;
                uint32_t off = (uint32_t)(r - r0) * kWRowBytes;
                r += cnt;
                while (cnt > 0) {
                    int hb = 31 - __clz(cnt);
                    hb = hb > 5 ? 5 : hb;
                    if (pass == 0) tma_2d(kdst + off, &maps.k[hb], 0, y, bar);
                    tma_2d(vdst + off, &maps.v[hb], 0, y, bar);
                    y += 1 << hb; off += (uint32_t)kWRowBytes << hb; cnt -= 1 << hb;
                }
            }
        };
        int next_issue = 0;
        if (lane == 0) {
            for (; next_issue < total && next_issue < D; ++next_issue, ++issued) issue(next_issue);
        }
        next_issue = __shfl_sync(0xffffffffu, next_issue, 0);
        issued = __shfl_sync(0xffffffffu, issued, 0);
        // after a stage has been read (all lanes), lane 0 refills it with the tile `depth` ahead
        auto release_and_refill = [&]() {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (next_issue < total) {
                if (lane == 0) issue(next_issue);
                ++next_issue; ++issued;
            }
        };

        // ---- which rows are attended, and the weights of the rows the next step scores -------------
        int n2 = n, p_next = 0;
        if constexpr (FUSED) {
            wait(bar_meta, streams_done & 1);
            const SelResult sel = warp_select(c, pos_s, scores_s, n, a.cur_pos, a.budget_rows, sm_keys, region, hist);
            n2 = n - (sel.p - sel.K) + 1;
            const int n_pad = n_tiles * kWTile;
            for (int base = 0; base < n_pad; base += 32) {
                const int slot = base + lane;
                const bool kept = slot < n && sel.keeps(region[slot], sm_keys[slot]);
                if (slot < n && (region[slot] & 3) == kRegionInvalid) set_status(c, ADSA_DEV_BAD_POSITION);
                const unsigned bk = __ballot_sync(0xffffffffu, kept);
                const bool cand = kept && (region[slot] & kCandNextBit);
                const unsigned bc = __ballot_sync(0xffffffffu, cand);
                if (lane == 0) { kmask[base >> 5] = bk; cmask[base >> 5] = bc; }
                p_next += __popc(bc);
                // w = 1/|v| for the rows the next step scores, as three bf16 parts (24 bits)
                float w = cand ? inv_s[slot] : 0.f;
                __nv_bfloat16 h = __float2bfloat16_rn(w);
                float r1 = w - __bfloat162float(h);
                __nv_bfloat16 md = __float2bfloat16_rn(r1);
                __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(md));
                wsplit[slot] = h; wsplit[L.w_rows + slot] = md; wsplit[2 * L.w_rows + slot] = lo;
            }
            p_next += new_cand ? 1 : 0;
        } else {
            const uint32_t *gm = c.keep_mask + (size_t)local * c.mask_words;
            for (int w = lane; w < n_tiles; w += 32) {
                uint32_t bits = gm[w];
                int valid = n - w * 32;
                kmask[w] = valid >= 32 ? bits : (bits & ((1u << valid) - 1u));
            }
        }
        __syncwarp();

        // ---- q as the A operand (rows 0-7 = q, rows 8-15 = 0), four k-steps of 16 elements ---------
        uint32_t qa0[4], qa2[4];
        {
            const uint32_t *q2 = reinterpret_cast<const uint32_t *>(a.q + (size_t)local * c.d);   // c.d is even
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                int e0 = 16 * ks + 2 * t, e1 = e0 + 8;
                qa0[ks] = e0 < c.d ? q2[e0 >> 1] : 0u;
                qa2[ks] = e1 < c.d ? q2[e1 >> 1] : 0u;
            }
        }
        // ---- the new row starts the running state: weight 1 in A' row 0, its 1/|v| in row 2 --------
        float m_run, l_run, o_run[8][2];
        {
            float s = 0.f, ss = 0.f;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int xx = 2 * lane + e;
                float qf = xx < c.d ? __bfloat162float(a.q[(size_t)local * c.d + xx]) : 0.f;
                float kf = xx < c.d ? __bfloat162float(a.k_new[(size_t)local * c.d + xx]) : 0.f;
                float vf = xx < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + xx]) : 0.f;
                s = fmaf(qf, kf, s);
                ss = fmaf(vf, vf, ss);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, o);
                ss += __shfl_xor_sync(0xffffffffu, ss, o);
            }
            const float inv_new = new_cand ? 1.0f / fmaxf(sqrtf(ss), kNormEps) : 0.f;
            m_run = s * c.scale_log2e;
            l_run = t == 0 ? 1.f : 0.f;   // summed over the four t lanes at the end
            const float wrow = g == 0 ? 1.f : g == 2 ? inv_new : 0.f;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    int xx = 8 * nb + 2 * t + e;
                    float vf = xx < c.d ? __bfloat162float(a.v_new[(size_t)local * c.d + xx]) : 0.f;
                    o_run[nb][e] = wrow * vf;
                }
            }
        }

        // ---- pass 1 --------------------------------------------------------------------------------
        for (int tl = 0; tl < n_tiles; ++tl, ++consumed) {
            const int stage = consumed % D;
            wait(smem_u32(bars + stage), (consumed / D) & 1);
            const uint32_t kb = stages_u32 + stage * kWStageBytes, vb = kb + kWTileBytes;
            const int r0 = tl * kWTile;
            const uint32_t kw = kmask[tl] >> (2 * t);   // bit 8*nb + e: row 8*nb + 2t + e is retained
            float sc[4][4];
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {   // S = q.K^T, blocks of 8 rows
                uint32_t kf0[4], kf1[4];
                ldsm_x4(kb + nb * 1024 + k_off, kf0);          // elements 0-31 of the 8 rows
                ldsm_x4(kb + nb * 1024 + (k_off ^ 64u), kf1);  // elements 32-63
                mma_bf16_z(sc[nb], qa0[0], 0u, qa2[0], 0u, kf0[0], kf0[1]);
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
                    bool kept = (kw >> (8 * nb + e)) & 1u;
                    x[nb][e] = kept ? sc[nb][e] * c.scale_log2e : -INFINITY;
                    mx = fmaxf(mx, x[nb][e]);
                }
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run, mx);
            const float corr = ex2(m_run - m_new);
            m_run = m_new;
            float psum = 0.f;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) { x[nb][e] = ex2(x[nb][e] - m_new); psum += x[nb][e]; }
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
            for (int nbp = 0; nbp < 4; ++nbp) {
                uint32_t vf[4];
                ldsm_x4_t(vb + (v_off ^ (uint32_t)(nbp << 5)), vf);
                mma_bf16_z(ot[2 * nbp], pa0[0], 0u, pa2[0], 0u, vf[0], vf[1]);
                mma_bf16_z(ot[2 * nbp + 1], pa0[0], 0u, pa2[0], 0u, vf[2], vf[3]);
            }
#pragma unroll
            for (int nbp = 0; nbp < 4; ++nbp) {
                uint32_t vf[4];
                ldsm_x4_t(vb + 2048 + (v_off ^ (uint32_t)(nbp << 5)), vf);
                mma_bf16(ot[2 * nbp], pa0[1], 0u, pa2[1], 0u, vf[0], vf[1]);
                mma_bf16(ot[2 * nbp + 1], pa0[1], 0u, pa2[1], 0u, vf[2], vf[3]);
            }
            release_and_refill();
            const float corr_row = g < 2 ? corr : 1.0f;     // the weight sums are not softmax-scaled
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
                o_run[nb][0] = fmaf(o_run[nb][0], corr_row, ot[nb][0]);
                o_run[nb][1] = fmaf(o_run[nb][1], corr_row, ot[nb][1]);
            }
        }

        // ---- softmax.V = rows 0 + 1 over l; s = rows 2 + 3 + 4 -------------------------------------
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        const float inv_l = 1.0f / l_run;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            float v0 = o_run[nb][0], v1 = o_run[nb][1];
            float a0 = __shfl_down_sync(0xffffffffu, v0, 4), a1 = __shfl_down_sync(0xffffffffu, v1, 4);
            float b0 = __shfl_down_sync(0xffffffffu, v0, 8), b1 = __shfl_down_sync(0xffffffffu, v1, 8);
            const int xx = 8 * nb + 2 * t;
            if (g == 0 && xx < c.d) {
                float o0 = (v0 + a0) * inv_l, o1 = (v1 + a1) * inv_l;
                if (a.out_f32) {
                    a.out_f32[(size_t)local * c.d + xx] = o0;
                    if (xx + 1 < c.d) a.out_f32[(size_t)local * c.d + xx + 1] = o1;
                }
                if (a.out_bf16)
                    *reinterpret_cast<uint32_t *>(a.out_bf16 + (size_t)local * c.d + xx) = pack_bf16(o0, o1);
            }
            if (g == 2) { svec[xx] = (v0 + a0) + b0; svec[xx + 1] = (v1 + a1) + b1; }
        }
        __syncwarp();

        if constexpr (FUSED) {
            // ---- Section 4.2 bookkeeping: holes below the new length, survivors above it ----------
            int32_t *holes = reinterpret_cast<int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;   // keys are dead now
            int nh = 0, ns = 0;
            const int top = max(n, n2);
            for (int base = 0; base < top; base += 32) {
                const int s = base + lane;
                const bool kept = s < n && ((kmask[s >> 5] >> (s & 31)) & 1u);
                const bool is_hole = s < n2 && !kept, is_surv = s >= n2 && s < n && kept;
                const unsigned bh = __ballot_sync(0xffffffffu, is_hole), bs = __ballot_sync(0xffffffffu, is_surv);
                const unsigned below = (1u << lane) - 1u;
                if (is_hole) holes[nh + __popc(bh & below)] = s;
                if (is_surv) surv[ns + __popc(bs & below)] = s;
                nh += __popc(bh); ns += __popc(bs);
            }
            __syncwarp();
            const int have = (n + c.page_rows - 1) / c.page_rows, need = (n2 + c.page_rows - 1) / c.page_rows;
            int okay = 1;
            if (lane == 0) {
                if (nh != ns + 1) { set_status(c, ADSA_DEV_BAD_EVICT); okay = 0; }
                else if (n2 > c.max_rows) { set_status(c, ADSA_DEV_ROW_OVERFLOW); okay = 0; }
                else if (need > have && !resize_pages(c, pt, have, need)) okay = 0;
            }
            okay = __shfl_sync(0xffffffffu, okay, 0);
            __syncwarp();   // lane 0 may have written a page-table entry the others are about to read
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

            // ---- pass 2: dot_i = v_i . s, S_i = (dot_i/|v_i| - u_i.u_i) / (p' - 1), at the row's new slot ----
            for (int tl = 0; tl < n_tiles; ++tl, ++consumed) {
                const int stage = consumed % D;
                wait(smem_u32(bars + stage), (consumed / D) & 1);
                const uint32_t vb = stages_u32 + stage * kWStageBytes + kWTileBytes;
                const unsigned char *vtile = smem + L.stages + stage * kWStageBytes + kWTileBytes;
                const int r0 = tl * kWTile;
                const uint32_t cw = okay ? cmask[tl] : 0u;
                float dt[2][4];
#pragma unroll
                for (int mbk = 0; mbk < 2; ++mbk) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        uint32_t af[4];
                        ldsm_x4(vb + mbk * 2048 + (v_off ^ (uint32_t)(ks << 5)), af);
                        if (ks == 0) mma_bf16_z(dt[mbk], af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                        else mma_bf16(dt[mbk], af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                    }
                }
#pragma unroll
                for (int mbk = 0; mbk < 2; ++mbk) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {   // rows 16*mbk + 8*hh + g: columns 0, 1 in lane t = 0, column 2 in t = 1
                        float lo = __shfl_down_sync(0xffffffffu, dt[mbk][2 * hh], 1);
                        const int row = r0 + 16 * mbk + 8 * hh + g;
                        const bool want = t == 0 && ((cw >> (16 * mbk + 8 * hh + g)) & 1u);
                        if (want) {
                            float dot = (dt[mbk][2 * hh] + dt[mbk][2 * hh + 1]) + lo;
                            float inv = inv_s[row], self = 1.0f;
                            if (inv >= 1.0f / kNormEps) {   // |v| was clamped: u.u is not 1, take it from the row
                                float ss = 0.f;
                                for (int ch = 0; ch < 8; ++ch) {
                                    float f[8];
                                    unpack8(*reinterpret_cast<const uint4 *>(vtile + swz(row - r0, ch)), f);
                                    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
                                }
                                self = inv * inv * ss;
                            }
                            int dst = row;
                            if (row >= n2) {   // a survivor: it moves into the hole of the same rank
                                int lo_i = 0, hi_i = ns - 1;
                                while (lo_i < hi_i) { int mid = (lo_i + hi_i) >> 1; if (surv[mid] < row) lo_i = mid + 1; else hi_i = mid; }
                                dst = holes[lo_i];
                            }
                            scores[dst] = p_next > 1 ? (inv * dot - self) / denom + 0.0f : 0.0f;
                        }
                    }
                }
                release_and_refill();
            }

            // ---- the update itself ---------------------------------------------------------------
            if (okay) {
                for (int i = 0; i < ns; ++i) {   // survivors move down: 8 + 8 pieces of 16 bytes
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
                if (new_cand) {   // the new row's own score for the next step
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
                write_row(c, pt, sid, holes[ns], a.k_new + (size_t)local * c.d, a.v_new + (size_t)local * c.d, a.cur_pos);
                if (lane == 0) {
                    if (need < have) resize_pages(c, pt, have, need);
                    c.n_live[sid] = n2;
                }
            }
        }
        __syncwarp();   // the stream's shared buffers are free for the next one
    }
}

// ---- host side ------------------------------------------------------------
bool wstep_supported(const DevCtx &c) { return c.row_stride == 64 && c.d % 2 == 0; }

// Tensor maps of both pools for boxes of 1, 2, 4, .. 32 rows (128-byte swizzle).  The encoder is
// cuTensorMapEncodeTiled, looked up at run time so that the library links cudart only.
int build_wstep_maps(const DevCtx &c, WStepMaps *out)
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
    if (dims[1] > (1ull << 31)) return -1;
    const cuuint64_t strides[1] = {kWRowBytes};
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

cudaError_t configure_wstep_kernel(const DevCtx &c)
{
    (void)c;
    cudaError_t e = cudaFuncSetAttribute(wstep_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(wstep_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmemLimit);
}

// Workers (warps) per CTA and ring depth per worker: enough workers that every stream of the layer
// has one if possible, at most 8, as many as fit with a ring of at least 2 (preferably 3+) stages.
WStepPlan plan_wstep(const DevCtx &c, bool fused, int sm_count, int max_depth)
{
    WStepPlan p = {};
    if (!wstep_supported(c)) return p;
    int want = (c.S + sm_count - 1) / sm_count;
    want = want < 1 ? 1 : want > 8 ? 8 : want;
    int cap = max_depth > 0 && max_depth < kWMaxDepth ? max_depth : kWMaxDepth;
    for (int w = want; w >= 1; --w) {
        const uint32_t fixed = w_layout(c.max_rows, c.max_pages, c.mask_words, 0, fused).per_warp;
        if ((uint64_t)fixed * w >= (uint64_t)kPSmemLimit) continue;
        int depth = (int)((kPSmemLimit - 1024) / w - fixed) / kWStageBytes;
        depth = depth > cap ? cap : depth;
        if (depth < 2 || (depth < 3 && w > 1)) continue;
        WLayout L = w_layout(c.max_rows, c.max_pages, c.mask_words, depth, fused);
        if ((uint64_t)L.per_warp * w + 1024 > (uint64_t)kPSmemLimit) { if (--depth < 2) continue; L = w_layout(c.max_rows, c.max_pages, c.mask_words, depth, fused); }
        p.n_workers = w; p.depth = depth; p.smem_bytes = (size_t)L.per_warp * w;
        int ctas = (c.S + w - 1) / w;
        p.grid = ctas < sm_count ? ctas : sm_count;
        return p;
    }
    return p;
}

cudaError_t launch_wstep(const DevCtx &c, const WStepPlan &plan, const WStepMaps &maps, bool fused, int layer, int cur_pos,
                         int budget_rows, const void *q, const void *k_new, const void *v_new, void *out_bf16,
                         float *out_f32, cudaStream_t st)
{
    WStepArgs a;
    a.layer = layer; a.cur_pos = cur_pos; a.budget_rows = budget_rows; a.depth = plan.depth; a.n_workers = plan.n_workers;
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    const int threads = plan.n_workers * 32;
    if (fused) wstep_kernel<true><<<plan.grid, threads, plan.smem_bytes, st>>>(c, a, maps);
    else wstep_kernel<false><<<plan.grid, threads, plan.smem_bytes, st>>>(c, a, maps);
    return cudaGetLastError();
}

}  // namespace adsa
