// The warp-per-stream kernel with tensor-core arithmetic, for pools whose rows are
// 64 elements (128 bytes) wide.  This is the kernel the benchmark's layer-step runs.
//
// Why a few warps per stream.  A layer-step of one stream is a chain of short,
// dependent phases (selection, attention sweep, reduction, score sweep, update).
// Spread over a whole CTA each phase ends in a CTA barrier and the SM idles on
// latency; measured, a CTA-wide version spent 27 us per stream.  Here a stream
// belongs to a small group of warps (1 to 4, chosen so that the SM's streams fill
// its warp slots): the tiles of the stream are dealt round-robin to the warps of the
// group, each warp keeps its own ring of tiles in shared memory and issues its own
// TMA copies, and the group meets only three times per stream (selection partials,
// softmax partials, before the update) on a named barrier.  Latency is hidden the
// way GPUs hide it best, by the other warps of the SM being elsewhere in their chains.
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
// Pass 1, per tile:  S = K.q  (A = 16 rows of K via ldmatrix, B = q in every column);
//   P = exp2(S*scale - m), split into bf16 hi + lo so the product keeps fp32-like
//   accuracy;  O^T_tile = V^T.B' (A = V^T via transposing ldmatrix) with B' columns
//   {P_hi, P_lo, w_hi, w_mid, w_lo}, where w_j = 1/|v_j| for the rows the next step will
//   score and 0 otherwise: columns 0-1 of the result accumulate softmax.V, columns 2-4
//   accumulate s = sum of normalised rows.  This orientation puts the long dimensions
//   (rows, head elements) on M, so a 32-row tile costs 16 MMAs instead of 32; on this
//   part the legacy mma.sync pipe is slow enough for that to matter (measured).
//   Each tile's product starts from zero and is folded into fp32 running sums with
//   round-to-nearest FMAs, so tensor-core accumulation rounding never compounds
//   beyond 32 rows.
// Next step's scores (fused).  Eq. 1-2 for the next step, S_i = (dot_i/|v_i| - u_i.u_i) / (p' - 1) with
//   dot_i = v_i . s, s = the sum of the normalised rows of the next step's previous region
//   (u_i.u_i = 1 unless |v_i| was clamped, in which case it is computed from the row).  s itself is
//   carried from step to step.  In the steady state the next previous region is this one minus the
//   evicted row, so s' = s - u_e is known once the selection has named e, and every pass-1 tile also
//   yields the scores of its rows: 4 more MMAs per 16 rows, s' split into three bf16 parts as B
//   columns 0-2 (single sweep).  Otherwise (nothing carried in, rows leaving the local window, more
//   than one eviction) a second sweep over V, which comes out of L2, uses the s just accumulated.
// Then the Section 4.2 update.  All rows of a stream are copied, retained or not
// (one row per step is not); the rows of a partial last tile that the copy does not
// write are cleared first, so that a zero weight never meets a NaN pattern.
//
// Launch overlap.  The kernel is launched with programmatic stream serialization.  What touches no
// global state (barrier set-up, launch-wide constants, L2 prefetch hints for the first stream's
// metadata and first tiles) runs ahead of griddepcontrol.wait, i.e. under the tail of the kernel
// before it in the stream; every load and store whose value matters comes after the wait.
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

// The kernel is compiled for three tile layouts (template parameters RS = elements per tile row in shared memory,
// TR = rows per ring stage).  The two swizzled ones also serve pools whose rows are narrower than the tile's: the
// tensor copies read the pool's rows and fill the rest of a tile row with zeros.
//   RS = 64,  TR = 32   128-byte rows written with the 128-byte swizzle; a stage is a whole 32-row block;
//   RS = 104, TR = 16   208-byte rows (head_dim 97 .. 104) written as they lie: a pitch of 208 bytes puts the eight
//                       rows of an ldmatrix on eight different bank groups without any swizzle; a stage is half a
//                       block (6.5 KB instead of 13 KB), so that shared memory still holds rings for ten warps.
//   RS = 128, TR = 16   256-byte rows as two 128-byte halves, each a swizzled tile of its own (elements 0-63 of
//                       every row, then elements 64-127), written by two tensor copies per pool; 8 KB per stage.
// Rows are always dealt to the warps of a group in 32-row blocks (one word of every row mask).
constexpr int kWTile = 32;                        // rows per block
constexpr int kWMaxDepth = 8;                     // stages per warp
constexpr int kWMaxGroupWarps = 4;                // warps that may share a stream
constexpr int kWWideMaxWarps = 10;                // warps per CTA of the 104-element instantiation (registers)
__host__ __device__ constexpr int w_stage_bytes(int rs, int tr) { return 2 * tr * rs * 2; }          // a K tile and a V tile
__host__ __device__ constexpr int w_sets(int rs) { return (rs + 63) / 64; }                           // 64-element sets of a row (two elements per lane)
__host__ __device__ constexpr int w_part_floats(int rs) { return 128 * w_sets(rs) + 8; }             // one warp's partial state: acc | s | m, l, flags

// ---- PTX wrappers ---------------------------------------------------------
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
// D += A(16x16, row) * B(16x8, col), bf16 in, fp32 accumulate
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D = A * B (accumulator starts at zero)
__device__ __forceinline__ void mma_bf16_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
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
// part `role` (0 hi, 1 mid, 2 lo) of the three-way bf16 split of the pair (w0, w1): hi = bf16(w), mid = bf16(w - hi),
// lo = bf16(w - hi - mid), 24 bits in all
__device__ __forceinline__ uint32_t split_part(float w0, float w1, int role)
{
    const uint32_t h = pack_bf16(w0, w1);
    const float r0 = w0 - bf16_lo(h), r1 = w1 - bf16_hi(h);
    const uint32_t m = pack_bf16(r0, r1);
    const uint32_t l = pack_bf16(r0 - bf16_lo(m), r1 - bf16_hi(m));
    return role == 0 ? h : role == 1 ? m : l;
}
// byte offset of 16-byte chunk c of row r inside a tile written with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// Shared memory of one group (the G warps that share a stream): a fixed part, then one ring per warp.
struct WLayout {
    uint32_t bars, hdr, pt, inv, prevm, candm, kmask, cmask, hist, part, rings;
    uint32_t inv_words, mwords;
    uint32_t ring_bytes;    // one warp's ring
    uint32_t per_group;
};

__host__ __device__ inline uint32_t w_align(uint32_t x, uint32_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline WLayout w_layout(int max_rows, int max_pages, int mask_words, int depth, int G, bool fused, int rs, int tr)
{
    WLayout L;
    uint32_t off = 0;
    L.bars = off;   off += (kWMaxGroupWarps * kWMaxDepth + 2) * 8;       // tile barriers per warp, then the metadata barrier
    L.hdr = off;    off += kWMaxGroupWarps * 32 + 32 + kWMaxGroupWarps * 16 + kWMaxGroupWarps * 8 + 16;   // per-warp selection partials, the threshold, per-warp highest carried scores, per-warp look at the next launch's stream, 16 zero bytes
    L.pt = off;     off += w_align(max_pages * 4, 16);
    L.inv_words = w_align(max_rows + 8, 4);
    L.inv = off;    off += fused ? L.inv_words * 4 : 0;                   // inverse norms by slot
    L.mwords = mask_words + 1;
    L.prevm = off;  off += fused ? w_align(L.mwords * 4, 16) : 0;         // rows of the previous region
    L.candm = off;  off += fused ? w_align(L.mwords * 4, 16) : 0;         // rows in the previous region of the next step
    L.kmask = off;  off += w_align(L.mwords * 4, 16);                     // retained rows
    L.cmask = off;  off += fused ? w_align(L.mwords * 4, 16) : 0;         // retained rows the next step scores
    L.part = off;   off += (G * w_part_floats(rs) * 4 > 1024 ? G * w_part_floats(rs) * 4 : 1024);   // per warp: acc | s | m, l, flags (at least the histogram's 1 KB)
    L.hist = L.part;                                                      // radix histogram: used before any partial state exists
    off = w_align(off, 1024);                                             // the swizzle pattern repeats every 1024 bytes
    L.rings = off;
    L.ring_bytes = depth * w_stage_bytes(rs, tr);
    L.per_group = off + G * L.ring_bytes;
    return L;
}

struct WStepArgs {
    int layer, cur_pos, budget_rows, depth;
    int n_run;                   // consecutive layers served by this launch, starting at `layer` (q, k_new, v_new, out: [n_run][S][d])
    int group_warps, n_groups;   // warps per stream, groups per CTA
    int l2_ahead;                // tiles per warp asked into L2 beyond the ring
    uint32_t g_magic;            // x / group_warps == __umulhi(x, g_magic) for the small x used here (group_warps > 1)
    int have_svec;               // the sum of normalised rows of this step's previous region was carried in
    int use_note;                // ... and with it the previous fused step's note (DevCtx::carry, cand_mask): which
                                 // slots hold this step's previous region and how many; it may stand in for the classification
    int early_state;             // the cache state of this layer is not being written by the kernel ahead in the stream
    int next_layer, next_tiles;  // the layer the next launch is expected to serve (-1 = unknown) and how many of its first
                                 // 32-row tiles per warp this launch asks into L2 once its own sweep is over
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out_bf16;
    float *out_f32;
    unsigned long long *scratch; // [grid][n_groups][2 * max_rows + 4] words of 8 bytes: keys, compaction lists
    const int *in_ready;         // null, or one word per layer of the context: layer l's q, k_new and v_new have landed (a copy
    int in_epoch;                // engine is still writing them when the launch starts) once in_ready[l] - in_epoch >= 0
};

struct WSelPartial {      // what one warp of a group found in its share of the rows (32 bytes)
    unsigned long long max_key;
    int max_slot, n_pre, n_loc, p, n_cand, n_cand_not_prev;
};

template <bool FUSED, int MAXW, int RS, int TR>
__global__ void __launch_bounds__(MAXW * 32, 1)
wstep_kernel(DevCtx c, WStepArgs a, const __grid_constant__ WStepMaps maps)
{
    constexpr int kWRowBytes = RS * 2;                 // bytes of a pool row
    constexpr int kWTileBytes = TR * kWRowBytes;       // one K (or V) tile of a stage
    constexpr int kWStageBytes = 2 * kWTileBytes;
    constexpr int KS = (RS + 15) / 16;                 // 16-element steps over a row: k-steps of S = K.q and of the score product, M blocks of O^T
    constexpr int NJ = w_sets(RS);                     // a lane holds elements 64*j + 2*lane, + 1 of a row, j < NJ
    constexpr int NH = kWTile / TR, MB = TR / 16;      // stages per 32-row block, 16-row MMA blocks per stage
    constexpr bool SWZ = RS % 64 == 0;                 // tiles written with the 128-byte swizzle, one sub-tile per 64 elements of a row
    constexpr int NSEG = SWZ ? RS / 64 : 1;            // sub-tiles of a K (or V) tile
    constexpr int PITCH = SWZ ? 128 : kWRowBytes;      // bytes from row to row inside a sub-tile
    constexpr int SEGB = TR * 128;                     // bytes of a swizzled sub-tile
    constexpr bool RAGGED = RS % 16 != 0;              // the last 16-element step has only its first 8 elements
    // RS is the row width of the tiles in shared memory.  The swizzled layouts also serve narrower pool rows (any
    // stride up to RS elements): the tensor copies fill what lies beyond a pool row with zeros.  The plain layout
    // is the pool's rows as they lie (row stride = RS).
    const int g_rs = SWZ ? c.row_stride : RS;          // elements per pool row
    constexpr int kWPart = w_part_floats(RS);
    constexpr bool SPLIT = KS > 4;                     // two accumulation chains per K.q and V.s product
    extern __shared__ __align__(1024) unsigned char smem_all[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = a.group_warps, D = a.depth;
    auto div_g = [&](int x) { return G == 1 ? x : (int)__umulhi((uint32_t)x, a.g_magic); };   // x / G without a division
    const int gi = div_g(warp), rk = warp - gi * G;      // group in the CTA, rank in the group
    const WLayout L = w_layout(c.max_rows, c.max_pages, c.mask_words, D, G, FUSED, RS, TR);
    unsigned char *smem = smem_all + (size_t)gi * L.per_group;
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem + L.bars) + rk * kWMaxDepth;
    const uint32_t bar_meta = smem_u32(reinterpret_cast<unsigned long long *>(smem + L.bars) + kWMaxGroupWarps * kWMaxDepth);
    unsigned char *ring = smem + L.rings + (size_t)rk * L.ring_bytes;
    const uint32_t stages_u32 = smem_u32(ring);
    WSelPartial *sel_part = reinterpret_cast<WSelPartial *>(smem + L.hdr);
    unsigned long long *sel_thr = reinterpret_cast<unsigned long long *>(smem + L.hdr + kWMaxGroupWarps * 32);
    int32_t *pt_s = reinterpret_cast<int32_t *>(smem + L.pt);
    // Selection keys (any K) and the compaction lists (several evictions at once) are needed on rare steps only:
    // they live in global memory, a slice per group of every CTA (same-SM traffic, served by L1/L2), so that shared
    // memory holds more streams.
    unsigned long long *sm_keys = a.scratch + ((size_t)blockIdx.x * a.n_groups + gi) * (size_t)(2 * c.max_rows + 4);
    uint32_t *prevm = reinterpret_cast<uint32_t *>(smem + L.prevm);
    uint32_t *candm = reinterpret_cast<uint32_t *>(smem + L.candm);
    uint32_t *kmask = reinterpret_cast<uint32_t *>(smem + L.kmask);
    uint32_t *cmask = reinterpret_cast<uint32_t *>(smem + L.cmask);
    int *hist = reinterpret_cast<int *>(smem + L.hist);
    float *part = reinterpret_cast<float *>(smem + L.part);

    const uint32_t zero_u32 = smem_u32(smem + L.hdr + kWMaxGroupWarps * 32 + 32 + kWMaxGroupWarps * 16 + kWMaxGroupWarps * 8);
    if (lane == 0) {
        for (int s = 0; s < D; ++s) mbar_init(smem_u32(bars + s), 1);
        if (rk == 0) {
            mbar_init(bar_meta, 1);
            *reinterpret_cast<uint4 *>(smem + L.hdr + kWMaxGroupWarps * 32 + 32 + kWMaxGroupWarps * 16 + kWMaxGroupWarps * 8) = make_uint4(0u, 0u, 0u, 0u);
        }
        mbar_init_fence();
    }
    // launch-wide constants (integer divisions among them) come before the dependency wait as well
    auto group_sync = [&]() {
        if (G == 1) __syncwarp();
        else asm volatile("bar.sync %0, %1;" ::"r"(1 + gi), "r"(32 * G) : "memory");
    };

    const int g = lane >> 2, t = lane & 3;          // MMA fragment coordinates
    const int mi = lane >> 3, lr = lane & 7;        // ldmatrix: matrix index, row within the matrix
    const bool new_cand = FUSED && region_of(c, a.cur_pos, a.cur_pos + 1) == kRegionPrevious;
    // ldmatrix addresses inside a K or V tile, for 16-row block `blk` of the tile and 16-element step `b` of the row:
    //   rows as the A operand: matrix mi holds rows 16*blk + 8*(mi&1) + lr, 16-byte chunk 2*b + (mi>>1)
    //   V^T (transposing loads): matrix mi holds rows 16*blk + 8*(mi>>1) + lr, chunk 2*b + (mi&1)
    // Swizzled tiles: the rows a lane uses are (multiple of 8) + lr, so the swizzle term is (chunk ^ lr) << 4 and the
    // address is a per-lane base xor (b << 5).  Plain tiles: base + 32*b.  When the row ends in the middle of the last
    // step, the lanes whose chunk lies beyond it read 16 zero bytes instead.
    const uint32_t v_off = SWZ ? (uint32_t)((8 * (mi & 1) + lr) * PITCH + (((mi >> 1) ^ lr) << 4))
                               : (uint32_t)((8 * (mi & 1) + lr) * PITCH + ((mi >> 1) << 4));
    const uint32_t vt_off = SWZ ? (uint32_t)((8 * (mi >> 1) + lr) * PITCH + (((mi & 1) ^ lr) << 4))
                                : (uint32_t)((8 * (mi >> 1) + lr) * PITCH + ((mi & 1) << 4));
    // (swizzled tiles: step b lies in sub-tile b / 4, at chunks 2 * (b % 4), + 1 of its 128-byte rows)
    auto a_addr = [&](uint32_t tile, int blk, int b) -> uint32_t {
        if (RAGGED && b == KS - 1 && (mi >> 1)) return zero_u32;
        return tile + blk * 16 * PITCH + (SWZ ? (uint32_t)((b >> 2) * SEGB) + (v_off ^ (uint32_t)((b & 3) << 5)) : v_off + (uint32_t)(b << 5));
    };
    auto t_addr = [&](uint32_t tile, int blk, int b) -> uint32_t {
        if (RAGGED && b == KS - 1 && (mi & 1)) return zero_u32;
        return tile + blk * 16 * PITCH + (SWZ ? (uint32_t)((b >> 2) * SEGB) + (vt_off ^ (uint32_t)((b & 3) << 5)) : vt_off + (uint32_t)(b << 5));
    };
    // byte offset of 16-byte chunk ch of row r inside a tile
    auto chunk_off = [&](int r, int ch) -> uint32_t {
        return SWZ ? (uint32_t)((ch >> 3) * SEGB) + swz(r, ch & 7) : (uint32_t)(r * kWRowBytes + (ch << 4));
    };
    // one L2 hint per 128-byte line of a pool row
    auto hint_row = [&](const __nv_bfloat16 *row) {
        const int row_bytes = g_rs * 2;
#pragma unroll
        for (int o = 0; o < kWRowBytes; o += 128)
            if (o < row_bytes) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(row) + o));
        if (row_bytes % 128 != 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(row) + row_bytes - 16));
    };
    const RegionCut cut_now = region_cut(c, a.cur_pos), cut_next = region_cut(c, a.cur_pos + 1);
    // the local window does not move between this step and the next, and the new row stays inside it: the next
    // step's previous region is this one's minus whatever is evicted
    const bool steady_cut = FUSED && cut_next.lo == cut_now.lo && !new_cand;
    {
        // The first stream's metadata is asked into L2 now.  A prefetch changes no state that a program can
        // see, so it may run before the kernel launched ahead of this one has completed; the loads after
        // the wait below then find their lines (and their address translations) close by.
        const int local0 = gi * gridDim.x + blockIdx.x;
        if (local0 < c.S * a.n_run && gi < a.n_groups) {
            const int sid0 = a.layer * c.S + local0;
            auto prefetch_span = [&](const void *ptr, size_t bytes) {
                const char *b = reinterpret_cast<const char *>(ptr);
                for (size_t off = (size_t)(rk * 32 + lane) * 128; off < bytes; off += (size_t)G * 32 * 128)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(b + off));
            };
            if (rk == 0 && lane < 3) {
                const __nv_bfloat16 *row = (lane == 0 ? a.q : lane == 1 ? a.k_new : a.v_new) + (size_t)local0 * c.d;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
            }
            if (a.early_state) {
                // the state is read for real right away (see dep_wait below): only the inputs need hints
                if constexpr (!FUSED) prefetch_span(c.keep_mask + (size_t)sid0 * c.mask_words, (size_t)c.mask_words * 4);
            } else {
            if (rk == 0 && lane == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(c.n_live + sid0));
            prefetch_span(c.page_table + (size_t)sid0 * c.max_pages, (size_t)c.max_pages * 4);
            if constexpr (FUSED) {
                prefetch_span(c.pos + (size_t)sid0 * c.max_rows, (size_t)c.max_rows * 4);
                prefetch_span(c.scores + (size_t)sid0 * c.max_rows, (size_t)c.max_rows * 4);
                prefetch_span(c.inv_norm + (size_t)sid0 * c.max_rows, (size_t)c.max_rows * 4);
                if (a.have_svec) prefetch_span(c.svec + (size_t)sid0 * 256 + (a.cur_pos & 1) * 128, 256);
            } else {
                prefetch_span(c.keep_mask + (size_t)sid0 * c.mask_words, (size_t)c.mask_words * 4);
            }
            {
                // The rows of the first tiles, too, located through a racy look at the row count and the
                // page table (read past L1, used for nothing but these hints, and range-checked: a stale
                // value costs a useless prefetch).
                const int n0 = __ldcg(c.n_live + sid0);
                const int32_t *pt0 = c.page_table + (size_t)sid0 * c.max_pages;
                for (int u = 0; u < (D + NH - 1) / NH + (FUSED ? a.l2_ahead : 0); ++u) {   // the blocks the ring will hold, and those asked ahead
                    const int row = (rk + u * G) * kWTile + lane;
                    if (row < n0 && row < c.max_rows) {
                        const uint32_t pg = __umulhi((uint32_t)row, c.pr_magic);
                        const int page = __ldcg(pt0 + pg);
                        if (page >= 0 && page < c.n_pages) {
                            const size_t off = ((size_t)page * c.page_rows + ((uint32_t)row - pg * (uint32_t)c.page_rows)) * (size_t)c.row_stride;
                            hint_row(c.k_pool + off);
                            hint_row(c.v_pool + off);
                        }
                    }
                }
            }
            }
        }
    }
    __syncthreads();   // the only CTA-wide barrier: every warp is still here
    // Programmatic dependent launch: everything above read no value from global memory, so it may run
    // while the kernel launched before this one is still finishing.  That kernel's writes are needed from
    // dep_wait() on.  Normally that is here.  When the host knows that the kernel ahead does not write this
    // layer's cache state (it served another layer; only the kernel directly ahead can still be running,
    // because every kernel of this library waits for its predecessor before it lets its successor start),
    // the state is read, the first tiles are requested and the whole selection is made first (all of it
    // shared-memory work on the cache state; nothing is written to global memory), and the wait comes
    // just before the caller's inputs (q, the new row, the keep mask) are touched.  After its own
    // wait a grid lets the next kernel in the stream be scheduled onto the SMs its CTAs leave.
    bool waited = false;
    auto dep_wait = [&]() {
        if (!waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            waited = true;
        }
    };
    if (!a.early_state) dep_wait();
    int spin_limit = kCopySpinLimit;
    int in_spin = kInputSpinLimit;   // polls of the inputs-have-landed word before giving up
    auto wait = [&](uint32_t bar, uint32_t parity) {
        if (!mbar_wait_sleepy(bar, parity, spin_limit)) {
            if (lane == 0) set_status(c, ADSA_DEV_COPY_TIMEOUT);
            spin_limit = kCopySpinAfterTimeout;
        }
    };

    // The warp's ring positions, kept without divisions: stage to fill next, stage to read next and the
    // parity of the barrier phase that read waits for (it flips each time the ring wraps).
    int i_stage = 0, c_stage = 0;
    uint32_t c_par = 0;
    int streams_done = 0;
    // `local` counts the streams of this launch: those of layer a.layer first, then of the layers after it
    // (the caller's tensors and the per-stream state are laid out in that order)
    const int stride = gridDim.x * a.n_groups, n_local = c.S * a.n_run;
    for (int local = gi * gridDim.x + blockIdx.x; local < n_local; local += stride, ++streams_done) {
        const int sid = a.layer * c.S + local;
        int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
        const float *inv_g = c.inv_norm + (size_t)sid * c.max_rows;
        // ---- everything that only needs addresses is requested first --------------------------------
        int n = c.n_live[sid];
        // the previous fused step's note for this one: {valid, rows in the previous region, flags}, and this lane's
        // word of the mask of those rows by slot (32-row block rk + lane * G)
        int4 note = make_int4(0, 0, 0, 0);
        uint32_t cand_w = 0u;
        const bool try_fast = FUSED && a.use_note && steady_cut;
        if (try_fast) {
            note = *reinterpret_cast<const int4 *>(c.carry + (size_t)sid * 4);
            if (rk + lane * G < c.mask_words) cand_w = c.cand_mask[(size_t)sid * c.mask_words + rk + lane * G];
        }
        for (int pg = lane; pg < c.max_pages; pg += 32) pt_s[pg] = pt[pg];   // every warp of the group writes the same values
        // A look at the same stream of the layer the next launch will serve (its row count and first page): used for
        // nothing but L2 hints after the sweep, range-checked, so a stale value costs a useless prefetch.
        int *const nxt = reinterpret_cast<int *>(smem + L.hdr + kWMaxGroupWarps * 32 + 32 + kWMaxGroupWarps * 16) + 2 * rk;
        // (one layer per launch: the same stream of the next layer; several: the stream this group serves next)
        const int sid2 = a.n_run == 1 ? (a.next_layer >= 0 ? a.next_layer * c.S + local : -1)
                                      : (local + stride < n_local ? sid + stride : -1);
        if (sid2 >= 0 && a.next_tiles > 0 && lane == 0) {
            nxt[0] = __ldcg(c.n_live + sid2);
            nxt[1] = __ldcg(c.page_table + (size_t)sid2 * c.max_pages);
        }
        // the caller's inputs: q as the B operand of S = K.q (the same in every column), KS k-steps of 16 elements; for
        // the first warp elements 64*j + 2*lane, + 1 of q and of the new row's K and V; attention alone: this lane's
        // first keep-mask word.  Requested with the other prologue loads when the dependency wait is behind us.
        uint32_t qa0[KS], qa2[KS];
        uint32_t qn[NJ], kn[NJ], vn[NJ], km0 = 0u;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) { qa0[ks] = 0u; qa2[ks] = 0u; }
#pragma unroll
        for (int j = 0; j < NJ; ++j) { qn[j] = 0u; kn[j] = 0u; vn[j] = 0u; }
        auto load_inputs = [&]() {
            if (a.in_ready) {
                // The caller's tensors may still be on their way (copies queued on another stream before this launch):
                // wait, for a bounded time, for the word that the copy after them writes.  The loads below bypass L1.
                const int *flag = a.in_ready + a.layer + local / c.S;
                int v = 0;
                for (int it = 0; it < in_spin; ++it) {
                    asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
                    if (v - a.in_epoch >= 0) break;
                    __nanosleep(200);
                }
                if (v - a.in_epoch < 0) {   // gave up: flag it, read what is there, and do not wait as long again
                    if (lane == 0) set_status(c, ADSA_DEV_COPY_TIMEOUT);
                    in_spin = kCopySpinAfterTimeout;
                }
            }
            const uint32_t *q2 = reinterpret_cast<const uint32_t *>(a.q + (size_t)local * c.d);   // c.d is even
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                int e0 = 16 * ks + 2 * t, e1 = e0 + 8;
                qa0[ks] = e0 < c.d ? __ldcg(q2 + (e0 >> 1)) : 0u;
                qa2[ks] = e1 < c.d ? __ldcg(q2 + (e1 >> 1)) : 0u;
            }
            if (rk == 0) {
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    if (64 * j + 2 * lane < c.d) {
                        qn[j] = __ldcg(q2 + 32 * j + lane);
                        kn[j] = __ldcg(reinterpret_cast<const uint32_t *>(a.k_new + (size_t)local * c.d) + 32 * j + lane);
                        vn[j] = __ldcg(reinterpret_cast<const uint32_t *>(a.v_new + (size_t)local * c.d) + 32 * j + lane);
                    }
                }
            }
            if constexpr (!FUSED) {
                if (rk + lane * G < c.mask_words) km0 = c.keep_mask[(size_t)sid * c.mask_words + rk + lane * G];
            }
        };
        if (waited) load_inputs();
        constexpr int kRound = 10;   // 32-row blocks whose selection inputs are fetched together
        int ps0[kRound];
        float sc0[kRound];
        // (the positions not when the previous step's note is expected to stand in for the classification)
        if constexpr (FUSED) {
            // positions and carried scores of this warp's first blocks: requested before n is known (the
            // arrays hold max_rows entries per stream, whatever n is), so that one memory latency covers
            // every load of the prologue
            const int32_t *pos_g = c.pos + (size_t)sid * c.max_rows;
            const float *sc_g = c.scores + (size_t)sid * c.max_rows;
#pragma unroll
            for (int u = 0; u < kRound; ++u) {
                const int slot = (rk + u * G) * 32 + lane;
                const bool in = slot < c.max_rows;
                ps0[u] = in && !try_fast ? pos_g[slot] : -1;
                sc0[u] = in ? sc_g[slot] : 0.f;
            }
        }
        float st0[NJ], st1[NJ];   // carried s[64*j + 2*lane], s[64*j + 2*lane + 1] of this step's previous region
#pragma unroll
        for (int j = 0; j < NJ; ++j) { st0[j] = 0.f; st1[j] = 0.f; }
        // (the two halves of a stream's 256 floats take turns: a step reads one and writes the other)
        float *const svec_in = c.svec + (size_t)sid * 256 + (a.cur_pos & 1) * 128, *const svec_out = c.svec + (size_t)sid * 256 + ((a.cur_pos + 1) & 1) * 128;
        if (FUSED && a.have_svec) {
#pragma unroll
            for (int j = 0; j < NJ; ++j) { st0[j] = svec_in[64 * j + 2 * lane]; st1[j] = svec_in[64 * j + 2 * lane + 1]; }
        }
        if (n < 0 || n > c.max_rows) { if (lane == 0 && rk == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW); n = 0; }
        const int n_tiles = (n + kWTile - 1) / kWTile;
        const int mt = rk < n_tiles ? div_g(n_tiles - rk + G - 1) : 0;   // this warp's tiles: rk, rk + G, ...
        int total = 0;    // stages to fetch: pass 1, and for the fused kernel pass 2 (V only) unless it can score during pass 1
        const float *inv_s = nullptr;
        if constexpr (FUSED) {
            // inverse norms into shared memory: aligned interior by bulk copy, ragged ends by plain loads
            const uint32_t *gp = reinterpret_cast<const uint32_t *>(inv_g);
            uint32_t *d = reinterpret_cast<uint32_t *>(smem + L.inv);
            const int lead = (int)(((uintptr_t)gp >> 2) & 3);
            inv_s = reinterpret_cast<const float *>(d + lead);
            if (rk == 0) {
                const int head = min(n, (4 - lead) & 3);
                const int body = (n - head) & ~3;
                if (lane < head) d[lead + lane] = gp[lane];
                if (lane < n - head - body) d[lead + head + body + lane] = gp[head + body + lane];
                __syncwarp();
                if (lane == 0) {
                    if (body > 0) bulk_g2s(smem_u32(d + lead + head), gp + head, (uint32_t)body * 4u, bar_meta);
                    mbar_expect_tx(bar_meta, (uint32_t)body * 4u);
                }
            }
        }
        __syncwarp();

        // ---- the warp's own copy pipeline ----------------------------------------------------------
        // Stages of this warp, in issue order: u = 0 .. ms-1 are pass 1 (K and V), u = ms .. 2ms-1 pass 2 (V only);
        // stage v of a pass is part v % NH (TR rows) of the warp's block v / NH, i.e. of block rk + (v / NH) * G.
        const int ms = mt * NH;
        total = ms;
        auto stage_row0 = [&](int u) {
            const int v = u >= ms ? u - ms : u;
            return (rk + (NH == 1 ? v : v >> 1) * G) * kWTile + (NH == 1 ? 0 : (v & 1) * TR);
        };
        auto issue = [&](int u) {   // all lanes (the copies themselves by lanes 0 and 1): this warp's u-th stage into the next free ring slot
            const int stage = i_stage;
            const int pass = u >= ms ? 1 : 0;
            const int r0 = stage_row0(u), r1 = max(r0, min(n, r0 + TR));
            const uint32_t kdst = stages_u32 + stage * kWStageBytes, vdst = kdst + kWTileBytes;
            const uint32_t bar = smem_u32(bars + stage);
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(r1 - r0) * kWRowBytes * (pass == 0 ? 2u : 1u));
            __syncwarp();
            const int pg0 = (int)__umulhi((uint32_t)r0, c.pr_magic), in0 = r0 - pg0 * c.page_rows;
            if constexpr (!SWZ) {
                // Plain tiles are the pool's rows as they lie: every page piece is one untiled bulk copy per pool
                // (a tensor copy wants its destination on a 128-byte boundary, which rows of 208 bytes do not keep).
                if (lane == 1 || (lane == 0 && pass == 0)) {
                    const __nv_bfloat16 *pool = lane ? c.v_pool : c.k_pool;
                    const uint32_t dst = lane ? vdst : kdst;
                    int r = r0, pg = pg0, in = in0;
                    if (r1 > r0 && in0 + (r1 - r0) <= c.page_rows) {   // the common case: the stage lies inside one page
                        bulk_g2s(dst, pool + ((size_t)pt_s[pg0] * c.page_rows + in0) * (size_t)RS, (uint32_t)(r1 - r0) * kWRowBytes, bar);
                        r = r1;
                    }
                    while (r < r1) {
                        const int cnt = min(r1 - r, c.page_rows - in);
                        bulk_g2s(dst + (uint32_t)(r - r0) * kWRowBytes, pool + ((size_t)pt_s[pg] * c.page_rows + in) * (size_t)RS,
                                 (uint32_t)cnt * kWRowBytes, bar);
                        r += cnt; in = 0; ++pg;
                    }
                }
            } else if (r1 - r0 == TR && in0 + TR <= c.page_rows) {
                // the common case: a whole tile inside one page is one box per pool; lane 0 copies K, lane 1 copies V
                constexpr int kBox = TR == 32 ? 5 : 4;
                const int y = pt_s[pg0] * c.page_rows + in0;
                if (lane == 1 || (lane == 0 && pass == 0)) {
#pragma unroll
                    for (int sg = 0; sg < NSEG; ++sg)
                        tma_2d((lane ? vdst : kdst) + sg * SEGB, lane ? &maps.v[kBox] : &maps.k[kBox], 64 * sg, y, bar);
                }
            } else if (lane == 0) {
                int r = r0, pg = pg0, in = in0;
                while (r < r1) {   // page pieces, each cut into boxes of 32, 16, 8, 4, 2 or 1 rows
                    int cnt = min(r1 - r, c.page_rows - in);
                    int y = pt_s[pg] * c.page_rows + in;
                    uint32_t off = (uint32_t)(r - r0) * PITCH;
                    r += cnt; in = 0; ++pg;
                    while (cnt > 0) {
                        int hb = 31 - __clz(cnt);
                        hb = hb > 5 ? 5 : hb;
#pragma unroll
                        for (int sg = 0; sg < NSEG; ++sg) {
                            if (pass == 0) tma_2d(kdst + sg * SEGB + off, &maps.k[hb], 64 * sg, y, bar);
                            tma_2d(vdst + sg * SEGB + off, &maps.v[hb], 64 * sg, y, bar);
                        }
                        y += 1 << hb; off += (uint32_t)PITCH << hb; cnt -= 1 << hb;
                    }
                }
            }
        };
        // Rows of a partial tile that the copy does not write must hold finite numbers (their weights
        // are zero, and 0 * NaN would not be): all lanes clear them before the tile is requested.
        auto clear_tail = [&](int u) {
            constexpr int kChunks = PITCH / 16;      // 16-byte chunks of a row inside a sub-tile (the swizzle moves chunks within their row only)
            const int r0 = stage_row0(u);
            const int rows = max(0, min(n - r0, TR));
            if (rows < TR) {
                uint4 *z = reinterpret_cast<uint4 *>(ring + i_stage * kWStageBytes);
#pragma unroll
                for (int sg = 0; sg < NSEG; ++sg)
                    for (int i = rows * kChunks + lane; i < TR * kChunks; i += 32) {
                        z[sg * (TR * kChunks) + i] = make_uint4(0u, 0u, 0u, 0u);
                        z[kWTileBytes / 16 + sg * (TR * kChunks) + i] = make_uint4(0u, 0u, 0u, 0u);
                    }
            }
        };
        // HBM is otherwise idle until the attention sweep starts (the ring holds `depth` stages and the
        // selection comes first), so the rows of the blocks after those are asked into L2 now, and one
        // block further with every block consumed: the sweep then finds them in L2.
        auto l2_ask = [&](int u) {   // this warp's u-th block: one hint per pool if a single page holds it, else a row per lane
            const int b0 = (rk + u * G) * kWTile, row = b0 + lane;
            if (u >= mt) return;
            const int rows = min(n - b0, kWTile);
            const int pg0 = (int)__umulhi((uint32_t)b0, c.pr_magic), in0 = b0 - pg0 * c.page_rows;
            if (in0 + rows <= c.page_rows) {
                if (lane < 2) {
                    const __nv_bfloat16 *src = (lane ? c.v_pool : c.k_pool) + ((size_t)pt_s[pg0] * c.page_rows + in0) * (size_t)g_rs;
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(rows * g_rs * 2) : "memory");
                }
            } else if (row < n) {
                const size_t off = c.max_pages == 1 ? ((size_t)pt_s[0] * c.page_rows + row) * (size_t)c.row_stride
                                                    : row_offset(c, pt_s, row);
                hint_row(c.k_pool + off);
                hint_row(c.v_pool + off);
            }
        };
        // stages with fewer than TR rows: only in the stream's last block, from the part that holds row n on
        const int partial_v = (n & (kWTile - 1)) && mt > 0 && rk + (mt - 1) * G == n_tiles - 1
                                  ? (mt - 1) * NH + (n & (kWTile - 1)) / TR : 0x7fffffff;
        int next_issue = 0;
        for (; next_issue < total && next_issue < D; ++next_issue) {
            if (next_issue >= partial_v) {   // generic-proxy stores into a stage are fenced before the copy that follows them
                clear_tail(next_issue);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            issue(next_issue);
            i_stage = i_stage + 1 == D ? 0 : i_stage + 1;
        }

        if constexpr (FUSED) {
            for (int u = (D + NH - 1) / NH; u < (D + NH - 1) / NH + a.l2_ahead; ++u) l2_ask(u);
        }
        // The row the previous step named as this step's evictee (its note, when this step is a steady one with a
        // full cache): its V row is asked for now, behind the first tiles.
        const int carried_slot = try_fast && n == a.budget_rows && note.x == 1 && note.y >= 1 && note.w >= 1 && note.w <= n ? note.w - 1 : -1;
        uint32_t ve[NJ];
#pragma unroll
        for (int j = 0; j < NJ; ++j) ve[j] = 0u;
        if (carried_slot >= 0) {
            const uint32_t *vrow = reinterpret_cast<const uint32_t *>(c.v_pool + row_offset(c, pt_s, carried_slot));
#pragma unroll
            for (int j = 0; j < NJ; ++j) ve[j] = 64 * j + 2 * lane < g_rs ? vrow[32 * j + lane] : 0u;
        }
        // after a stage has been read (all lanes), lane 0 refills it with the tile `depth` ahead
        // (the reads are complete once their results have been used, which in-order issue guarantees
        // for this thread and __syncwarp for the others; a fence is needed only after the generic-proxy
        // stores of clear_tail)
        auto release_and_refill = [&]() {
            if (FUSED && a.l2_ahead > 0 && (NH == 1 || (next_issue & 1) == 0)) l2_ask((NH == 1 ? next_issue : next_issue >> 1) + a.l2_ahead);
            if (next_issue < total) {
                if ((next_issue >= ms ? next_issue - ms : next_issue) >= partial_v) {
                    clear_tail(next_issue);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                __syncwarp();
                issue(next_issue);
                ++next_issue;
                i_stage = i_stage + 1 == D ? 0 : i_stage + 1;
            }
            c_stage = c_stage + 1 == D ? 0 : c_stage + 1;   // the stage just read is done with
            if (c_stage == 0) c_par ^= 1u;
        };
        // the barrier of the tile after the current one is tested early, so that the test's latency
        // overlaps the arithmetic; `ready` is true when that test already saw the tile complete
        bool ready = false;
        auto peek_next = [&](bool more) {
            const int ns = c_stage + 1 == D ? 0 : c_stage + 1;
            ready = more && mbar_try_wait(smem_u32(bars + ns), ns == 0 ? c_par ^ 1u : c_par);
        };

        // s (lane-distributed: s[64*j + 2*lane], + 1) as the B operand of the score product: columns
        // 0, 1, 2 = its bf16 hi, mid, lo parts
        uint32_t sb0[KS], sb1[KS];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) { sb0[ks] = 0u; sb1[ks] = 0u; }
        auto make_sb = [&](const float (&s0)[NJ], const float (&s1)[NJ]) {
            // each lane splits its own elements (hi = bf16(x), mid = bf16(x - hi), lo = bf16(x - hi - mid)),
            // packed in pairs; the fragments are then gathered with shuffles
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const uint32_t ph = pack_bf16(s0[j], s1[j]);
                const float r0 = s0[j] - bf16_lo(ph), r1 = s1[j] - bf16_hi(ph);
                const uint32_t pm = pack_bf16(r0, r1);
                const uint32_t pl = pack_bf16(r0 - bf16_lo(pm), r1 - bf16_hi(pm));
#pragma unroll
                for (int ks = 4 * j; ks < 4 * j + 4 && ks < KS; ++ks) {
                    const int src = 8 * (ks & 3) + t;   // elements 16*ks + 2t, + 1 live in lane 8*(ks % 4) + t of set ks / 4; + 8, + 9 four lanes on
                    const uint32_t ah = __shfl_sync(0xffffffffu, ph, src), am = __shfl_sync(0xffffffffu, pm, src),
                                   al = __shfl_sync(0xffffffffu, pl, src);
                    const uint32_t bh = __shfl_sync(0xffffffffu, ph, src + 4), bm = __shfl_sync(0xffffffffu, pm, src + 4),
                                   bl = __shfl_sync(0xffffffffu, pl, src + 4);
                    sb0[ks] = g == 0 ? ah : g == 1 ? am : g == 2 ? al : 0u;
                    sb1[ks] = g == 0 ? bh : g == 1 ? bm : g == 2 ? bl : 0u;
                }
            }
        };
        // Eq. 1-2 for the next step on one tile of V rows: dot_i = v_i . s by MMA,
        // S_i = (dot_i/|v_i| - u_i.u_i) / (p' - 1), written at the row's new slot
        int list_ns = 0, n2 = n;   // survivors of the general compaction; live rows after the update
        bool warp_rare = false, warp_clamped = false;   // warp_clamped: one of the rows this warp scores has a clamped norm
        float rden = 0.f;
        // (two halves, so that the products can be issued early and their results used later)
        auto score_mma = [&](uint32_t vb, float (&dt)[MB][4]) {
#pragma unroll
            for (int mbk = 0; mbk < MB; ++mbk) {
                float dt2[4];   // the odd k-steps: two short chains of MMAs instead of one long one
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t af[4];
                    ldsm_x4(a_addr(vb, mbk, ks), af);
                    if (ks == 0) mma_bf16_z(dt[mbk], af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                    else if (SPLIT && ks == 1) mma_bf16_z(dt2, af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                    else if (SPLIT && (ks & 1)) mma_bf16(dt2, af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                    else mma_bf16(dt[mbk], af[0], af[1], af[2], af[3], sb0[ks], sb1[ks]);
                }
                if (SPLIT) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) dt[mbk][i] += dt2[i];
                }
            }
        };
        // r0: the stream row of the tile's first row; cw: bit i = row r0 + i is to be scored
        float *const scores_g = c.scores + (size_t)sid * c.max_rows;
        // the highest score this lane has written, the slot it went to, and whether another of its rows had the same
        // score: the next step's evictee if that step keeps all but one of these rows (Eq. 3 with K = p - 1)
        float top_s = -INFINITY;
        int top_slot = -1;
        bool top_tie = false;
        auto note_top = [&](float s_out, int dst) {
            if (s_out > top_s) { top_s = s_out; top_slot = dst; top_tie = false; }
            else if (s_out == top_s) top_tie = true;
        };
        auto score_write = [&](const float (&dt)[MB][4], const unsigned char *vtile, int r0, uint32_t cw) {
            // Rows 16*mbk + 8*hh + g of the product: columns 0, 1 sit in lane t = 0 of the row's group of four, column 2
            // in lane t = 1 (whose second column is zero).  The three parts are added up across the pair and the sums
            // are then handed round so that lane i holds row i of the stage: one row per lane from here on.
            float dot = 0.f;
#pragma unroll
            for (int mbk = 0; mbk < MB; ++mbk) {
                float a = dt[mbk][0] + dt[mbk][1], b = dt[mbk][2] + dt[mbk][3];
                a += __shfl_xor_sync(0xffffffffu, a, 1);
                b += __shfl_xor_sync(0xffffffffu, b, 1);
                const float va = __shfl_sync(0xffffffffu, a, 4 * (lane & 7)), vb = __shfl_sync(0xffffffffu, b, 4 * (lane & 7));
                if (MB == 1 || (lane >> 4) == mbk) dot = (lane & 8) ? vb : va;
            }
            const int row = r0 + lane;
            if (!(lane < TR && ((cw >> lane) & 1u))) return;
            const float inv = inv_s[row];
            // warp_rare (set when the row weights were made): one of this warp's scored rows has a clamped
            // norm, or rows move down in the update; otherwise every row is written where it stands
            if (!warp_rare) {
                const float s_out = (inv * dot - 1.0f) * rden + 0.0f;
                scores_g[row] = s_out;
                note_top(s_out, row);
                return;
            }
            float s_out = (inv * dot - 1.0f) * rden + 0.0f;
            if (inv >= 1.0f / kNormEps) {   // |v| was clamped: u.u is not 1, take it from the row
                float ss = 0.f;
                for (int ch = 0; ch < RS / 8; ++ch) {
                    float f[8];
                    unpack8(*reinterpret_cast<const uint4 *>(vtile + chunk_off(lane, ch)), f);
                    for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
                }
                s_out = (inv * dot - inv * inv * ss) * rden + 0.0f;
            }
            int dst = row;
            if (row >= n2) {   // a survivor: it moves into the hole of the same rank
                const int32_t *holes = reinterpret_cast<const int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;
                int lo_i = 0, hi_i = list_ns - 1;
                while (lo_i < hi_i) { int mid = (lo_i + hi_i) >> 1; if (surv[mid] < row) lo_i = mid + 1; else hi_i = mid; }
                dst = holes[lo_i];
            }
            scores_g[dst] = s_out;
            note_top(s_out, dst);
        };
        // this warp's highest written score into its partial state: {score, slot or -1 if two rows share it}
        auto publish_top = [&](float *w, int at) {
            float v = top_s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            const bool mine = top_slot >= 0 && top_s == v;
            const unsigned who = __ballot_sync(0xffffffffu, mine);
            const bool tie = __any_sync(0xffffffffu, mine && top_tie) || __popc(who) > 1;
            const int wslot = who ? __shfl_sync(0xffffffffu, top_slot, __ffs(who) - 1) : -1;
            if (lane == 0) { w[at] = v; reinterpret_cast<int *>(w)[at + 1] = tie ? -1 : wslot; }
        };

        // ---- which rows are attended, and the weights of the rows the next step scores -------------
        // Each warp of the group looks at the 32-row blocks it will also sweep (rk, rk + G, ...).
        int p_next = 0, n_evict = 0, evict_slot = -1;
        // Single sweep: when the next step's previous region is this step's minus the evicted row (no
        // row leaves the local window, at most one eviction), its sum of normalised rows is the carried
        // sum minus that row, known before the sweep, and the next scores are taken during pass 1.
        bool single = false;
        // The short way.  The previous fused step has scored this step's previous region and left a mask of its
        // slots and its size; if the cache is exactly full (n = budget: K = p - 1, one row goes) and the next
        // step's previous region is this one's minus that row, nothing has to be classified: the evicted row is
        // the highest carried score under the mask (two equal highest scores: positions decide, the long way
        // looks at them), all other rows are kept, the rows to score are the mask minus that row, and
        // s' = s - u_e.  The sum of normalised rows is not summed again: s' is carried on (it is summed afresh
        // whenever the long way runs, at least once per grid row).
        bool fast = false;
        if (carried_slot >= 0) {
            // the previous step has named the row: the highest of the scores it wrote (one row alone had it)
            fast = true;
            evict_slot = carried_slot;
        } else if (try_fast && n == a.budget_rows && note.x == 1 && note.y >= 1) {   // the same decision in every warp of the group
            const float *sc_g = c.scores + (size_t)sid * c.max_rows;
            float best = -INFINITY;
            int best_slot = -1;
            bool tie = false;
            for (int b0 = rk, idx0 = 0; b0 < n_tiles; b0 += kRound * G, idx0 += kRound) {
#pragma unroll
                for (int u = 0; u < kRound; ++u) {
                    const int b = b0 + u * G;
                    if (b >= n_tiles) break;
                    const int slot = b * 32 + lane;
                    const float sc = b0 == rk ? sc0[u] : (slot < n ? sc_g[slot] : 0.f);
                    const uint32_t w = idx0 + u < 32 ? __shfl_sync(0xffffffffu, cand_w, idx0 + u)
                                                     : c.cand_mask[(size_t)sid * c.mask_words + b];
                    if (((w >> lane) & 1u) && slot < n) {
                        if (sc > best) { best = sc; best_slot = slot; tie = false; }
                        else if (sc == best) tie = true;
                    }
                }
            }
            float v = best;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            const bool mine = best_slot >= 0 && best == v;
            const unsigned who = __ballot_sync(0xffffffffu, mine);
            tie = __any_sync(0xffffffffu, mine && tie) || __popc(who) > 1;
            const int wslot = who ? __shfl_sync(0xffffffffu, best_slot, __ffs(who) - 1) : -1;
            float *tops = reinterpret_cast<float *>(smem + L.hdr + kWMaxGroupWarps * 32 + 32);
            if (lane == 0) { tops[rk * 4] = v; reinterpret_cast<int *>(tops)[rk * 4 + 1] = tie ? -1 : wslot; }
            group_sync();
            float gbest = -INFINITY;
            int gslot = -1;
            bool gtie = false;
            for (int w = 0; w < G; ++w) {
                const float wv = tops[w * 4];
                const int ws = reinterpret_cast<const int *>(tops)[w * 4 + 1];
                if (wv > gbest) { gbest = wv; gslot = ws; gtie = false; }
                else if (wv == gbest && wv > -INFINITY) gtie = true;
            }
            fast = gslot >= 0 && !gtie;
            if (fast) evict_slot = gslot;
        }
        if (fast) {
            n_evict = 1; n2 = n; single = true;
            p_next = note.y - 1;
            rden = p_next > 1 ? 1.0f / (float)(p_next - 1) : 0.0f;
            warp_clamped = (note.z & 1) != 0;   // known for the stream as a whole
            warp_rare = warp_clamped;
            if (carried_slot < 0) {
                const uint32_t *vrow = reinterpret_cast<const uint32_t *>(c.v_pool + row_offset(c, pt_s, evict_slot));
#pragma unroll
                for (int j = 0; j < NJ; ++j) ve[j] = 64 * j + 2 * lane < g_rs ? vrow[32 * j + lane] : 0u;
            }
            const uint32_t *cm_g = c.cand_mask + (size_t)sid * c.mask_words;
            for (int b = rk + lane * G; b < n_tiles; b += 32 * G) {   // one block per lane
                const int valid = n - b * 32;
                uint32_t keep = valid >= 32 ? 0xffffffffu : ((1u << valid) - 1u);
                if ((evict_slot >> 5) == b) keep &= ~(1u << (evict_slot & 31));
                kmask[b] = keep; cmask[b] = (b == rk + lane * G ? cand_w : cm_g[b]) & keep;
            }
            wait(bar_meta, streams_done & 1);   // the inverse norms are in shared memory
            const float inv_e = inv_s[evict_slot];
            float sp0[NJ], sp1[NJ];
#pragma unroll
            for (int j = 0; j < NJ; ++j) { sp0[j] = fmaf(-inv_e, bf16_lo(ve[j]), st0[j]); sp1[j] = fmaf(-inv_e, bf16_hi(ve[j]), st1[j]); }
            make_sb(sp0, sp1);
            if (rk == 0) {   // s' is what the next step starts from
#pragma unroll
                for (int j = 0; j < NJ; ++j) { svec_out[64 * j + 2 * lane] = sp0[j]; svec_out[64 * j + 2 * lane + 1] = sp1[j]; }
            }
        } else if constexpr (FUSED) {
            const int32_t *pos_g = c.pos + (size_t)sid * c.max_rows;
            const float *sc_g = c.scores + (size_t)sid * c.max_rows;
            WSelPartial mine = {0ull, -1, 0, 0, 0, 0, 0};
            uint32_t my_hi = 0u, my_lo = 0u;   // the lane's largest key so far: orderable score, position
            int my_slot = -1;
            const bool same_cut = cut_next.lo == cut_now.lo;   // the local window does not move: candidates = previous region
            // previous region now: n_prefix <= pos < min(lo, cur); at the next step (for rows valid now): < min(lo', cur)
            const uint32_t pre = (uint32_t)c.n_prefix;
            const uint32_t span_now = (uint32_t)max(0, min(cut_now.lo, cut_now.cur) - c.n_prefix);
            const uint32_t span_next = (uint32_t)max(0, min(cut_next.lo, cut_now.cur) - c.n_prefix);
            for (int b0 = rk; b0 < n_tiles; b0 += kRound * G) {   // kRound blocks per round: their loads overlap
                int ps[kRound];
                float sc[kRound];
#pragma unroll
                for (int u = 0; u < kRound; ++u) {
                    if (b0 == rk && !try_fast) { ps[u] = ps0[u]; sc[u] = sc0[u]; continue; }   // the first round came with the prologue
                    const int slot = (b0 + u * G) * 32 + lane;
                    const bool live = b0 + u * G < n_tiles && slot < n;
                    ps[u] = live ? pos_g[slot] : -1;
                    sc[u] = live ? sc_g[slot] : 0.f;
                }
#pragma unroll
                for (int u = 0; u < kRound; ++u) {
                    const int b = b0 + u * G;
                    if (b >= n_tiles) break;
                    const int slot = b * 32 + lane;
                    const bool live = slot < n;
                    const uint32_t pu = (uint32_t)ps[u];
                    const bool is_prev = live && pu - pre < span_now;
                    if (live && pu >= (uint32_t)cut_now.cur) set_status(c, ADSA_DEV_BAD_POSITION);   // negative, or not before the current position
                    if (is_prev) {
                        const uint32_t hi = orderable(sc[u]);
                        if (hi > my_hi || (hi == my_hi && pu > my_lo)) { my_hi = hi; my_lo = pu; my_slot = slot; }
                    }
                    const unsigned bp = __ballot_sync(0xffffffffu, is_prev);
                    unsigned bc = bp;
                    if (!same_cut) {
                        bc = __ballot_sync(0xffffffffu, live && pu < (uint32_t)cut_now.cur && pu - pre < span_next);
                        mine.n_cand += __popc(bc);
                        mine.n_cand_not_prev += __popc(bc & ~bp);
                    }
                    mine.p += __popc(bp);
                    if (lane == 0) { prevm[b] = bp; candm[b] = bc; }
                }
            }
            if (same_cut) mine.n_cand = mine.p;
            unsigned long long my_key;
            {   // the warp's largest key (keys are distinct: the low word is the position) and its slot
                const uint32_t kh = my_hi, kl = my_lo;
                const uint32_t mh = __reduce_max_sync(0xffffffffu, kh);
                const uint32_t ml = __reduce_max_sync(0xffffffffu, kh == mh ? kl : 0u);
                const int src = __ffs(__ballot_sync(0xffffffffu, kh == mh && kl == ml)) - 1;
                my_slot = __shfl_sync(0xffffffffu, my_slot, src);
                my_key = ((unsigned long long)mh << 32) | ml;
            }
            mine.max_key = my_key; mine.max_slot = my_slot;
            if (lane == 0) {
                sel_part[rk] = mine;
                // the row this warp would evict is one of the group's candidates: a hint now makes the load of
                // the chosen one, after the group has met, a short one
                if (my_slot >= 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(c.v_pool + row_offset(c, pt_s, my_slot)));
            }
            group_sync();
            int p = 0, n_cand = 0, n_cand_np = 0;
            unsigned long long max_key = 0ull;
            int max_slot = -1;
            for (int w = 0; w < G; ++w) {
                const WSelPartial o = sel_part[w];
                p += o.p; n_cand += o.n_cand; n_cand_np += o.n_cand_not_prev;
                if (o.max_key > max_key) { max_key = o.max_key; max_slot = o.max_slot; }
            }
            int K = a.budget_rows - (n - p) - 1;   // every live row outside the previous region is kept; 1 = the new row
            K = K < 0 ? 0 : (K > p ? p : K);
            n_evict = p - K;
            n2 = n - n_evict + 1;
            wait(bar_meta, streams_done & 1);   // the inverse norms are in shared memory
            const bool general = K > 0 && K < p - 1;
            single = a.have_svec && !general && n_evict <= 1 && n_cand_np == 0 && !new_cand;
            uint32_t ve[NJ];       // single sweep: the evicted row's elements 64*j + 2*lane, + 1, requested as early as possible
#pragma unroll
            for (int j = 0; j < NJ; ++j) ve[j] = 0u;
            float inv_e = 0.f;
            if (!general) {
                if (K == p - 1 && p > 0) evict_slot = max_slot;
                if (single && evict_slot >= 0) {
                    const uint32_t *vrow = reinterpret_cast<const uint32_t *>(c.v_pool + row_offset(c, pt_s, evict_slot));
#pragma unroll
                    for (int j = 0; j < NJ; ++j) ve[j] = 64 * j + 2 * lane < g_rs ? vrow[32 * j + lane] : 0u;
                    inv_e = inv_s[evict_slot];
                }
                const bool drop_prev = K == 0 && p > 0;
                for (int b = rk + lane * G; b < n_tiles; b += 32 * G) {   // one block per lane
                    const int valid = n - b * 32;
                    uint32_t keep = valid >= 32 ? 0xffffffffu : ((1u << valid) - 1u);
                    if (drop_prev) keep &= ~prevm[b];
                    if (evict_slot >= 0 && (evict_slot >> 5) == b) keep &= ~(1u << (evict_slot & 31));
                    kmask[b] = keep; cmask[b] = candm[b] & keep;
                }
                p_next = K >= p ? n_cand : drop_prev ? n_cand_np : n_cand - ((candm[evict_slot >> 5] >> (evict_slot & 31)) & 1u);
            } else {
                // arbitrary K: the keys of all rows into shared memory (each warp its blocks), radix select
                // over them by the first warp, then every warp marks every block
                for (int b = rk; b < n_tiles; b += G) {
                    const int slot = b * 32 + lane;
                    if (slot < n)
                        sm_keys[slot] = ((prevm[b] >> lane) & 1u)
                                            ? ((unsigned long long)orderable(sc_g[slot]) << 32) | (uint32_t)pos_g[slot] : ~0ull;
                }
                group_sync();
                if (rk == 0) {
                    unsigned long long mask = 0ull, thr = 0ull;
                    int k_rem = K;
                    for (int shift = 56; shift >= 0; shift -= 8) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) hist[lane * 8 + i] = 0;
                        __syncwarp();
                        for (int slot = lane; slot < n; slot += 32) {
                            unsigned long long key = sm_keys[slot];
                            if (((prevm[slot >> 5] >> (slot & 31)) & 1u) && (key & mask) == thr)
                                atomicAdd(&hist[(int)((key >> shift) & 255ull)], 1);
                        }
                        __syncwarp();
                        int h[8], tot = 0;
#pragma unroll
                        for (int i = 0; i < 8; ++i) { h[i] = hist[lane * 8 + i]; tot += h[i]; }
                        int incl = tot;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            int tt = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= o) incl += tt;
                        }
                        int excl = incl - tot, digit = 0, krem = 0, bin = 0;
                        const bool own = excl < k_rem && k_rem <= incl;   // exactly one lane holds the bin of the k_rem-th key
                        if (own) {
                            int cum = excl;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (cum < k_rem && k_rem <= cum + h[i]) { digit = lane * 8 + i; krem = k_rem - cum; bin = h[i]; }
                                cum += h[i];
                            }
                        }
                        const int src = __ffs(__ballot_sync(0xffffffffu, own)) - 1;
                        digit = __shfl_sync(0xffffffffu, digit, src);
                        krem = __shfl_sync(0xffffffffu, krem, src);
                        bin = __shfl_sync(0xffffffffu, bin, src);
                        thr |= (unsigned long long)digit << shift;
                        mask |= 255ull << shift;
                        k_rem = krem;
                        __syncwarp();
                        if (k_rem == bin) break;             // the whole bin is kept: masked compare decides
                    }
                    if (lane == 0) { sel_thr[0] = mask; sel_thr[1] = thr; }
                }
                group_sync();
                const unsigned long long mask = sel_thr[0], thr = sel_thr[1];
                for (int b = 0; b < n_tiles; ++b) {   // all blocks: the compaction lists need them all
                    const int slot = b * 32 + lane;
                    const bool live = slot < n;
                    const bool is_prev = (prevm[b] >> lane) & 1u;
                    const bool kept = live && (!is_prev || (sm_keys[slot] & mask) <= thr);
                    const unsigned bk = __ballot_sync(0xffffffffu, kept);
                    const unsigned bcm = candm[b] & bk;
                    p_next += __popc(bcm);
                    __syncwarp();
                    if (lane == 0) { kmask[b] = bk; cmask[b] = bcm; }   // every warp writes the same words
                }
            }
            p_next += new_cand ? 1 : 0;
            if (!single) total = 2 * ms;
            rden = p_next > 1 ? 1.0f / (float)(p_next - 1) : 0.0f;   // p' <= 1: every score is 0
            __syncwarp();
            // does one of the rows this warp will score have a clamped norm?  (their weights 1/|v| are split into
            // bf16 parts tile by tile during the sweep)
            if (general) group_sync();
            {
                float w_big = 0.f;   // the largest 1/|v| among the rows this warp will score
                for (int i = 0; rk + i * G < n_tiles; ++i) {
                    const int b = rk + i * G;
                    if ((cmask[b] >> lane) & 1u) w_big = fmaxf(w_big, inv_s[b * 32 + lane]);
                }
                warp_clamped = __any_sync(0xffffffffu, w_big >= 1.0f / kNormEps);
                warp_rare = warp_clamped || n2 < n;
            }
            if (single)   // s' = s - u_e: the evicted row (if any) leaves the previous region
            {
                float sp0[NJ], sp1[NJ];
#pragma unroll
                for (int j = 0; j < NJ; ++j) { sp0[j] = fmaf(-inv_e, bf16_lo(ve[j]), st0[j]); sp1[j] = fmaf(-inv_e, bf16_hi(ve[j]), st1[j]); }
                make_sb(sp0, sp1);
            }
        } else {
            if (!waited) { dep_wait(); load_inputs(); }
            const uint32_t *gm = c.keep_mask + (size_t)sid * c.mask_words;
            for (int b = rk + lane * G; b < n_tiles; b += 32 * G) {
                uint32_t bits = b == rk + lane * G ? km0 : gm[b];
                int valid = n - b * 32;
                kmask[b] = valid >= 32 ? bits : (bits & ((1u << valid) - 1u));
            }
        }
        __syncwarp();

        if (FUSED && !waited) { dep_wait(); load_inputs(); }   // the whole selection came first: it reads the cache state only
        // ---- the running state; the first warp starts from the new row: weight 1 for role 0, its 1/|v| for role 2 ----
        // o_run[md][0..3]: dimension 16*md + g (0, 1) and 16*md + g + 8 (2, 3), roles 2t (0, 2) and 2t + 1 (1, 3), where
        // role 0/1 = softmax.V through P_hi / P_lo and roles 2/3/4 = s through w_hi / w_mid / w_lo.
        float m_run = -FLT_MAX, l_run = 0.f, o_run[KS][4];
#pragma unroll
        for (int md = 0; md < KS; ++md) { o_run[md][0] = o_run[md][1] = o_run[md][2] = o_run[md][3] = 0.f; }
        float ss_new = 0.f, inv_row_new = 0.f;   // first warp: |v_new|^2 and 1 / max(|v_new|, eps)
        if (rk == 0) {
            float s = 0.f, ss = 0.f;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                s = fmaf(bf16_hi(qn[j]), bf16_hi(kn[j]), fmaf(bf16_lo(qn[j]), bf16_lo(kn[j]), s));
                ss = fmaf(bf16_hi(vn[j]), bf16_hi(vn[j]), fmaf(bf16_lo(vn[j]), bf16_lo(vn[j]), ss));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, o);
                ss += __shfl_xor_sync(0xffffffffu, ss, o);
            }
            ss_new = ss;
            inv_row_new = 1.0f / fmaxf(sqrtf(ss), kNormEps);
            const float inv_new = new_cand ? inv_row_new : 0.f;
            m_run = s * c.scale_log2e;
            l_run = g == 0 ? 1.f : 0.f;   // summed over the eight g lanes at the end
            const float wrole = t == 0 ? 1.f : t == 1 ? inv_new : 0.f;   // role 0 in lanes t = 0, role 2 in lanes t = 1
#pragma unroll
            for (int md = 0; md < KS; ++md) {
                // elements 16*md + g and 16*md + g + 8 sit in set md / 4, lanes 8*(md % 4) + g/2 and + 4, half g & 1
                const uint32_t w0 = __shfl_sync(0xffffffffu, vn[md >> 2], 8 * (md & 3) + (g >> 1)),
                               w1 = __shfl_sync(0xffffffffu, vn[md >> 2], 8 * (md & 3) + (g >> 1) + 4);
                o_run[md][0] = wrole * ((g & 1) ? bf16_hi(w0) : bf16_lo(w0));
                o_run[md][2] = wrole * ((g & 1) ? bf16_hi(w1) : bf16_lo(w1));
            }
        }

        // ---- pass 1: block by block, a block in NH stages of TR rows --------------------------------
        for (int tl = rk; tl < n_tiles; tl += G) {
#pragma unroll
          for (int part_i = 0; part_i < NH; ++part_i) {
            const int stage = c_stage;
            if (!ready) wait(smem_u32(bars + stage), c_par);
            const uint32_t kb = stages_u32 + stage * kWStageBytes, vb = kb + kWTileBytes;
            const int r0 = tl * kWTile + part_i * TR;
            const uint32_t kw = (kmask[tl] >> (part_i * TR)) >> g;   // bits 0, 8 (, 16, 24): rows g, g + 8 (, g + 16, g + 24) of the stage are retained
            // S = K.q: A = 16 rows of K, B = q in every column, so every lane of a group of four holds the
            // logits of rows 16*mb + g (c0 = c1) and 16*mb + g + 8 (c2 = c3)
            // (wide rows: even and odd k-steps accumulate apart, so that a product is two short chains of MMAs instead of one long one)
            float sc[MB][4];
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
                float sc2[4];
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t kf[4];
                    ldsm_x4(a_addr(kb, mb, ks), kf);
                    if (ks == 0) mma_bf16_z(sc[mb], kf[0], kf[1], kf[2], kf[3], qa0[ks], qa2[ks]);
                    else if (SPLIT && ks == 1) mma_bf16_z(sc2, kf[0], kf[1], kf[2], kf[3], qa0[ks], qa2[ks]);
                    else if (SPLIT && (ks & 1)) mma_bf16(sc2, kf[0], kf[1], kf[2], kf[3], qa0[ks], qa2[ks]);
                    else mma_bf16(sc[mb], kf[0], kf[1], kf[2], kf[3], qa0[ks], qa2[ks]);
                }
                if (SPLIT) { sc[mb][0] += sc2[0]; sc[mb][2] += sc2[2]; }   // (columns 1 and 3 repeat 0 and 2)
            }
            peek_next(part_i + 1 < NH || tl + G < n_tiles || (FUSED && !single));
            float dts[MB][4];   // the score products of this tile, started before the softmax arithmetic
            if constexpr (FUSED) {
                if (single) score_mma(vb, dts);
            }
            float x[MB][2], mx = -INFINITY;   // x[mb][h]: row 16*mb + 8*h + g
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    bool kept = (kw >> (16 * mb + 8 * h)) & 1u;
                    x[mb][h] = kept ? sc[mb][2 * h] * c.scale_log2e : -INFINITY;
                    mx = fmaxf(mx, x[mb][h]);
                }
            }
            // the running maximum moves in few tiles of a stream: a vote tells whether the reduction over lanes is needed
            float m_new = m_run, corr = 1.0f;
            if (__any_sync(0xffffffffu, mx > m_run)) {
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                m_new = fmaxf(m_run, mx);
                corr = ex2(m_run - m_new);
                m_run = m_new;
            }
            float psum = 0.f;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
                for (int h = 0; h < 2; ++h) { x[mb][h] = ex2(x[mb][h] - m_new); psum += x[mb][h]; }
            }
            l_run = fmaf(l_run, corr, psum);
            // B' fragments for the 16-row k-steps of O^T = V^T.B': column g of B' is P_hi, P_lo, w_hi, w_mid, w_lo, 0, 0, 0.
            // The weights of rows 2t, 2t + 1 (+ 8) of a k-step sit in the lanes of groups g' = 2t and 2t + 1.
            uint32_t pb0[MB], pb2[MB];
#pragma unroll
            for (int ks = 0; ks < MB; ++ks) {
                const float p00 = __shfl_sync(0xffffffffu, x[ks][0], 8 * t), p01 = __shfl_sync(0xffffffffu, x[ks][0], 8 * t + 4);
                const float p10 = __shfl_sync(0xffffffffu, x[ks][1], 8 * t), p11 = __shfl_sync(0xffffffffu, x[ks][1], 8 * t + 4);
                uint32_t h0 = pack_bf16(p00, p01), h2 = pack_bf16(p10, p11);
                uint32_t l0 = pack_bf16(p00 - bf16_lo(h0), p01 - bf16_hi(h0));
                uint32_t l2 = pack_bf16(p10 - bf16_lo(h2), p11 - bf16_hi(h2));
                uint32_t w0 = 0u, w2 = 0u;
                if (FUSED && !fast) {   // the short way carries s' on instead of summing it again: no row weights
                    // w = 1/|v| of rows 2t, 2t + 1 (+ 8) of this k-step if the next step scores them, else 0; this
                    // lane's part of the split (g = 2, 3, 4: hi, mid, lo)
                    const int s0 = r0 + 16 * ks + 2 * t;
                    const uint32_t cm = cmask[tl] >> (part_i * TR + 16 * ks + 2 * t);
                    w0 = split_part((cm & 1u) ? inv_s[s0] : 0.f, (cm & 2u) ? inv_s[s0 + 1] : 0.f, g - 2);
                    w2 = split_part((cm & 0x100u) ? inv_s[s0 + 8] : 0.f, (cm & 0x200u) ? inv_s[s0 + 9] : 0.f, g - 2);
                }
                pb0[ks] = g == 0 ? h0 : g == 1 ? l0 : g <= 4 ? w0 : 0u;
                pb2[ks] = g == 0 ? h2 : g == 1 ? l2 : g <= 4 ? w2 : 0u;
            }
            // The running sums follow the running maximum (roles 0, 1 carry softmax weights; the weight sums of the other
            // roles are not rescaled).  The maximum is the same in every lane and moves in few tiles of a stream.
            if (corr != 1.0f) {
                const float corr_role = t == 0 ? corr : 1.0f;
#pragma unroll
                for (int md = 0; md < KS; ++md) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) o_run[md][i] *= corr_role;
                }
            }
            // O^T += V^T.B' (A = V^T through transposing ldmatrix), accumulated in the running sums themselves
#pragma unroll
            for (int mbk = 0; mbk < MB; ++mbk) {
#pragma unroll
                for (int md = 0; md < KS; ++md) {
                    uint32_t vf[4];
                    ldsm_x4_t(t_addr(vb, mbk, md), vf);
                    mma_bf16(o_run[md], vf[0], vf[1], vf[2], vf[3], pb0[mbk], pb2[mbk]);
                }
            }
            if constexpr (FUSED) {
                if (single) score_write(dts, ring + stage * kWStageBytes + kWTileBytes, r0, n2 <= c.max_rows ? cmask[tl] >> (part_i * TR) : 0u);
            }
            release_and_refill();
          }
        }

        // ---- HBM has nothing more to do for this stream: the first tiles the next launch will ask for go into L2 now,
        //      while this launch merges, updates and drains and the next one starts up ----
        if (sid2 >= 0 && a.next_tiles > 0) {
            const int nn = __shfl_sync(0xffffffffu, lane == 0 ? nxt[0] : 0, 0), pg0 = __shfl_sync(0xffffffffu, lane == 0 ? nxt[1] : 0, 0);
            if (nn > 0 && nn <= c.max_rows && pg0 >= 0 && pg0 < c.n_pages) {
                const int32_t *pt2 = c.page_table + (size_t)sid2 * c.max_pages;
                for (int u = 0; u < a.next_tiles; ++u) {
                    const int r0 = (rk + u * G) * kWTile, rows = min(nn, r0 + kWTile) - r0;
                    if (rows <= 0) break;
                    if (r0 + rows <= c.page_rows) {   // inside the first page: one bulk hint per pool
                        if (lane < 2) {
                            const __nv_bfloat16 *src = (lane ? c.v_pool : c.k_pool) + ((size_t)pg0 * c.page_rows + r0) * (size_t)c.row_stride;
                            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(rows * g_rs * 2) : "memory");
                        }
                    } else if (lane < rows) {         // a row per lane, located through the next stream's page table
                        const int row = r0 + lane;
                        const uint32_t pg = __umulhi((uint32_t)row, c.pr_magic);
                        const int page = __ldcg(pt2 + pg);
                        if (page >= 0 && page < c.n_pages) {
                            const size_t off = ((size_t)page * c.page_rows + ((uint32_t)row - pg * (uint32_t)c.page_rows)) * (size_t)c.row_stride;
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(c.k_pool + off));
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(c.v_pool + off));
                        }
                    }
                }
            }
        }
        // ---- this warp's state: softmax.V = roles 0 + 1, s = roles 2 + 3 + 4; then the warps of the group ----
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 4);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 8);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);
        constexpr int kAcc = 0, kSum = 64 * NJ, kML = 128 * NJ;   // offsets inside a warp's partial state
        {
            float *w = part + rk * kWPart;
#pragma unroll
            for (int md = 0; md < KS; ++md) {
                const float lo0 = __shfl_down_sync(0xffffffffu, o_run[md][0], 1), lo2 = __shfl_down_sync(0xffffffffu, o_run[md][2], 1);
                const int x0 = 16 * md + g, x1 = x0 + 8;
                if (t == 0) { w[kAcc + x0] = o_run[md][0] + o_run[md][1]; w[kAcc + x1] = o_run[md][2] + o_run[md][3]; }
                if (t == 1) { w[kSum + x0] = (o_run[md][0] + o_run[md][1]) + lo0; w[kSum + x1] = (o_run[md][2] + o_run[md][3]) + lo2; }
            }
            if (lane == 0) { w[kML] = m_run; w[kML + 1] = l_run; reinterpret_cast<int *>(w)[kML + 2] = warp_clamped ? 1 : 0; }
            if constexpr (FUSED) {
                if (single) publish_top(w, kML + 3);
            }
        }
        group_sync();
        float sv0[NJ], sv1[NJ];   // s[64*j + 2*lane], s[64*j + 2*lane + 1]
        {
            float M = -FLT_MAX;
            for (int w = 0; w < G; ++w) M = fmaxf(M, part[w * kWPart + kML]);
            float Lb = 0.f, A0[NJ], A1[NJ];
#pragma unroll
            for (int j = 0; j < NJ; ++j) { A0[j] = 0.f; A1[j] = 0.f; sv0[j] = 0.f; sv1[j] = 0.f; }
            for (int w = 0; w < G; ++w) {
                const float *ws = part + w * kWPart;
                float wgt = ex2(ws[kML] - M);
                Lb = fmaf(ws[kML + 1], wgt, Lb);
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    A0[j] = fmaf(ws[kAcc + 64 * j + 2 * lane], wgt, A0[j]);
                    A1[j] = fmaf(ws[kAcc + 64 * j + 2 * lane + 1], wgt, A1[j]);
                    sv0[j] += ws[kSum + 64 * j + 2 * lane];
                    sv1[j] += ws[kSum + 64 * j + 2 * lane + 1];
                }
            }
            const float rl = 1.0f / Lb;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const int xx = 64 * j + 2 * lane;
                if (rk == 0 && xx < c.d) {
                    float o0 = A0[j] * rl, o1 = A1[j] * rl;
                    if (a.out_f32) {
                        a.out_f32[(size_t)local * c.d + xx] = o0;
                        if (xx + 1 < c.d) a.out_f32[(size_t)local * c.d + xx + 1] = o1;
                    }
                    if (a.out_bf16)
                        *reinterpret_cast<uint32_t *>(a.out_bf16 + (size_t)local * c.d + xx) = pack_bf16(o0, o1);
                }
            }
        }

        if constexpr (FUSED) {
            if (rk == 0 && !fast) {   // carried to the next step together with the scores (the short way has written s' already)
#pragma unroll
                for (int j = 0; j < NJ; ++j) { svec_out[64 * j + 2 * lane] = sv0[j]; svec_out[64 * j + 2 * lane + 1] = sv1[j]; }
            }
            // ---- Section 4.2 bookkeeping: holes below the new length, survivors above it ----------
            int32_t *holes = reinterpret_cast<int32_t *>(sm_keys), *surv = holes + c.max_rows + 1;   // keys are dead now
            int nh = 1, ns = 0, last_hole = n;   // nothing evicted: the new row goes to the end
            if (n_evict == 1 && evict_slot >= 0) {
                last_hole = evict_slot;          // one eviction: the new row takes its place
            } else if (n_evict > 0) {
                // the general case; every warp builds the same lists (identical values to the same places)
                nh = 0;
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
                last_hole = nh > ns && nh > 0 ? holes[ns] : n;
            }
            list_ns = ns;
            // pages for n and for n2 rows (n2 beyond max_rows is refused below)
            const int have = n > 0 ? (int)__umulhi((uint32_t)(n - 1), c.pr_magic) + 1 : 0;
            const int need = (int)__umulhi((uint32_t)(min(n2, c.max_rows) - 1), c.pr_magic) + 1;
            int okay = 1;
            if (lane == 0) {
                if (nh != ns + 1) { if (rk == 0) set_status(c, ADSA_DEV_BAD_EVICT); okay = 0; }
                else if (n2 > c.max_rows) { if (rk == 0) set_status(c, ADSA_DEV_ROW_OVERFLOW); okay = 0; }
                else if (rk == 0 && need > have && !resize_pages(c, pt, have, need)) okay = 0;
            }
            okay = __shfl_sync(0xffffffffu, okay, 0);
            __syncwarp();   // lane 0 may have written a page-table entry the others are about to read
            float *scores = c.scores + (size_t)sid * c.max_rows;

            if (!single) {
                // ---- pass 2: the next step's scores from a second sweep over V, against the sum just completed ----
                make_sb(sv0, sv1);
                for (int tl = rk; tl < n_tiles; tl += G) {
#pragma unroll
                    for (int part_i = 0; part_i < NH; ++part_i) {
                        const int stage = c_stage;
                        if (!ready) wait(smem_u32(bars + stage), c_par);
                        peek_next(part_i + 1 < NH || tl + G < n_tiles);
                        float dt2[MB][4];
                        score_mma(stages_u32 + stage * kWStageBytes + kWTileBytes, dt2);
                        score_write(dt2, ring + stage * kWStageBytes + kWTileBytes, tl * kWTile + part_i * TR,
                                    okay ? cmask[tl] >> (part_i * TR) : 0u);
                        release_and_refill();
                    }
                }
                publish_top(part + rk * kWPart, kML + 3);
            }
            // every warp's copies of this stream have landed before rows move or pages are freed (after a single
            // sweep the group has met since its last copy landed: at the merge of the partial states)
            if (!single) group_sync();

            // ---- the note for the next step: its previous region by slot and by size, clamped-norm flag ----
            if (okay) {
                uint32_t *cm_g = c.cand_mask + (size_t)sid * c.mask_words;
                const uint32_t new_bit = new_cand ? 1u << (last_hole & 31) : 0u;
                if (fast) {   // one word changes: the evicted row's slot now holds the new row, which is local
                    const int b = evict_slot >> 5;
                    if (lane == 0 && b - div_g(b) * G == rk) cm_g[b] = cmask[b];
                } else {
                    for (int b = rk + lane * G; b * 32 < n2; b += 32 * G) {
                        uint32_t word = b < n_tiles ? cmask[b] : 0u;
                        if (b * 32 + 32 > n2) word &= (1u << (n2 - b * 32)) - 1u;   // bits of slots the update vacates
                        if ((last_hole >> 5) == b) word |= new_bit;
                        cm_g[b] = word;
                    }
                }
            }
            if (rk == 0 && lane == 0) {
                int clamped = 0;
                for (int w = 0; w < G; ++w) clamped |= reinterpret_cast<const int *>(part + w * kWPart)[kML + 2];
                // the highest of the scores just written and its slot (the new row's own score is not among them)
                float gbest = -INFINITY;
                int gslot = -1;
                for (int w = 0; w < G; ++w) {
                    const float wv = part[w * kWPart + kML + 3];
                    const int ws = reinterpret_cast<const int *>(part + w * kWPart)[kML + 4];
                    if (wv > gbest) { gbest = wv; gslot = ws; }
                    else if (wv == gbest && wv > -INFINITY) gslot = -1;
                }
                if (new_cand) gslot = -1;
                // rows that moved were scored at their new slots, but the mask above is by old slot: no note then
                *reinterpret_cast<int4 *>(c.carry + (size_t)sid * 4) = make_int4(okay && ns == 0 ? 1 : 0, p_next, clamped, gslot + 1);
            }

            // ---- the update itself, by the first warp ---------------------------------------------------
            if (okay && rk == 0) {
                for (int i = 0; i < ns; ++i) {   // survivors move down: K and V rows in pieces of 16 bytes
                    const int kChunks = g_rs / 8;   // 16-byte pieces of a pool row
                    const int row = surv[i], dst = holes[i];
                    size_t so = row_offset(c, pt, row), go = row_offset(c, pt, dst);
                    if (lane < 2 * kChunks) {
                        __nv_bfloat16 *pool = lane < kChunks ? c.k_pool : c.v_pool;
                        const int ch = lane < kChunks ? lane : lane - kChunks;
                        reinterpret_cast<uint4 *>(pool + go)[ch] = reinterpret_cast<const uint4 *>(pool + so)[ch];
                    }
                    if (lane == 0) {
                        c.pos[(size_t)sid * c.max_rows + dst] = c.pos[(size_t)sid * c.max_rows + row];
                        c.inv_norm[(size_t)sid * c.max_rows + dst] = inv_s[row];
                    }
                }
                if (new_cand) {   // the new row's own score for the next step
                    float dot = 0.f;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) dot = fmaf(bf16_hi(vn[j]), sv1[j], fmaf(bf16_lo(vn[j]), sv0[j], dot));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    if (lane == 0) scores[last_hole] = (inv_row_new * dot - inv_row_new * inv_row_new * ss_new) * rden + 0.0f;
                }
                {   // the new row, from the registers that hold it since the prologue (zero beyond d)
                    if (need > have) {   // the page table grew: take the new entries
                        for (int pg = have + lane; pg < need; pg += 32) pt_s[pg] = pt[pg];
                        __syncwarp();
                    }
                    const size_t off = row_offset(c, pt_s, last_hole);
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        if (64 * j + 2 * lane < g_rs) {
                            *reinterpret_cast<uint32_t *>(c.k_pool + off + 64 * j + 2 * lane) = kn[j];
                            *reinterpret_cast<uint32_t *>(c.v_pool + off + 64 * j + 2 * lane) = vn[j];
                        }
                    }
                }
                if (lane == 0) {
                    c.pos[(size_t)sid * c.max_rows + last_hole] = a.cur_pos;
                    c.inv_norm[(size_t)sid * c.max_rows + last_hole] = inv_row_new;
                    if (need < have) resize_pages(c, pt, have, need);
                    c.n_live[sid] = n2;
                }
            }
        }
        if (local + stride < n_local) group_sync();   // the stream's shared buffers are free for the next one
    }
}

// ---- host side ------------------------------------------------------------
// Tile layouts the kernel is compiled for: 64-element rows (32-row stages), 104- and 128-element rows (16-row stages).
// A pool whose rows are narrower than 64 (or 128) elements is served by the 64- (or 128-) element layout: the tensor
// copies read the pool's rows and fill the rest of a tile row with zeros.  104-element rows keep their own layout.
bool wstep_supported(const DevCtx &c) { return c.row_stride >= 8 && c.row_stride <= 128 && c.row_stride % 8 == 0 && c.d % 2 == 0; }
static int wstep_tile_rs(const DevCtx &c) { return c.row_stride == 104 ? 104 : c.row_stride <= 64 ? 64 : 128; }
static int wstep_stage_rows(const DevCtx &c) { return wstep_tile_rs(c) == 64 ? 32 : 16; }

// Tensor maps of both pools for boxes of 1, 2, 4, .. 32 rows (128-byte swizzle for 128-byte rows, none
// otherwise).  The encoder is cuTensorMapEncodeTiled, looked up at run time so that the library links cudart only.
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
    const cuuint64_t dims[2] = {(cuuint64_t)c.row_stride, (cuuint64_t)c.n_pages * (cuuint64_t)c.page_rows};
    if (dims[1] > (1ull << 31)) return -1;
    const cuuint64_t strides[1] = {(cuuint64_t)c.row_stride * 2};
    const cuuint32_t estr[2] = {1, 1};
    for (int pool = 0; pool < 2; ++pool) {
        for (int hb = 0; hb < 6; ++hb) {
            const cuuint32_t box[2] = {(cuuint32_t)(c.row_stride == 104 ? 104 : 64), 1u << hb};   // swizzled tiles: 64 elements (128 bytes) wide
            CUtensorMap *m = pool == 0 ? &out->k[hb] : &out->v[hb];
            CUresult r = encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, pool == 0 ? (void *)c.k_pool : (void *)c.v_pool,
                                dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                c.row_stride == 104 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return -1;
        }
    }
    return 0;
}

typedef void (*wstep_fn)(DevCtx, WStepArgs, WStepMaps);

// the instantiation for a row layout, a CTA size and a flavour (nullptr: not compiled)
static wstep_fn wstep_variant(int row_stride, int warps, bool fused)
{
    if (row_stride == 64) {
        if (warps <= 8) return fused ? wstep_kernel<true, 8, 64, 32> : wstep_kernel<false, 8, 64, 32>;
        if (warps <= 10) return fused ? wstep_kernel<true, 10, 64, 32> : wstep_kernel<false, 10, 64, 32>;   // 5 streams x 2 warps, the LlamaGen-XL shape
        if (warps <= 12) return fused ? wstep_kernel<true, 12, 64, 32> : wstep_kernel<false, 12, 64, 32>;   // 6 streams x 2 warps: 168 registers per thread
        return fused ? wstep_kernel<true, 16, 64, 32> : wstep_kernel<false, 16, 64, 32>;
    }
    if (row_stride == 104) {
        if (warps <= 8) return fused ? wstep_kernel<true, 8, 104, 16> : wstep_kernel<false, 8, 104, 16>;
        if (warps <= kWWideMaxWarps) return fused ? wstep_kernel<true, kWWideMaxWarps, 104, 16> : wstep_kernel<false, kWWideMaxWarps, 104, 16>;
    }
    if (row_stride == 128) {
        if (warps <= 8) return fused ? wstep_kernel<true, 8, 128, 16> : wstep_kernel<false, 8, 128, 16>;
        if (warps <= kWWideMaxWarps && !fused) return wstep_kernel<false, kWWideMaxWarps, 128, 16>;   // the fused step would spill at ten warps
    }
    return nullptr;
}

cudaError_t configure_wstep_kernel(const DevCtx &c)
{
    cudaError_t e = cudaSuccess;
    for (int warps : {8, 10, 12, 16})
        for (int fused = 0; fused < 2 && e == cudaSuccess; ++fused) {
            wstep_fn f = wstep_variant(wstep_tile_rs(c), warps, fused != 0);
            if (f) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kWSmemLimit);
        }
    return e;
}

// Groups per CTA, warps per group and ring depth per warp.  As many groups as the SM has streams to
// serve (at most 8), then as many warps per group as shared memory and the 16 warps of a CTA allow
// with a ring of at least two stages each.  group_warps > 0 fixes the group size.
WStepPlan plan_wstep(const DevCtx &c, bool fused, int sm_count, int max_depth, int group_warps, int n_run)
{
    WStepPlan p = {};
    if (!wstep_supported(c)) return p;
    const int rs = wstep_tile_rs(c), tr = wstep_stage_rows(c), stage_bytes = w_stage_bytes(rs, tr);
    const int max_warps = rs == 64 ? 16 : (rs == 128 && fused) ? 8 : kWWideMaxWarps;   // the wide-row kernels need more registers per thread
    const int n_streams = c.S * (n_run < 1 ? 1 : n_run);   // streams one launch serves
    int groups = (n_streams + sm_count - 1) / sm_count;
    groups = groups < 1 ? 1 : groups > kScratchGroups ? kScratchGroups : groups;
    const int cap = max_depth > 0 && max_depth < kWMaxDepth ? max_depth : kWMaxDepth;
    if (n_streams > 5 * sm_count + sm_count / 2 && group_warps <= 0) {
        // A launch with more streams than any grouping can hold at once (several layers, or a large batch): what
        // counts is how many streams an SM keeps in flight and how fast each moves.  Measured on the XL shape (us
        // per layer-step): 5 streams x 2 warps 19.2, 8 x 1 20.8, 3 x 4 22.9.  So: two warps per stream, as many
        // streams as shared memory allows with rings of two stages; one warp per stream if even one pair does not fit.
        for (int G = 2; G >= 1 && group_warps <= 0; --G)
            for (int gr = groups; gr >= 1; --gr) {
                if (gr * G > max_warps) continue;
                const uint32_t fixed = w_layout(c.max_rows, c.max_pages, c.mask_words, 0, G, fused, rs, tr).per_group;
                if ((long long)kWSmemLimit / gr - fixed >= 2ll * G * stage_bytes) { groups = gr; group_warps = G; break; }
            }
    }
    for (; groups >= 1; --groups) {
        for (int G = group_warps > 0 ? group_warps : kWMaxGroupWarps; G >= 1; --G) {
            if (G > kWMaxGroupWarps || groups * G > max_warps) { if (group_warps > 0) break; continue; }
            const uint32_t fixed = w_layout(c.max_rows, c.max_pages, c.mask_words, 0, G, fused, rs, tr).per_group;
            const long long room = (long long)kWSmemLimit / groups - fixed;
            int depth = room > 0 ? (int)(room / ((long long)G * stage_bytes)) : 0;
            depth = depth > cap ? cap : depth;
            if (depth >= 2 || (depth >= 1 && G == 1 && groups == 1)) {
                WLayout L = w_layout(c.max_rows, c.max_pages, c.mask_words, depth, G, fused, rs, tr);
                p.n_groups = groups; p.group_warps = G; p.depth = depth;
                p.l2_ahead = fused ? 1 : 0;   // measured: with the ring this makes a three-deep pipeline; deeper is slower
                p.smem_bytes = (size_t)L.per_group * groups;
                p.grid = n_streams < sm_count ? n_streams : sm_count;   // spread the streams over every SM
                if (p.grid > kScratchCtas) p.grid = kScratchCtas;
                return p;
            }
            if (group_warps > 0) break;
        }
    }
    return p;
}

cudaError_t launch_wstep(const DevCtx &c, const WStepPlan &plan, const WStepMaps &maps, bool fused, int layer, int cur_pos,
                         int budget_rows, const void *q, const void *k_new, const void *v_new, void *out_bf16,
                         float *out_f32, cudaStream_t st, bool have_svec, bool early_state, bool use_note, int next_layer, int next_tiles,
                         int n_run, const int *in_ready, int in_epoch)
{
    WStepArgs a;
    a.in_ready = in_ready; a.in_epoch = in_epoch;
    a.n_run = n_run < 1 ? 1 : n_run;
    a.next_layer = next_layer; a.next_tiles = next_tiles;
    a.have_svec = have_svec ? 1 : 0;
    a.use_note = have_svec && use_note ? 1 : 0;
    a.early_state = early_state ? 1 : 0;
    a.layer = layer; a.cur_pos = cur_pos; a.budget_rows = budget_rows; a.depth = plan.depth;
    a.group_warps = plan.group_warps; a.n_groups = plan.n_groups; a.l2_ahead = plan.l2_ahead;
    a.g_magic = (uint32_t)((1ull << 32) / (uint32_t)plan.group_warps) + 1u;   // exact for x < 2^16 at least (group_warps <= 4)
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    a.scratch = c.wscratch;
    const int warps = plan.n_groups * plan.group_warps, threads = warps * 32;
    wstep_fn kern = wstep_variant(wstep_tile_rs(c), warps, fused);
    if (!kern) return cudaErrorInvalidConfiguration;
    // launched so that its set-up overlaps the tail of the kernel before it in the stream (the kernel
    // itself waits for that kernel's completion before it reads or writes global memory)
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid); cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = plan.smem_bytes; cfg.stream = st;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, c, a, maps);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace adsa
