// adsa_score (Eq. 1-2 through the row-sum identity) and adsa_select (Eq. 3 plus
// the always-kept prefix and local window).  One block per stream: a stream's
// candidate set is at most a few thousand rows, so its scores, keys and the
// selection state fit in one SM's shared memory and no inter-block step exists.
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"
#include "adsa_select.cuh"

namespace adsa {

constexpr int kSSThreads = 256;
constexpr int kSSWarps = kSSThreads / 32;

// ---------------------------------------------------------------------------
// Eq. 1-2.  With u_j = v_j / max(|v_j|, eps) and s = sum_{j in P} u_j,
//   sum_{j != i} cos(v_i, v_j) = u_i . s - u_i . u_i,
// so S_i = (u_i . s - u_i . u_i) / (p - 1): two sweeps over the V rows of the
// previous region P (the second one normally served by L2) instead of the
// p^2 pairs of the definition.  u_i . u_i is computed, not assumed to be 1, so
// that a zero row scores 0 as the clamped definition says.
//
// LPR lanes share a row, 8 elements (16 bytes) each.  Summation order is fixed
// by the thread layout (strided slots per lane group, xor tree across groups,
// warps in index order), so scores are reproducible run to run.
// ---------------------------------------------------------------------------
template <int LPR>
__global__ void __launch_bounds__(kSSThreads)
score_kernel(DevCtx c, int layer, int cur_pos, float *scores_out)
{
    constexpr int RPW = 32 / LPR;
    __shared__ float s_part[kSSWarps][256];
    __shared__ float s_vec[256];
    __shared__ int s_p;
    const int local = blockIdx.x, sid = layer * c.S + local;
    const int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    const int32_t *pos = c.pos + (size_t)sid * c.max_rows;
    const float *inv_norm = c.inv_norm + (size_t)sid * c.max_rows;
    float *scores = c.scores + (size_t)sid * c.max_rows;
    if (scores_out) scores_out += (size_t)local * c.max_rows;
    const int n = c.n_live[sid];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < c.row_stride;
    if (threadIdx.x == 0) s_p = 0;
    __syncthreads();

    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    int cnt = 0;
    // U rows per lane group are requested before the first is used (positions, then rows and norms): a block holds
    // U times as many bytes in flight; the rows are still added in ascending slot order.
    constexpr int U = 4, kStep = kSSWarps * RPW;
    for (int slot0 = warp * RPW + grp; slot0 < n; slot0 += U * kStep) {   // no shuffles inside: lanes may leave early
        int ps[U];
#pragma unroll
        for (int u = 0; u < U; ++u) ps[u] = slot0 + u * kStep < n ? pos[slot0 + u * kStep] : -1;
        uint4 raw[U];
        float inv[U];
        bool prev[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int slot = slot0 + u * kStep;
            const int reg = slot < n ? region_of(c, ps[u], cur_pos) : kRegionLocal;
            if (reg == kRegionInvalid && sub == 0) set_status(c, ADSA_DEV_BAD_POSITION);
            prev[u] = reg == kRegionPrevious;
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            inv[u] = 0.f;
            if (prev[u] && piece_ok) {
                raw[u] = ldg128(c.v_pool + row_offset(c, pt, slot) + sub * 8);
                inv[u] = inv_norm[slot];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!prev[u]) continue;
            if (sub == 0) ++cnt;
            if (piece_ok) {
                float f[8];
                unpack8(raw[u], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(inv[u], f[e], acc[e]);
            }
        }
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (grp == 0 && piece_ok) {
#pragma unroll
        for (int e = 0; e < 8; ++e) s_part[warp][sub * 8 + e] = acc[e];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0 && cnt) atomicAdd(&s_p, cnt);
    __syncthreads();
    if (threadIdx.x < c.row_stride) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kSSWarps; ++w) t += s_part[w][threadIdx.x];
        s_vec[threadIdx.x] = t;
    }
    __syncthreads();
    const int p = s_p;
    float sv[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) sv[e] = piece_ok ? s_vec[sub * 8 + e] : 0.f;

    for (int sb0 = warp * RPW; sb0 < n; sb0 += U * kStep) {   // warp-uniform bounds: all lanes join the shuffles
        int ps[U];
#pragma unroll
        for (int u = 0; u < U; ++u) ps[u] = sb0 + u * kStep + grp < n ? pos[sb0 + u * kStep + grp] : -1;
        uint4 raw[U];
        float inv[U];
        int regs[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int slot = sb0 + u * kStep + grp;
            regs[u] = slot < n ? region_of(c, ps[u], cur_pos) : kRegionInvalid;
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            inv[u] = 0.f;
            if (regs[u] == kRegionPrevious) {
                if (piece_ok) raw[u] = ldg128(c.v_pool + row_offset(c, pt, slot) + sub * 8);
                if (sub == 0) inv[u] = inv_norm[slot];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (sb0 + u * kStep >= n) break;   // (warp-uniform)
            const int slot = sb0 + u * kStep + grp;
            float dot = 0.f, self = 0.f;
            if (regs[u] == kRegionPrevious && piece_ok) {
                float f[8];
                unpack8(raw[u], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], sv[e], dot); self = fmaf(f[e], f[e], self); }
            }
#pragma unroll
            for (int o = 1; o < LPR; o <<= 1) {
                dot += __shfl_xor_sync(0xffffffffu, dot, o);
                self += __shfl_xor_sync(0xffffffffu, self, o);
            }
            if (sub == 0 && slot < n) {
                float S = CUDART_NAN_F;
                if (regs[u] == kRegionPrevious) {
                    // (p-1) S_i = u_i.s - u_i.u_i; dividing (not multiplying by a reciprocal) keeps the
                    // last bit where the definition puts it; "+ 0" folds -0 into +0 for the integer ordering
                    S = p > 1 ? (inv[u] * dot - inv[u] * inv[u] * self) / (float)(p - 1) + 0.0f : 0.0f;
                }
                scores[slot] = S;
                if (scores_out) scores_out[slot] = S;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 1-2 at the granularity of a layer: a token's V rows of all heads of a batch row are one vector of
// n_heads * d elements, so u_j = v_j / |v_j| with |v_j|^2 summed over the heads, one score per (batch row,
// token), written to every head's stream.  One block per batch row; the heads' caches must hold the same
// positions slot by slot (they do when they are always stepped together; a difference raises
// ADSA_DEV_BAD_POSITION).  Same row-sum identity as above, head after head.
// Dynamic shared memory: 1/|v_j| by slot (0 = not a candidate), then s for every head.
// ---------------------------------------------------------------------------
template <int LPR>
__global__ void __launch_bounds__(kSSThreads)
score_shared_kernel(DevCtx c, int layer, int cur_pos, float *scores_out)
{
    constexpr int RPW = 32 / LPR;
    extern __shared__ float sh_f[];
    __shared__ float s_part[kSSWarps][256];
    __shared__ int s_p;
    float *invn = sh_f, *svec = sh_f + c.max_rows;
    const int H = c.n_heads, b = blockIdx.x, local0 = b * H, sid0 = layer * c.S + local0;
    const int n = c.n_live[sid0];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < c.row_stride;
    if (threadIdx.x == 0) s_p = 0;
    if (threadIdx.x < H && c.n_live[sid0 + threadIdx.x] != n) set_status(c, ADSA_DEV_BAD_POSITION);
    __syncthreads();
    // the tokens' norms over all heads, which of them are candidates, and whether the heads agree
    for (int base = 0; base < n; base += kSSThreads) {
        const int slot = base + threadIdx.x;
        bool cand = false;
        if (slot < n) {
            const int ps = c.pos[(size_t)sid0 * c.max_rows + slot];
            float ss = 0.f;
            for (int h = 0; h < H; ++h) {
                const size_t at = (size_t)(sid0 + h) * c.max_rows + slot;
                const float nr = 1.0f / c.inv_norm[at];   // the head's |v| (1e-8 for an all-zero row)
                ss = fmaf(nr, nr, ss);
                if (c.pos[at] != ps) set_status(c, ADSA_DEV_BAD_POSITION);
            }
            const int reg = region_of(c, ps, cur_pos);
            if (reg == kRegionInvalid) set_status(c, ADSA_DEV_BAD_POSITION);
            cand = reg == kRegionPrevious;
            invn[slot] = cand ? 1.0f / fmaxf(sqrtf(ss), kNormEps) : 0.f;
        }
        const unsigned bc = __ballot_sync(0xffffffffu, cand);
        if (lane == 0 && bc) atomicAdd(&s_p, __popc(bc));
    }
    __syncthreads();
    const int p = s_p;
    // s^h = sum over the candidates of v_j^h / |v_j|, for every head
    for (int h = 0; h < H; ++h) {
        const int32_t *pt = c.page_table + (size_t)(sid0 + h) * c.max_pages;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        for (int slot = warp * RPW + grp; slot < n; slot += kSSWarps * RPW) {
            const float w = invn[slot];
            if (w == 0.f || !piece_ok) continue;
            float f[8];
            unpack8(ldg128(c.v_pool + row_offset(c, pt, slot) + sub * 8), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(w, f[e], acc[e]);
        }
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
        }
        if (grp == 0 && piece_ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e) s_part[warp][sub * 8 + e] = acc[e];
        }
        __syncthreads();
        if (threadIdx.x < c.row_stride) {
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < kSSWarps; ++w) t += s_part[w][threadIdx.x];
            svec[h * c.row_stride + threadIdx.x] = t;
        }
        __syncthreads();
    }
    // S_j = (u_j . s - u_j . u_j) / (p - 1), the dot products summed over the heads
    for (int sb = warp * RPW; sb < n; sb += kSSWarps * RPW) {   // warp-uniform bounds: all lanes join the shuffles
        const int slot = sb + grp;
        const float w = slot < n ? invn[slot] : 0.f;
        float dot = 0.f, self = 0.f;
        if (w != 0.f && piece_ok) {
            for (int h = 0; h < H; ++h) {
                float f[8];
                unpack8(ldg128(c.v_pool + row_offset(c, c.page_table + (size_t)(sid0 + h) * c.max_pages, slot) + sub * 8), f);
                const float *sv = svec + h * c.row_stride + sub * 8;
#pragma unroll
                for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], sv[e], dot); self = fmaf(f[e], f[e], self); }
            }
        }
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) {
            dot += __shfl_xor_sync(0xffffffffu, dot, o);
            self += __shfl_xor_sync(0xffffffffu, self, o);
        }
        if (sub == 0 && slot < n) {
            float S = CUDART_NAN_F;
            if (w != 0.f) S = p > 1 ? (w * dot - w * w * self) / (float)(p - 1) + 0.0f : 0.0f;
            for (int h = 0; h < H; ++h) {
                c.scores[(size_t)(sid0 + h) * c.max_rows + slot] = S;
                if (scores_out) scores_out[(size_t)(local0 + h) * c.max_rows + slot] = S;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Eq. 3 plus the always-kept regions: the threshold comes from block_select, this
// kernel turns it into the keep mask, the retained / evicted lists and the counts.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kSSThreads)
select_kernel(DevCtx c, int layer, int cur_pos, int budget_rows, int32_t *sel_slots, int32_t *sel_pos,
              int32_t *evict_pos, int32_t *counts_out)
{
    extern __shared__ unsigned long long sm_keys[];  // [max_rows], then uint8 region[max_rows]
    __shared__ SelScratch s_sel;
    __shared__ int s_wk[kSSWarps], s_we[kSSWarps], s_bk, s_be;
    const int local = blockIdx.x, sid = layer * c.S + local;
    const int32_t *pos = c.pos + (size_t)sid * c.max_rows;
    const float *scores = c.scores + (size_t)sid * c.max_rows;
    uint8_t *region = reinterpret_cast<uint8_t *>(sm_keys + c.max_rows);
    const int n = c.n_live[sid];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_bk = 0; s_be = 0; }
    const SelResult sel = block_select(c, pos, scores, n, cur_pos, budget_rows, sm_keys, region, s_sel);
    const int p = sel.p, K = sel.K;

    // retained / evicted lists in ascending slot order, keep mask, counts
    uint32_t *keep_mask = c.keep_mask + (size_t)sid * c.mask_words;
    const size_t ob = (size_t)local * c.max_rows;
    for (int base = 0; base < n; base += kSSThreads) {
        int slot = base + threadIdx.x;
        bool live = slot < n, kept = false;
        if (live) {
            kept = sel.keeps(region[slot], sm_keys[slot]);
        }
        unsigned bk = __ballot_sync(0xffffffffu, kept), be = __ballot_sync(0xffffffffu, live && !kept);
        if (lane == 0) {
            s_wk[warp] = __popc(bk); s_we[warp] = __popc(be);
            if (base + warp * 32 < n) keep_mask[(base >> 5) + warp] = bk;
        }
        __syncthreads();
        int ok_ = s_bk, oe = s_be;
        for (int w = 0; w < warp; ++w) { ok_ += s_wk[w]; oe += s_we[w]; }
        unsigned below = (1u << lane) - 1u;
        if (kept) {
            int i = ok_ + __popc(bk & below);
            if (sel_slots) sel_slots[ob + i] = slot;
            if (sel_pos) sel_pos[ob + i] = pos[slot];
        } else if (live) {
            int i = oe + __popc(be & below);
            if (evict_pos) evict_pos[ob + i] = pos[slot];
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 0; w < kSSWarps; ++w) { s_bk += s_wk[w]; s_be += s_we[w]; }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int32_t *cn = c.counts + (size_t)sid * 4;
        cn[0] = p; cn[1] = s_be; cn[2] = s_bk; cn[3] = K;
        if (counts_out) { counts_out[local * 4 + 0] = p; counts_out[local * 4 + 1] = s_be;
                          counts_out[local * 4 + 2] = s_bk; counts_out[local * 4 + 3] = K; }
    }
}

// Scores carried in from the previous fused step, laid out like adsa_score's optional output:
// by slot, NaN outside the previous region.
__global__ void scores_copy_kernel(DevCtx c, int layer, int cur_pos, float *scores_out)
{
    const int local = blockIdx.x, sid = layer * c.S + local;
    const int n = c.n_live[sid];
    for (int slot = threadIdx.x; slot < n; slot += blockDim.x) {
        int reg = region_of(c, c.pos[(size_t)sid * c.max_rows + slot], cur_pos);
        scores_out[(size_t)local * c.max_rows + slot] =
            reg == kRegionPrevious ? c.scores[(size_t)sid * c.max_rows + slot] : CUDART_NAN_F;
    }
}

cudaError_t launch_scores_copy(const DevCtx &c, int layer, int cur_pos, float *scores_out, cudaStream_t st)
{
    scores_copy_kernel<<<c.S, 256, 0, st>>>(c, layer, cur_pos, scores_out);
    return cudaGetLastError();
}

// ---- host launchers -------------------------------------------------------
static int lanes_per_row(int row_stride)
{
    int pieces = row_stride / 8;
    return pieces <= 4 ? 4 : pieces <= 8 ? 8 : pieces <= 16 ? 16 : 32;
}

static size_t score_shared_smem(const DevCtx &c) { return ((size_t)c.max_rows + (size_t)c.n_heads * c.row_stride) * sizeof(float); }

cudaError_t configure_score_kernel(const DevCtx &c)
{
    if (!c.score_share || score_shared_smem(c) <= 48 * 1024) return cudaSuccess;
    const int b = (int)score_shared_smem(c);
    cudaError_t e = cudaFuncSetAttribute(score_shared_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, b);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_shared_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, b);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_shared_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, b);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(score_shared_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, b);
    return e;
}

cudaError_t launch_score(const DevCtx &c, int layer, int cur_pos, float *scores_out, cudaStream_t st)
{
    if (c.score_share) {   // one block per batch row: a token's V over all heads is one vector
        const int batch = c.S / c.n_heads;
        const size_t sm = score_shared_smem(c);
        switch (lanes_per_row(c.row_stride)) {
        case 4: score_shared_kernel<4><<<batch, kSSThreads, sm, st>>>(c, layer, cur_pos, scores_out); break;
        case 8: score_shared_kernel<8><<<batch, kSSThreads, sm, st>>>(c, layer, cur_pos, scores_out); break;
        case 16: score_shared_kernel<16><<<batch, kSSThreads, sm, st>>>(c, layer, cur_pos, scores_out); break;
        default: score_shared_kernel<32><<<batch, kSSThreads, sm, st>>>(c, layer, cur_pos, scores_out); break;
        }
        return cudaGetLastError();
    }
    switch (lanes_per_row(c.row_stride)) {
    case 4: score_kernel<4><<<c.S, kSSThreads, 0, st>>>(c, layer, cur_pos, scores_out); break;
    case 8: score_kernel<8><<<c.S, kSSThreads, 0, st>>>(c, layer, cur_pos, scores_out); break;
    case 16: score_kernel<16><<<c.S, kSSThreads, 0, st>>>(c, layer, cur_pos, scores_out); break;
    default: score_kernel<32><<<c.S, kSSThreads, 0, st>>>(c, layer, cur_pos, scores_out); break;
    }
    return cudaGetLastError();
}

size_t select_smem_bytes(const DevCtx &c) { return (size_t)c.max_rows * 9 + 16; }

cudaError_t configure_select_kernel(const DevCtx &c)
{
    size_t b = select_smem_bytes(c);
    if (b <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)b);
}

cudaError_t launch_select(const DevCtx &c, int layer, int cur_pos, int budget_rows, int32_t *sel_slots,
                          int32_t *sel_pos, int32_t *evict_pos, int32_t *counts_out, cudaStream_t st)
{
    select_kernel<<<c.S, kSSThreads, select_smem_bytes(c), st>>>(c, layer, cur_pos, budget_rows, sel_slots, sel_pos,
                                                                 evict_pos, counts_out);
    return cudaGetLastError();
}

}  // namespace adsa
