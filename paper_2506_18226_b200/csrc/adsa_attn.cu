// adsa_sparse_decode_attn: softmax(q.K^T * scale).V over the retained rows of a
// stream plus the new row (Eq. 4 feeding the attention of Fig. 3).
//
// One query per private KV stream means every K/V byte is used once, by one
// dot product: 1 flop per byte, bound by HBM, no tensor-core shape.  The work
// is split over (stream, chunk of cached rows); each block streams its chunk
// with 16-byte loads, keeps an online-softmax state per lane group, merges the
// groups with warp shuffles and the warps through shared memory, and writes a
// partial (m, l, acc[d]).  The last block to finish a stream (atomic ticket, no
// waiting) folds the partials in chunk order and writes the output row.
#include <float.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"

namespace adsa {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kAttnUnroll = 4;

// merge online-softmax state (m2, l2, a2) into (m, l, a); logits are in log2 units
__device__ __forceinline__ void merge_state(float &m, float &l, float (&a)[8], float m2, float l2, const float (&a2)[8])
{
    float M = fmaxf(m, m2);
    float w1 = exp2f(m - M), w2 = exp2f(m2 - M);
    l = l * w1 + l2 * w2;
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = a[e] * w1 + a2[e] * w2;
    m = M;
}

template <int LPR>
__global__ void __launch_bounds__(kAttnThreads)
attn_kernel(DevCtx c, int layer, int chunk_rows, int n_splits, const __nv_bfloat16 *__restrict__ q,
            const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
            __nv_bfloat16 *__restrict__ out_bf16, float *__restrict__ out_f32)
{
    constexpr int RPW = 32 / LPR;            // rows a warp covers per load
    constexpr int STEP = kAttnWarps * RPW;   // rows the block covers per load
    __shared__ float sm_acc[kAttnWarps][256];
    __shared__ float sm_m[kAttnWarps], sm_l[kAttnWarps];
    __shared__ int s_last;

    const int split = blockIdx.x, local = blockIdx.y, sid = layer * c.S + local;
    const int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    const uint32_t *mask = c.keep_mask + (size_t)sid * c.mask_words;
    const int n = c.n_live[sid];
    const int c0 = split * chunk_rows, c1 = min(n, c0 + chunk_rows);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < c.row_stride;

    // this lane's 8 query elements, pre-multiplied by scale * log2(e)
    float qf[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int x = sub * 8 + e;
        qf[e] = x < c.d ? __bfloat162float(q[(size_t)local * c.d + x]) * c.scale_log2e : 0.f;
    }

    float m = -FLT_MAX, l = 0.f, acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    // the new row (always attended) is folded in by the first warp of the first chunk
    if (split == 0 && warp == 0) {
        float s = 0.f, vf[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int x = sub * 8 + e;
            float kf = x < c.d ? __bfloat162float(k_new[(size_t)local * c.d + x]) : 0.f;
            vf[e] = x < c.d ? __bfloat162float(v_new[(size_t)local * c.d + x]) : 0.f;
            s = fmaf(qf[e], kf, s);
        }
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (grp == 0) {
            m = s; l = 1.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = vf[e];
            if (c.score_mode == 1 && sub == 0) c.ml[(size_t)sid * 4 + 2] = s;
        }
    }

    for (int it0 = c0 + warp * RPW; it0 < c1; it0 += STEP * kAttnUnroll) {
        uint4 kr[kAttnUnroll], vr[kAttnUnroll];
        bool ok[kAttnUnroll];
#pragma unroll
        for (int u = 0; u < kAttnUnroll; ++u) {
            int slot = it0 + u * STEP + grp;
            ok[u] = slot < c1 && ((__ldg(mask + (slot >> 5)) >> (slot & 31)) & 1u);
            kr[u] = make_uint4(0u, 0u, 0u, 0u);
            vr[u] = make_uint4(0u, 0u, 0u, 0u);
            if (ok[u] && piece_ok) {
                size_t off = row_offset(c, pt, slot) + sub * 8;
                kr[u] = ldg128_stream(c.k_pool + off);
                vr[u] = ldg128_stream(c.v_pool + off);
            }
        }
        float s[kAttnUnroll], m_new = m;
#pragma unroll
        for (int u = 0; u < kAttnUnroll; ++u) {
            float kf[8];
            unpack8(kr[u], kf);
            float t = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) t = fmaf(qf[e], kf[e], t);
#pragma unroll
            for (int o = 1; o < LPR; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            s[u] = ok[u] ? t : -INFINITY;
            m_new = fmaxf(m_new, s[u]);
            // attention-mass mode: the row's logit is kept for the update, which turns it into this step's weight
            if (c.score_mode == 1 && ok[u] && sub == 0) c.logit[(size_t)sid * c.max_rows + it0 + u * STEP + grp] = t;
        }
        float corr = exp2f(m - m_new);
        l *= corr;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= corr;
#pragma unroll
        for (int u = 0; u < kAttnUnroll; ++u) {
            float pw = exp2f(s[u] - m_new), vf[8];
            unpack8(vr[u], vf);
            l += pw;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(pw, vf[e], acc[e]);
        }
        m = m_new;
    }

    // lane groups of a warp -> one state per warp
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o), a2[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a2[e] = __shfl_xor_sync(0xffffffffu, acc[e], o);
        merge_state(m, l, acc, m2, l2, a2);
    }
    if (grp == 0) {
        if (piece_ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sm_acc[warp][sub * 8 + e] = acc[e];
        }
        if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    }
    __syncthreads();

    // warps -> one state per block, one element per thread
    const int x = threadIdx.x;
    float M = -FLT_MAX, L = 0.f, A = 0.f;
    if (x < c.row_stride) {
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) {
            float wgt = exp2f(sm_m[w] - M);
            L = fmaf(sm_l[w], wgt, L);
            A = fmaf(sm_acc[w][x], wgt, A);
        }
    }
    if (n_splits == 1) {
        if (c.score_mode == 1 && x == 0) { c.ml[(size_t)sid * 4] = M; c.ml[(size_t)sid * 4 + 1] = L; }
        if (x < c.d) {
            float o = A / L;
            if (out_f32) out_f32[(size_t)local * c.d + x] = o;
            if (out_bf16) out_bf16[(size_t)local * c.d + x] = __float2bfloat16_rn(o);
        }
        return;
    }

    float *part = c.partials + ((size_t)local * kMaxSplits + split) * c.partial_stride;
    if (x < c.row_stride) part[x] = A;
    if (x == 0) { part[c.row_stride] = M; part[c.row_stride + 1] = L; }
    __threadfence();
    __syncthreads();
    if (x == 0) {
        int t = atomicAdd(&c.tickets[local], 1);
        s_last = (t == n_splits - 1);
        if (s_last) c.tickets[local] = 0;  // every chunk has arrived; ready for the next launch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (x < c.d) {
        const float *base = c.partials + (size_t)local * kMaxSplits * c.partial_stride;
        float Mx = -FLT_MAX;
        for (int sp = 0; sp < n_splits; ++sp) Mx = fmaxf(Mx, __ldcg(base + sp * c.partial_stride + c.row_stride));
        float Lx = 0.f, Ax = 0.f;
        for (int sp = 0; sp < n_splits; ++sp) {
            const float *ps = base + sp * c.partial_stride;
            float wgt = exp2f(__ldcg(ps + c.row_stride) - Mx);
            Lx = fmaf(__ldcg(ps + c.row_stride + 1), wgt, Lx);
            Ax = fmaf(__ldcg(ps + x), wgt, Ax);
        }
        if (c.score_mode == 1 && x == 0) { c.ml[(size_t)sid * 4] = Mx; c.ml[(size_t)sid * 4 + 1] = Lx; }
        float o = Ax / Lx;
        if (out_f32) out_f32[(size_t)local * c.d + x] = o;
        if (out_bf16) out_bf16[(size_t)local * c.d + x] = __float2bfloat16_rn(o);
    }
}

cudaError_t launch_attn(const DevCtx &c, const AttnPlan &plan, int layer, int cur_pos, const void *q,
                        const void *k_new, const void *v_new, void *out_bf16, float *out_f32, cudaStream_t st)
{
    (void)cur_pos;
    dim3 grid(plan.n_splits, c.S);
    const __nv_bfloat16 *qb = (const __nv_bfloat16 *)q, *kb = (const __nv_bfloat16 *)k_new,
                        *vb = (const __nv_bfloat16 *)v_new;
    __nv_bfloat16 *ob = (__nv_bfloat16 *)out_bf16;
    int pieces = c.row_stride / 8;
    if (pieces <= 4)
        attn_kernel<4><<<grid, kAttnThreads, 0, st>>>(c, layer, plan.chunk_rows, plan.n_splits, qb, kb, vb, ob, out_f32);
    else if (pieces <= 8)
        attn_kernel<8><<<grid, kAttnThreads, 0, st>>>(c, layer, plan.chunk_rows, plan.n_splits, qb, kb, vb, ob, out_f32);
    else if (pieces <= 16)
        attn_kernel<16><<<grid, kAttnThreads, 0, st>>>(c, layer, plan.chunk_rows, plan.n_splits, qb, kb, vb, ob, out_f32);
    else
        attn_kernel<32><<<grid, kAttnThreads, 0, st>>>(c, layer, plan.chunk_rows, plan.n_splits, qb, kb, vb, ob, out_f32);
    return cudaGetLastError();
}

}  // namespace adsa
