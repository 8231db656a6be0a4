// Entering the condition into an empty cache: dense causal attention over its rows (Section 4.2: while
// the cache has room the method is plain attention), and the two-dimensional rotary embedding that sits on
// Q and K (Section 4.1).
//
// The attention is a real contraction (n x n x d per stream, n = 120 text rows for the LlamaGen shapes), so it
// runs on tensor cores; it is also tiny and runs once per generation (against H*W decode steps), which is why
// it uses plain mma.sync tiles of 16 query rows per warp and 64 cached rows per shared-memory chunk: a
// tcgen05 pipeline (tensor-memory allocation, descriptors, a 128-row M tile for 120 rows) would cost more to
// set up than the 3.7 MFLOP of a stream take to compute.
#include <float.h>
#include <math_constants.h>

#include "adsa_dev.cuh"
#include "adsa_launch.h"

namespace adsa {

namespace {

constexpr int kPfThreads = 256, kPfWarps = kPfThreads / 32;
constexpr int kPfChunk = 64;                 // cached rows per shared-memory chunk
constexpr int kPfMaxKS = 16;                 // 16-element steps over a row: head_dim <= 256

__device__ __forceinline__ void pf_ldsm(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void pf_ldsm_t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void pf_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pf_pack(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float pf_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float pf_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// One block per stream.  q, k, v, out: [S][n][d] for the layer.  A warp owns 16 query rows at a time; the K
// and V rows come through shared memory in chunks of 64, with a pitch of 16*KS + 8 elements so that the
// eight rows of an ldmatrix fall on different banks.  KS = 16-element steps over a row.
template <int KS>
__global__ void __launch_bounds__(kPfThreads)
prefill_attn_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                    __nv_bfloat16 *__restrict__ out_bf16, float *__restrict__ out_f32, int n, int d, float scale_log2e)
{
    constexpr int PITCH = 16 * KS + 8;                      // elements
    extern __shared__ __align__(16) unsigned char pf_smem[];
    __nv_bfloat16 *Ks = reinterpret_cast<__nv_bfloat16 *>(pf_smem), *Vs = Ks + kPfChunk * PITCH;
    const int sid = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3, mi = lane >> 3, lr = lane & 7;
    const size_t base = (size_t)sid * n * d;
    const uint32_t ks_u32 = (uint32_t)__cvta_generic_to_shared(Ks), vs_u32 = (uint32_t)__cvta_generic_to_shared(Vs);

    for (int q0 = 0; q0 < n; q0 += 16 * kPfWarps) {         // 128 query rows at a time, 16 per warp
        const int qr = q0 + 16 * warp;                      // this warp's first query row
        // Q as the A operand: rows qr + g and qr + g + 8, elements 16*ks + 2t, + 1 and + 8, + 9
        uint32_t qa[KS][4];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = qr + g + (i & 1) * 8, col = 16 * ks + 2 * t + (i >> 1) * 8;
                qa[ks][i] = row < n && col < d ? *reinterpret_cast<const uint32_t *>(q + base + (size_t)row * d + col) : 0u;
            }
        }
        float o[2 * KS][4], m_run[2] = {-FLT_MAX, -FLT_MAX}, l_run[2] = {0.f, 0.f};
#pragma unroll
        for (int nb = 0; nb < 2 * KS; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }
        const int kv_end = min(n, q0 + 16 * kPfWarps);      // causal: no query of this round sees beyond its own row
        for (int c0 = 0; c0 < kv_end; c0 += kPfChunk) {
            __syncthreads();                                // the previous chunk has been read by every warp
            for (int i = threadIdx.x; i < kPfChunk * (PITCH / 8); i += kPfThreads) {   // 16-byte pieces, zero beyond n and d
                const int r = i / (PITCH / 8), pc = i % (PITCH / 8), row = c0 + r;
                uint4 kk = make_uint4(0u, 0u, 0u, 0u), vv = kk;
                if (row < n && pc * 8 < d) {
                    if (pc * 8 + 8 <= d && ((reinterpret_cast<uintptr_t>(k + base + (size_t)row * d + pc * 8) |
                                             reinterpret_cast<uintptr_t>(v + base + (size_t)row * d + pc * 8)) & 15) == 0) {
                        kk = *reinterpret_cast<const uint4 *>(k + base + (size_t)row * d + pc * 8);
                        vv = *reinterpret_cast<const uint4 *>(v + base + (size_t)row * d + pc * 8);
                    } else {                                // a ragged or unaligned piece: element by element
                        unsigned short kb[8] = {0, 0, 0, 0, 0, 0, 0, 0}, vb[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                        for (int e = 0; e < 8 && pc * 8 + e < d; ++e) {
                            kb[e] = __bfloat16_as_ushort(k[base + (size_t)row * d + pc * 8 + e]);
                            vb[e] = __bfloat16_as_ushort(v[base + (size_t)row * d + pc * 8 + e]);
                        }
                        kk = make_uint4(kb[0] | (kb[1] << 16), kb[2] | (kb[3] << 16), kb[4] | (kb[5] << 16), kb[6] | (kb[7] << 16));
                        vv = make_uint4(vb[0] | (vb[1] << 16), vb[2] | (vb[3] << 16), vb[4] | (vb[5] << 16), vb[6] | (vb[7] << 16));
                    }
                }
                *reinterpret_cast<uint4 *>(Ks + r * PITCH + pc * 8) = kk;
                *reinterpret_cast<uint4 *>(Vs + r * PITCH + pc * 8) = vv;
            }
            __syncthreads();
            if (qr >= n || c0 > qr + 15) continue;          // nothing of this chunk is visible to the warp's rows
            // S = Q.K^T for 16 query rows x 64 cached rows: eight 8-column blocks
            float s[8][4];
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) { s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f; }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {            // a pair of 8-row blocks of K per ldmatrix
                    uint32_t kf[4];
                    pf_ldsm(ks_u32 + (uint32_t)(((np * 16 + (mi >> 1) * 8 + lr) * PITCH + ks * 16 + (mi & 1) * 8) * 2), kf);
                    pf_mma(s[2 * np], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kf[0], kf[1]);
                    pf_mma(s[2 * np + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kf[2], kf[3]);
                }
            }
            // causal mask, online softmax for rows qr + g (h = 0) and qr + g + 8 (h = 1)
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = qr + g + (i >> 1) * 8, col = c0 + nb * 8 + 2 * t + (i & 1);
                    s[nb][i] = col <= row && col < n ? s[nb][i] * scale_log2e : -INFINITY;
                    mx[i >> 1] = fmaxf(mx[i >> 1], s[nb][i]);
                }
            }
            float corr[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
                const float m_new = fmaxf(m_run[h], mx[h]);   // finite: the chunk holds column c0 <= row for every row that exists
                corr[h] = exp2f(m_run[h] - m_new);
                m_run[h] = m_new;
                l_run[h] *= corr[h];
            }
#pragma unroll
            for (int nb = 0; nb < 2 * KS; ++nb) { o[nb][0] *= corr[0]; o[nb][1] *= corr[0]; o[nb][2] *= corr[1]; o[nb][3] *= corr[1]; }
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    s[nb][i] = m_run[i >> 1] == -FLT_MAX ? 0.f : exp2f(s[nb][i] - m_run[i >> 1]);
                    l_run[i >> 1] += s[nb][i];
                }
            }
            // O += P.V: P as the A operand in two bf16 parts (hi + lo), V^T blocks through transposing ldmatrix
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {                // 16 cached rows per k-step
                uint32_t ph[4], pl[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float a = s[2 * kk + (i >> 1)][(i & 1) * 2], b = s[2 * kk + (i >> 1)][(i & 1) * 2 + 1];
                    ph[i] = pf_pack(a, b);
                    pl[i] = pf_pack(a - pf_lo(ph[i]), b - pf_hi(ph[i]));
                }
#pragma unroll
                for (int dp = 0; dp < KS; ++dp) {           // a pair of 8-element blocks of the head dimension per ldmatrix
                    uint32_t vf[4];
                    pf_ldsm_t(vs_u32 + (uint32_t)(((kk * 16 + (mi & 1) * 8 + lr) * PITCH + dp * 16 + (mi >> 1) * 8) * 2), vf);
                    pf_mma(o[2 * dp], ph[0], ph[1], ph[2], ph[3], vf[0], vf[1]);
                    pf_mma(o[2 * dp], pl[0], pl[1], pl[2], pl[3], vf[0], vf[1]);
                    pf_mma(o[2 * dp + 1], ph[0], ph[1], ph[2], ph[3], vf[2], vf[3]);
                    pf_mma(o[2 * dp + 1], pl[0], pl[1], pl[2], pl[3], vf[2], vf[3]);
                }
            }
        }
        // rows' sums over the four lanes that share them, then the output
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
            l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
        }
#pragma unroll
        for (int nb = 0; nb < 2 * KS; ++nb) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int row = qr + g + h * 8, col = nb * 8 + 2 * t;
                if (row < n && col < d) {
                    const float a = o[nb][2 * h] / l_run[h], b = o[nb][2 * h + 1] / l_run[h];
                    if (out_f32) { out_f32[base + (size_t)row * d + col] = a; if (col + 1 < d) out_f32[base + (size_t)row * d + col + 1] = b; }
                    if (out_bf16) {
                        out_bf16[base + (size_t)row * d + col] = __float2bfloat16_rn(a);
                        if (col + 1 < d) out_bf16[base + (size_t)row * d + col + 1] = __float2bfloat16_rn(b);
                    }
                }
            }
        }
    }
}

// x: [n][d] bf16, rotated in place; pos: [n] context positions.  One thread per pair of elements.
__global__ void rope_2d_kernel(__nv_bfloat16 *x, const int32_t *pos, long long n, int d, int n_text, int grid_w, float log2_base)
{
    const int quarter = d / 4, half = d / 2;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n * half; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / half;
        const int pr = (int)(i - r * half);
        const int cell = pos[r] - n_text;
        if (cell < 0) continue;                             // the text condition is not rotated
        const int index = pr < quarter ? cell / grid_w : cell % grid_w;
        const float angle = (float)index * exp2f(-log2_base * (float)(pr % quarter) / (float)quarter);
        float sn, cs;
        sincosf(angle, &sn, &cs);
        uint32_t *p2 = reinterpret_cast<uint32_t *>(x + r * d) + pr;
        const uint32_t w = *p2;
        const float a = pf_lo(w), b = pf_hi(w);
        *p2 = pf_pack(a * cs - b * sn, a * sn + b * cs);
    }
}

template <int KS>
cudaError_t launch_prefill_ks(const DevCtx &c, const void *q, const void *k, const void *v, void *out_bf16, float *out_f32,
                              int n_rows, cudaStream_t st)
{
    const size_t smem = (size_t)2 * kPfChunk * (16 * KS + 8) * sizeof(__nv_bfloat16);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(prefill_attn_kernel<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    prefill_attn_kernel<KS><<<c.S, kPfThreads, smem, st>>>((const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v,
                                                           (__nv_bfloat16 *)out_bf16, out_f32, n_rows, c.d, c.scale_log2e);
    return cudaGetLastError();
}

}  // namespace

// q, k, v, out: [S][n_rows][d] of one layer
cudaError_t launch_prefill_attn(const DevCtx &c, const void *q, const void *k, const void *v, void *out_bf16, float *out_f32,
                                int n_rows, cudaStream_t st)
{
    const int ks = (c.d + 15) / 16;
    if (ks <= 2) return launch_prefill_ks<2>(c, q, k, v, out_bf16, out_f32, n_rows, st);
    if (ks <= 4) return launch_prefill_ks<4>(c, q, k, v, out_bf16, out_f32, n_rows, st);
    if (ks <= 7) return launch_prefill_ks<7>(c, q, k, v, out_bf16, out_f32, n_rows, st);
    if (ks <= 8) return launch_prefill_ks<8>(c, q, k, v, out_bf16, out_f32, n_rows, st);
    return launch_prefill_ks<kPfMaxKS>(c, q, k, v, out_bf16, out_f32, n_rows, st);
}

cudaError_t launch_rope_2d(const DevCtx &c, void *x, const int32_t *pos, long long n_rows, float base, cudaStream_t st)
{
    const long long work = n_rows * (c.d / 2);
    const int blocks = (int)(work < 256 ? 1 : work / 256 > 4096 ? 4096 : (work + 255) / 256);
    rope_2d_kernel<<<blocks, 256, 0, st>>>((__nv_bfloat16 *)x, pos, n_rows, c.d, c.n_text, c.grid_w, log2f(base));
    return cudaGetLastError();
}

}  // namespace adsa
