// The host model's element-wise and sampling steps around the attention (Section 5 integrates the method with a
// LlamaGen decoder): root-mean-square normalisation, the gated activation of the feed-forward block, and
// classifier-free guidance + top-k + inverse-CDF sampling of the next image token.  None of them has state: plain
// C-ABI calls on caller-owned device buffers, no context, no workspace.  The projections between them are plain
// GEMMs and are left to the caller's BLAS.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "adsa_dev.cuh"

namespace adsa {

__device__ __forceinline__ void unpack8_bf16(uint4 r, float (&f)[8])
{
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&p);
}

// ---- y = x / sqrt(mean(x^2) + eps) * w: one warp per row, 16-byte pieces ----------------------------------------
constexpr int kNormWarps = 4;
__global__ void __launch_bounds__(kNormWarps * 32)
rmsnorm_kernel(const __nv_bfloat16 *x, const __nv_bfloat16 *w, __nv_bfloat16 *out, long long rows, int dim, float eps)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kNormWarps + (threadIdx.x >> 5);
    if (row >= rows) return;
    const uint4 *xr = reinterpret_cast<const uint4 *>(x + row * dim);
    const uint4 *wr = reinterpret_cast<const uint4 *>(w);
    uint4 *orow = reinterpret_cast<uint4 *>(out + row * dim);
    const int pieces = dim / 8;
    float ss = 0.f;
    for (int p = lane; p < pieces; p += 32) {
        float f[8];
        unpack8_bf16(xr[p], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float inv = rsqrtf(ss / (float)dim + eps);
    for (int p = lane; p < pieces; p += 32) {   // the row is read again (it sits in L1 by now)
        float f[8], g[8];
        unpack8_bf16(xr[p], f);
        unpack8_bf16(wr[p], g);
        uint4 r;
        r.x = pack2_bf16(f[0] * inv * g[0], f[1] * inv * g[1]);
        r.y = pack2_bf16(f[2] * inv * g[2], f[3] * inv * g[3]);
        r.z = pack2_bf16(f[4] * inv * g[4], f[5] * inv * g[5]);
        r.w = pack2_bf16(f[6] * inv * g[6], f[7] * inv * g[7]);
        orow[p] = r;
    }
}

// ---- out = silu(gate) * up ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
swiglu_kernel(const __nv_bfloat16 *gate, const __nv_bfloat16 *up, __nv_bfloat16 *out, long long rows, int hidden, long long ld_in)
{
    const int per_row = hidden / 8;
    const long long total = rows * per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / per_row;
        const int p = (int)(i - r * per_row);
        float g[8], u[8];
        unpack8_bf16(reinterpret_cast<const uint4 *>(gate + r * ld_in)[p], g);
        unpack8_bf16(reinterpret_cast<const uint4 *>(up + r * ld_in)[p], u);
        float y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) y[e] = g[e] / (1.0f + __expf(-g[e])) * u[e];
        uint4 o;
        o.x = pack2_bf16(y[0], y[1]); o.y = pack2_bf16(y[2], y[3]); o.z = pack2_bf16(y[4], y[5]); o.w = pack2_bf16(y[6], y[7]);
        reinterpret_cast<uint4 *>(out + r * (long long)hidden)[p] = o;
    }
}

// ---- guidance, top-k, sampling: one block per image ----------------------------------------------------------------
constexpr int kSampleThreads = 1024;
constexpr int kSampleMaxItems = 32;   // consecutive token ids per thread: vocabularies up to 32768

// order-preserving map of a float onto unsigned integers (larger float, larger key)
__device__ __forceinline__ uint32_t float_key(float f)
{
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

template <int kSampleItems>   // ids per thread the kernel is compiled for (the vocabulary fits kSampleThreads * kSampleItems)
__global__ void __launch_bounds__(kSampleThreads, 1)
cfg_sample_kernel(const __nv_bfloat16 *logits, int n_images, int vocab, float scale, int top_k, float inv_temperature,
                  const float *uniforms, int32_t *tokens)
{
    __shared__ unsigned int hist[256];
    __shared__ float warp_f[32];
    __shared__ int warp_i[32];
    __shared__ unsigned int s_prefix, s_need;
    __shared__ float s_total;
    __shared__ int s_first, s_last;
    const int img = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const __nv_bfloat16 *lc = logits + (size_t)img * vocab, *lu = logits + (size_t)(n_images + img) * vocab;
    const int per = (vocab + kSampleThreads - 1) / kSampleThreads;   // ids per thread, <= kSampleItems
    const int id0 = tid * per;
    // mixed logits of this thread's ids (uncond + scale * (cond - uncond)), and their keys
    float mixed[kSampleItems];
#pragma unroll
    for (int i = 0; i < kSampleItems; ++i) {
        const int id = id0 + i;
        mixed[i] = -INFINITY;
        if (i < per && id < vocab) {
            const float c = __bfloat162float(lc[id]), u = __bfloat162float(lu[id]);
            mixed[i] = fmaf(scale, c - u, u);
        }
    }
    // ---- the key of the top_k-th largest logit: most significant byte first ----
    if (tid == 0) { s_prefix = 0u; s_need = (unsigned int)top_k; s_first = 0x7fffffff; s_last = -1; }
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned int prefix = s_prefix, mask = shift == 24 ? 0u : 0xffffffffu << (shift + 8);
#pragma unroll
        for (int i = 0; i < kSampleItems; ++i) {
            if (i < per && id0 + i < vocab) {
                const uint32_t k = float_key(mixed[i]);
                if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1u);
            }
        }
        __syncthreads();
        if (tid == 0) {   // walk the bins from the top until `need` keys are covered
            unsigned int need = s_need, b = 255u;
            for (;; --b) {
                if (hist[b] >= need || b == 0u) break;
                need -= hist[b];
            }
            s_prefix = prefix | (b << shift);
            s_need = need;
        }
        __syncthreads();
    }
    const uint32_t thr = s_prefix;          // key of the top_k-th largest logit
    const int need_equal = (int)s_need;     // how many of the logits equal to it are kept: the lowest ids
    // ---- rank of every equal logit in id order: count per thread, scan over the threads ----
    int n_eq = 0;
#pragma unroll
    for (int i = 0; i < kSampleItems; ++i)
        if (i < per && id0 + i < vocab && float_key(mixed[i]) == thr) ++n_eq;
    int incl = n_eq;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) warp_i[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int v = warp_i[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += t; }
        warp_i[lane] = v;
    }
    __syncthreads();
    const int eq_rank0 = incl - n_eq + (warp > 0 ? warp_i[warp - 1] : 0);   // equal logits before this thread's first id
    // whether id0 + i is kept (bit i): above the threshold, or one of the first need_equal logits equal to it
    uint32_t kept_bits = 0u;
    {
        int eq_rank = eq_rank0;
#pragma unroll
        for (int i = 0; i < kSampleItems; ++i) {
            if (i < per && id0 + i < vocab) {
                const uint32_t k = float_key(mixed[i]);
                bool kept = k > thr;
                if (k == thr) { kept = eq_rank < need_equal; ++eq_rank; }
                if (kept) kept_bits |= 1u << i;
            }
        }
    }
    // ---- the largest logit (always kept) ----
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < kSampleItems; ++i) mx = fmaxf(mx, mixed[i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) warp_f[warp] = mx;
    __syncthreads();
    mx = warp_f[0];
    for (int w = 1; w < kSampleThreads / 32; ++w) mx = fmaxf(mx, warp_f[w]);
    __syncthreads();
    // ---- weights of the kept ids, their running sum in id order ----
    float local = 0.f;
#pragma unroll
    for (int i = 0; i < kSampleItems; ++i)
        if ((kept_bits >> i) & 1u) local += __expf((mixed[i] - mx) * inv_temperature);
    const int last_kept = kept_bits ? id0 + 31 - __clz((int)kept_bits) : -1;
    float run = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const float t = __shfl_up_sync(0xffffffffu, run, o); if (lane >= o) run += t; }
    if (lane == 31) warp_f[warp] = run;
    __syncthreads();
    if (warp == 0) {
        float v = warp_f[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const float t = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += t; }
        warp_f[lane] = v;
        if (lane == 31) s_total = v;
    }
    __syncthreads();
    float before = run - local + (warp > 0 ? warp_f[warp - 1] : 0.f);   // sum over the ids before this thread's first
    const float target = uniforms[img] * s_total;
    // the first kept id at which the running sum reaches the target; no such id (rounding at u close to 1): the last kept one
    int first = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kSampleItems; ++i) {
        if ((kept_bits >> i) & 1u) {
            before += __expf((mixed[i] - mx) * inv_temperature);   // (the same values in the same order as above)
            if (before >= target && first == 0x7fffffff) first = id0 + i;
        }
    }
    if (first != 0x7fffffff) atomicMin(&s_first, first);
    if (last_kept >= 0) atomicMax(&s_last, last_kept);
    __syncthreads();
    if (tid == 0) tokens[img] = s_first != 0x7fffffff ? s_first : s_last;
}

}  // namespace adsa

extern "C" {

int adsa_rmsnorm(const void *x, const void *w, void *out, long long rows, int dim, float eps, adsa_stream_t stream)
{
    if (!x || !w || !out || rows < 0 || dim < 8 || dim % 8 || !(eps >= 0.f)) return ADSA_EINVAL;
    if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)out) & 15u) return ADSA_EINVAL;
    if (rows == 0) return ADSA_OK;
    const long long blocks = (rows + adsa::kNormWarps - 1) / adsa::kNormWarps;
    if (blocks > 0x7fffffffLL) return ADSA_EINVAL;
    adsa::rmsnorm_kernel<<<(unsigned)blocks, adsa::kNormWarps * 32, 0, (cudaStream_t)stream>>>(
        (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, (__nv_bfloat16 *)out, rows, dim, eps);
    return cudaGetLastError() == cudaSuccess ? ADSA_OK : ADSA_ECUDA;
}

int adsa_swiglu(const void *gate, const void *up, void *out, long long rows, int hidden, long long ld_in, adsa_stream_t stream)
{
    if (!gate || !up || !out || rows < 0 || hidden < 8 || hidden % 8 || ld_in < hidden || ld_in % 8) return ADSA_EINVAL;
    if (((uintptr_t)gate | (uintptr_t)up | (uintptr_t)out) & 15u) return ADSA_EINVAL;
    if (rows == 0) return ADSA_OK;
    const long long pieces = rows * (hidden / 8);
    long long blocks = (pieces + 255) / 256;
    if (blocks > 148 * 128) blocks = 148 * 128;
    adsa::swiglu_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16 *)gate, (const __nv_bfloat16 *)up,
                                                                              (__nv_bfloat16 *)out, rows, hidden, ld_in);
    return cudaGetLastError() == cudaSuccess ? ADSA_OK : ADSA_ECUDA;
}

int adsa_cfg_sample(const void *logits, int n_images, int vocab, float scale, int top_k, float temperature, const float *uniforms,
                    int32_t *tokens, adsa_stream_t stream)
{
    if (!logits || !uniforms || !tokens || n_images < 0 || vocab < 1 || vocab > adsa::kSampleThreads * adsa::kSampleMaxItems)
        return ADSA_EINVAL;
    if (top_k < 1 || top_k > vocab || !(temperature > 0.f)) return ADSA_EINVAL;
    if (n_images == 0) return ADSA_OK;
    const int per = (vocab + adsa::kSampleThreads - 1) / adsa::kSampleThreads;
    const __nv_bfloat16 *lg = (const __nv_bfloat16 *)logits;
    const float inv_t = 1.0f / temperature;
    cudaStream_t st = (cudaStream_t)stream;
    if (per <= 8) adsa::cfg_sample_kernel<8><<<n_images, adsa::kSampleThreads, 0, st>>>(lg, n_images, vocab, scale, top_k, inv_t, uniforms, tokens);
    else if (per <= 16) adsa::cfg_sample_kernel<16><<<n_images, adsa::kSampleThreads, 0, st>>>(lg, n_images, vocab, scale, top_k, inv_t, uniforms, tokens);
    else adsa::cfg_sample_kernel<32><<<n_images, adsa::kSampleThreads, 0, st>>>(lg, n_images, vocab, scale, top_k, inv_t, uniforms, tokens);
    return cudaGetLastError() == cudaSuccess ? ADSA_OK : ADSA_ECUDA;
}

}  // extern "C"
