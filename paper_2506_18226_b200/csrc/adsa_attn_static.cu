// adsa_decode_attn_static: the split decode-attention kernel for callers that
// must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc (or any allocator) at the
// point where they need attention: a serving loop whose memory plan was frozen
// at start-up, a plugin interface that forbids the allocation calls, a process
// whose device memory was handed in full to a framework's pool.  Such a caller
// cannot provide the workspace a context wants either.  This entry point needs
// neither: the rows come in as plain dense tensors, and the scratch of the
// split reduction (per-chunk partial softmax states and the arrival counters)
// lives in a fixed array that is part of the library image.
//
// Every GPU that loads the library carries kStaticScratchBytes of it until the
// process exits.  All calls share it and it keeps what the last call left, so
// the counters are cleared on the stream before each launch, and two calls
// whose kernels could overlap on the GPU (different streams, different threads)
// race on it: serialise them.
#include <float.h>
#include <mutex>

#include "adsa_dev.cuh"

namespace adsa {

constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB per GPU
constexpr int kStaticMaxStreams = 4096;            // arrival counters: 16 KiB of the array
constexpr int kStaticMaxRows = 1 << 20;
constexpr int kStaticThreads = 256;
constexpr int kStaticWarps = kStaticThreads / 32;
constexpr int kStaticUnroll = 4;
constexpr int kStaticMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; kernels get the device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticAttnArgs {
    const __nv_bfloat16 *q, *k, *v, *k_new, *v_new;
    const int32_t *n_rows;
    __nv_bfloat16 *out_bf16;
    float *out_f32;
    int32_t *tickets;      // [n_streams], zero on entry
    float *partials;       // [n_streams][n_splits][row_stride + 2]
    int max_rows, d, row_stride, chunk_rows, n_splits;
    float scale_log2e;
};

__device__ __forceinline__ void fold_state(float &m, float &l, float (&a)[8], float m2, float l2, const float (&a2)[8])
{
    float M = fmaxf(m, m2);
    float w1 = exp2f(m - M), w2 = exp2f(m2 - M);
    l = l * w1 + l2 * w2;
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = a[e] * w1 + a2[e] * w2;
    m = M;
}

// grid (n_splits, n_streams).  Rows of stream s are k[s][0 .. n_rows[s]) with row_stride elements each.
template <int LPR>
__global__ void __launch_bounds__(kStaticThreads) attn_static_kernel(StaticAttnArgs a)
{
    constexpr int RPW = 32 / LPR;
    constexpr int STEP = kStaticWarps * RPW;
    __shared__ float sm_acc[kStaticWarps][256];
    __shared__ float sm_m[kStaticWarps], sm_l[kStaticWarps];
    __shared__ int s_last;

    const int split = blockIdx.x, sid = blockIdx.y;
    const int n = min(max(a.n_rows[sid], 0), a.max_rows);
    const int c0 = split * a.chunk_rows, c1 = min(n, c0 + a.chunk_rows);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const bool piece_ok = sub * 8 < a.row_stride;
    const __nv_bfloat16 *kb = a.k + (size_t)sid * a.max_rows * a.row_stride;
    const __nv_bfloat16 *vb = a.v + (size_t)sid * a.max_rows * a.row_stride;

    float qf[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int x = sub * 8 + e;
        qf[e] = x < a.d ? __bfloat162float(a.q[(size_t)sid * a.d + x]) * a.scale_log2e : 0.f;
    }
    float m = -FLT_MAX, l = 0.f, acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    if (split == 0 && warp == 0) {   // the new row, always attended
        float s = 0.f, vf[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int x = sub * 8 + e;
            float kf = x < a.d ? __bfloat162float(a.k_new[(size_t)sid * a.d + x]) : 0.f;
            vf[e] = x < a.d ? __bfloat162float(a.v_new[(size_t)sid * a.d + x]) : 0.f;
            s = fmaf(qf[e], kf, s);
        }
#pragma unroll
        for (int o = 1; o < LPR; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (grp == 0) {
            m = s; l = 1.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = vf[e];
        }
    }

    // elements past head_dim inside the last 16-byte piece are the caller's padding: masked out here
    const int valid = min(8, max(0, a.d - sub * 8));
    for (int it0 = c0 + warp * RPW; it0 < c1; it0 += STEP * kStaticUnroll) {
        uint4 kr[kStaticUnroll], vr[kStaticUnroll];
        bool ok[kStaticUnroll];
#pragma unroll
        for (int u = 0; u < kStaticUnroll; ++u) {
            int row = it0 + u * STEP + grp;
            ok[u] = row < c1;
            kr[u] = make_uint4(0u, 0u, 0u, 0u);
            vr[u] = make_uint4(0u, 0u, 0u, 0u);
            if (ok[u] && piece_ok) {
                size_t off = (size_t)row * a.row_stride + sub * 8;
                kr[u] = ldg128_stream(kb + off);
                vr[u] = ldg128_stream(vb + off);
            }
        }
        float s[kStaticUnroll], m_new = m;
#pragma unroll
        for (int u = 0; u < kStaticUnroll; ++u) {
            float kf[8];
            unpack8(kr[u], kf);
            float t = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) t = fmaf(qf[e], e < valid ? kf[e] : 0.f, t);
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
        for (int u = 0; u < kStaticUnroll; ++u) {
            float pw = exp2f(s[u] - m_new), vf[8];
            unpack8(vr[u], vf);
            l += pw;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(pw, e < valid ? vf[e] : 0.f, acc[e]);
        }
        m = m_new;
    }

#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
        float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o), a2[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) a2[e] = __shfl_xor_sync(0xffffffffu, acc[e], o);
        fold_state(m, l, acc, m2, l2, a2);
    }
    if (grp == 0) {
        if (piece_ok) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sm_acc[warp][sub * 8 + e] = acc[e];
        }
        if (sub == 0) { sm_m[warp] = m; sm_l[warp] = l; }
    }
    __syncthreads();

    const int x = threadIdx.x;
    float M = -FLT_MAX, L = 0.f, A = 0.f;
    if (x < a.row_stride) {
#pragma unroll
        for (int w = 0; w < kStaticWarps; ++w) M = fmaxf(M, sm_m[w]);
#pragma unroll
        for (int w = 0; w < kStaticWarps; ++w) {
            float wgt = exp2f(sm_m[w] - M);
            L = fmaf(sm_l[w], wgt, L);
            A = fmaf(sm_acc[w][x], wgt, A);
        }
    }
    if (a.n_splits == 1) {
        if (x < a.d) {
            float o = A / L;
            if (a.out_f32) a.out_f32[(size_t)sid * a.d + x] = o;
            if (a.out_bf16) a.out_bf16[(size_t)sid * a.d + x] = __float2bfloat16_rn(o);
        }
        return;
    }
    const int pstride = a.row_stride + 2;
    float *part = a.partials + ((size_t)sid * a.n_splits + split) * pstride;
    if (x < a.row_stride) part[x] = A;
    if (x == 0) { part[a.row_stride] = M; part[a.row_stride + 1] = L; }
    __threadfence();
    __syncthreads();
    if (x == 0) s_last = (atomicAdd(&a.tickets[sid], 1) == a.n_splits - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (x < a.d) {
        const float *base = a.partials + (size_t)sid * a.n_splits * pstride;
        float Mx = -FLT_MAX;
        for (int sp = 0; sp < a.n_splits; ++sp) Mx = fmaxf(Mx, __ldcg(base + sp * pstride + a.row_stride));
        float Lx = 0.f, Ax = 0.f;
        for (int sp = 0; sp < a.n_splits; ++sp) {
            const float *ps = base + sp * pstride;
            float wgt = exp2f(__ldcg(ps + a.row_stride) - Mx);
            Lx = fmaf(__ldcg(ps + a.row_stride + 1), wgt, Lx);
            Ax = fmaf(__ldcg(ps + x), wgt, Ax);
        }
        float o = Ax / Lx;
        if (a.out_f32) a.out_f32[(size_t)sid * a.d + x] = o;
        if (a.out_bf16) a.out_bf16[(size_t)sid * a.d + x] = __float2bfloat16_rn(o);
    }
}

namespace {

struct StaticDevice {
    unsigned char *scratch = nullptr;   // device address of g_static_scratch on this GPU
    int sm_count = 0;
};
StaticDevice g_static_dev[kStaticMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: the device address of the scratch array.
int static_device_setup(StaticDevice **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return ADSA_ECUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice &sd = g_static_dev[dev];
    if (!sd.scratch) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ADSA_ECUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return ADSA_ECUDA;
        sd.sm_count = sms;
        sd.scratch = (unsigned char *)p;
    }
    *out = &sd;
    return ADSA_OK;
}

}  // namespace
}  // namespace adsa

using namespace adsa;

extern "C" int adsa_decode_attn_static(const void *q, const void *k, const void *v, const int32_t *n_rows,
                                       const void *k_new, const void *v_new, int n_streams, int max_rows, int head_dim,
                                       int row_stride, float softmax_scale, void *out_bf16, float *out_f32,
                                       adsa_stream_t stream)
{
    if (!q || !k || !v || !n_rows || !k_new || !v_new || (!out_bf16 && !out_f32)) return ADSA_EINVAL;
    if (n_streams < 1 || max_rows < 0 || head_dim < 8 || head_dim > 256) return ADSA_EINVAL;
    if (row_stride < head_dim || row_stride % 8 != 0 || row_stride > 256) return ADSA_EINVAL;
    if (((uintptr_t)k | (uintptr_t)v) & 15u) return ADSA_EINVAL;
    if (!(softmax_scale >= 0.f) || softmax_scale > FLT_MAX) return ADSA_EINVAL;
    if (n_streams > kStaticMaxStreams || max_rows > kStaticMaxRows) return ADSA_ENOMEM;   // beyond the built-in scratch

    StaticDevice *sd = nullptr;
    int rc = static_device_setup(&sd);
    if (rc != ADSA_OK) return rc;

    // chunks: enough blocks for several per SM, at least 64 rows each, and partials that fit the array
    const size_t ticket_bytes = (size_t)kStaticMaxStreams * sizeof(int32_t);
    const size_t per_split = (size_t)n_streams * (row_stride + 2) * sizeof(float);
    int fit = (int)((kStaticScratchBytes - ticket_bytes) / per_split);
    if (fit < 1) fit = 1;   // a single chunk per stream writes its output directly: no partial state, no counter
    int rows = max_rows < 1 ? 1 : max_rows;
    int splits = (sd->sm_count * 8 + n_streams - 1) / n_streams;
    splits = splits < 1 ? 1 : splits > kMaxSplits ? kMaxSplits : splits;
    if (splits > fit) splits = fit;
    int chunk = ((rows + splits - 1) / splits + 31) / 32 * 32;
    if (chunk < 64) chunk = 64;
    splits = (rows + chunk - 1) / chunk;

    StaticAttnArgs a;
    a.q = (const __nv_bfloat16 *)q; a.k = (const __nv_bfloat16 *)k; a.v = (const __nv_bfloat16 *)v;
    a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.n_rows = n_rows;
    a.out_bf16 = (__nv_bfloat16 *)out_bf16; a.out_f32 = out_f32;
    a.tickets = (int32_t *)sd->scratch;
    a.partials = (float *)(sd->scratch + ticket_bytes);
    a.max_rows = max_rows; a.d = head_dim; a.row_stride = row_stride; a.chunk_rows = chunk; a.n_splits = splits;
    float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    a.scale_log2e = scale * 1.4426950408889634f;

    cudaStream_t st = (cudaStream_t)stream;
    if (splits > 1 && cudaMemsetAsync(a.tickets, 0, (size_t)n_streams * sizeof(int32_t), st) != cudaSuccess) return ADSA_ECUDA;
    dim3 grid(splits, n_streams);
    int pieces = row_stride / 8;
    if (pieces <= 4) attn_static_kernel<4><<<grid, kStaticThreads, 0, st>>>(a);
    else if (pieces <= 8) attn_static_kernel<8><<<grid, kStaticThreads, 0, st>>>(a);
    else if (pieces <= 16) attn_static_kernel<16><<<grid, kStaticThreads, 0, st>>>(a);
    else attn_static_kernel<32><<<grid, kStaticThreads, 0, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? ADSA_OK : ADSA_ECUDA;
}
