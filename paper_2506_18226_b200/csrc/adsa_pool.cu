// Paged KV pool maintenance: reset, appending rows (text condition), replacing
// a stream's rows, and the Section 4.2 cache update (evict, insert, compact).
#include "adsa_dev.cuh"
#include "adsa_launch.h"

namespace adsa {

__global__ void reset_kernel(DevCtx c, int n_streams)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    int stride = gridDim.x * blockDim.x;
    for (int p = i; p < c.n_pages; p += stride) c.free_ring[p] = p;
    for (int s = i; s < n_streams; s += stride) c.n_live[s] = 0;
    for (int s = i; s < c.S; s += stride) { c.tickets[s] = 0; }
    if (i == 0) {
        c.free_state[0] = 0;          // head
        c.free_state[1] = 0;          // tail (ring full: tail wraps onto head)
        c.free_state[2] = c.n_pages;  // free count
        c.free_state[3] = c.n_pages;  // low-water mark
        *c.status = 0u;
    }
}

// One block per stream of the layer: append n_rows rows at first_pos...
__global__ void append_rows_kernel(DevCtx c, int layer, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                                   const int32_t *pos, int n_rows, int first_pos)
{
    __shared__ int ok;
    int local = blockIdx.x, sid = layer * c.S + local;
    int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    int n0 = c.n_live[sid], n1 = n0 + n_rows;
    if (threadIdx.x == 0) {
        ok = 1;
        if (n1 > c.max_rows) { set_status(c, ADSA_DEV_ROW_OVERFLOW); ok = 0; }
        else if (!resize_pages(c, pt, (n0 + c.page_rows - 1) / c.page_rows, (n1 + c.page_rows - 1) / c.page_rows)) ok = 0;
    }
    __syncthreads();
    if (!ok) return;
    int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int r = warp; r < n_rows; r += nwarps) {
        size_t src = ((size_t)local * n_rows + r) * c.d;
        write_row(c, pt, sid, n0 + r, k + src, v + src, pos ? pos[(size_t)local * n_rows + r] : first_pos + r);
    }
    __syncthreads();
    if (threadIdx.x == 0) c.n_live[sid] = n1;
}

// One block: replace the rows of stream sid.
__global__ void set_rows_kernel(DevCtx c, int sid, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                                const int32_t *pos, int n_rows)
{
    __shared__ int ok;
    int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    int n0 = c.n_live[sid];
    if (threadIdx.x == 0)
        ok = resize_pages(c, pt, (n0 + c.page_rows - 1) / c.page_rows, (n_rows + c.page_rows - 1) / c.page_rows) ? 1 : 0;
    __syncthreads();
    if (!ok) return;
    int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int r = warp; r < n_rows; r += nwarps)
        write_row(c, pt, sid, r, k + (size_t)r * c.d, v + (size_t)r * c.d, pos[r]);
    __syncthreads();
    if (threadIdx.x == 0) c.n_live[sid] = n_rows;
}

// Section 4.2 update, one block (kUpdateThreads) per stream.
//
// n rows are live, e of them are marked for eviction (keep_mask bit clear), the
// new row arrives: n2 = n - e + 1 rows remain.  Every slot below n2 that is
// evicted or beyond the old end is a hole; every retained slot at or above n2
// is a survivor that must move down.  There is exactly one more hole than
// survivors: the i-th survivor fills the i-th hole and the new row takes the
// last one.  Sources (>= n2) and destinations (< n2) are disjoint, so moves need
// no ordering.  In steady state (one eviction per step) the new row simply
// lands in the evicted slot and nothing moves.
constexpr int kUpdateThreads = 128;

__global__ void __launch_bounds__(kUpdateThreads)
kv_update_kernel(DevCtx c, int layer, int cur_pos, const __nv_bfloat16 *k_new, const __nv_bfloat16 *v_new)
{
    extern __shared__ int32_t sm_lists[];  // holes[max_rows + 1], survivors[max_rows]
    __shared__ int s_ok, s_nholes, s_nsurv;
    __shared__ int warp_cnt[2][kUpdateThreads / 32];
    int local = blockIdx.x, sid = layer * c.S + local;
    int32_t *pt = c.page_table + (size_t)sid * c.max_pages;
    const uint32_t *mask = c.keep_mask + (size_t)sid * c.mask_words;
    int32_t *holes = sm_lists, *surv = sm_lists + c.max_rows + 1;
    int n = c.n_live[sid], e = c.counts[(size_t)sid * 4 + 1];
    int n2 = n - e + 1;
    int have = (n + c.page_rows - 1) / c.page_rows, need = (n2 + c.page_rows - 1) / c.page_rows;
    if (threadIdx.x == 0) {
        s_ok = 1; s_nholes = 0; s_nsurv = 0;
        if (n2 > c.max_rows) { set_status(c, ADSA_DEV_ROW_OVERFLOW); s_ok = 0; }
        else if (need > have && !resize_pages(c, pt, have, need)) s_ok = 0;
    }
    __syncthreads();
    if (!s_ok) return;

    // ordered lists of holes and survivors: block-wide prefix sums over the slot flags
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int top = max(n, n2);
    for (int base = 0; base < top; base += kUpdateThreads) {
        int s = base + threadIdx.x;
        bool kept = s < n && ((mask[s >> 5] >> (s & 31)) & 1u);
        bool is_hole = s < n2 && !kept;
        bool is_surv = s >= n2 && s < n && kept;
        unsigned bh = __ballot_sync(0xffffffffu, is_hole), bs = __ballot_sync(0xffffffffu, is_surv);
        if (lane == 0) { warp_cnt[0][warp] = __popc(bh); warp_cnt[1][warp] = __popc(bs); }
        __syncthreads();
        int oh = s_nholes, os = s_nsurv;
        for (int w = 0; w < warp; ++w) { oh += warp_cnt[0][w]; os += warp_cnt[1][w]; }
        unsigned below = (1u << lane) - 1u;
        if (is_hole) holes[oh + __popc(bh & below)] = s;
        if (is_surv) surv[os + __popc(bs & below)] = s;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 0; w < kUpdateThreads / 32; ++w) { s_nholes += warp_cnt[0][w]; s_nsurv += warp_cnt[1][w]; }
        }
        __syncthreads();
    }
    int nh = s_nholes, ns = s_nsurv;
    if (nh != ns + 1) {  // cannot happen when counts and mask agree; refuse rather than corrupt
        if (threadIdx.x == 0) set_status(c, ADSA_DEV_BAD_EVICT);
        return;
    }
    // attention-mass mode: every retained row's mass grows by the softmax weight it had in this step's attention
    // (logits, maximum and denominator were left by the attention kernel), before rows move
    float *mass = c.scores + (size_t)sid * c.max_rows;
    float w_new = 0.f;
    if (c.score_mode == 1) {
        const float *lg = c.logit + (size_t)sid * c.max_rows;
        const float M = c.ml[(size_t)sid * 4], Ld = c.ml[(size_t)sid * 4 + 1];
        w_new = exp2f(c.ml[(size_t)sid * 4 + 2] - M) / Ld;
        for (int s = threadIdx.x; s < n; s += kUpdateThreads)
            if ((mask[s >> 5] >> (s & 31)) & 1u) mass[s] += exp2f(lg[s] - M) / Ld;
        __syncthreads();
    }
    // survivors move down: a row is row_stride bf16 = row_stride/8 16-byte pieces, for K and for V
    int pieces = c.row_stride >> 3;
    for (int i = warp; i < ns; i += kUpdateThreads / 32) {
        size_t src = row_offset(c, pt, surv[i]), dst = row_offset(c, pt, holes[i]);
        for (int x = lane; x < 2 * pieces; x += 32) {
            __nv_bfloat16 *pool = x < pieces ? c.k_pool : c.v_pool;
            int pc = x < pieces ? x : x - pieces;
            reinterpret_cast<uint4 *>(pool + dst)[pc] = reinterpret_cast<const uint4 *>(pool + src)[pc];
        }
        if (lane == 0) {
            size_t m = (size_t)sid * c.max_rows;
            c.pos[m + holes[i]] = c.pos[m + surv[i]];
            c.inv_norm[m + holes[i]] = c.inv_norm[m + surv[i]];
            if (c.score_mode == 1) mass[holes[i]] = mass[surv[i]];
        }
    }
    if (warp == 0) {
        write_row(c, pt, sid, holes[ns], k_new + (size_t)local * c.d, v_new + (size_t)local * c.d, cur_pos);
        if (c.score_mode == 1 && lane == 0) mass[holes[ns]] = w_new;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (need < have) resize_pages(c, pt, have, need);
        c.n_live[sid] = n2;
    }
}

// ---- host launchers -------------------------------------------------------
cudaError_t launch_reset(const DevCtx &c, int n_streams, cudaStream_t st)
{
    int work = max(c.n_pages, n_streams);
    int blocks = min(1024, (work + 255) / 256);
    reset_kernel<<<blocks, 256, 0, st>>>(c, n_streams);
    return cudaGetLastError();
}

cudaError_t launch_append_rows(const DevCtx &c, int layer, const void *k, const void *v, const int32_t *pos,
                               int n_rows, int first_pos, cudaStream_t st)
{
    append_rows_kernel<<<c.S, 256, 0, st>>>(c, layer, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, pos, n_rows,
                                             first_pos);
    return cudaGetLastError();
}

cudaError_t launch_set_rows(const DevCtx &c, int sid, const void *k, const void *v, const int32_t *pos, int n_rows,
                            cudaStream_t st)
{
    set_rows_kernel<<<1, 256, 0, st>>>(c, sid, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, pos, n_rows);
    return cudaGetLastError();
}

size_t kv_update_smem_bytes(const DevCtx &c) { return (size_t)(2 * c.max_rows + 1) * sizeof(int32_t); }

cudaError_t configure_update_kernel(const DevCtx &c)
{
    size_t b = kv_update_smem_bytes(c);
    if (b <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kv_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)b);
}

cudaError_t launch_kv_update(const DevCtx &c, int layer, int cur_pos, const void *k_new, const void *v_new,
                             cudaStream_t st)
{
    kv_update_kernel<<<c.S, kUpdateThreads, kv_update_smem_bytes(c), st>>>(c, layer, cur_pos,
                                                                          (const __nv_bfloat16 *)k_new,
                                                                          (const __nv_bfloat16 *)v_new);
    return cudaGetLastError();
}

}  // namespace adsa
