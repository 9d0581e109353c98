// GAT: attention scores, the fused logit + online-softmax + weighted-sum aggregation, and the
// materialised edge softmax.
//
// The attention logits always use the full head width (scores are computed once from all of z);
// feature decomposition only cuts the weighted sum into column chunks, so the chunked result equals
// the undecomposed one.  The fused kernel walks a row once, keeping a running maximum m, a running
// denominator l and the un-normalised weighted sum per lane; edge-parallel groups and hub segments
// are merged by the usual log-sum-exp rule in a fixed order.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "schedule.cuh"

namespace gnnfd {

struct GatArgs {
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* row_order;
    const int32_t* seg_row;
    const int32_t* seg_begin;
    const float* s_src;
    const float* s_dst;
    const void* z;
    void* out;
    float* partial;      // [n_segments, fpad] un-normalised sums of hub segments
    float* partial_ml;   // [n_segments, heads, 2] running max and denominator of hub segments
    int64_t ldz, ldo;
    float slope;
    int32_t f, heads, dim, chunk_width, n_ctiles, blocks_per_tile, fpad, out_bf16;
    int32_t n_ranges;
    Range range[kMaxRanges];
};

template <typename T, int VECN> struct ZVec;
template <> struct ZVec<float, 4> {
    float4 v;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
    __device__ __forceinline__ void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ float get(int i) const { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }
};
template <> struct ZVec<float, 1> {
    float v;
    __device__ __forceinline__ void load(const float* p) { v = __ldg(p); }
    __device__ __forceinline__ void zero() { v = 0.f; }
    __device__ __forceinline__ float get(int) const { return v; }
};
template <> struct ZVec<__nv_bfloat16, 8> {
    uint4 v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ void zero() { v = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ float get(int i) const
    {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
    }
};
template <> struct ZVec<__nv_bfloat16, 1> {
    unsigned short v;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const unsigned short*>(p)); }
    __device__ __forceinline__ void zero() { v = 0; }
    __device__ __forceinline__ float get(int) const { return __uint_as_float((uint32_t)v << 16); }
};

__device__ __forceinline__ float widen(float x) { return x; }
__device__ __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }

__device__ __forceinline__ float leaky(float x, float slope) { return x >= 0.f ? x : slope * x; }

// weight of a partial result with running maximum m when merged under the maximum m_new
__device__ __forceinline__ float merge_scale(float m, float m_new)
{
    return m == -CUDART_INF_F ? 0.f : expf(m - m_new);
}

__device__ __forceinline__ void store_out(void* out, int out_bf16, int64_t idx, float val)
{
    if (out_bf16) static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(val);
    else __stcs(static_cast<float*>(out) + idx, val);
}

// ------------------------------------------------------------------ scores

template <typename T>
__global__ void __launch_bounds__(kBlock)
gat_scores(const T* __restrict__ z, int64_t ldz, const float* __restrict__ a_src, const float* __restrict__ a_dst,
           int64_t n, int heads, int dim, float* __restrict__ s_src, float* __restrict__ s_dst)
{
    const int64_t idx = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (idx >= n * heads) return;
    const int64_t v = idx / heads;
    const int h = (int)(idx % heads);
    const T* zr = z + v * ldz + (int64_t)h * dim;
    float ss = 0.f, sd = 0.f;
    for (int d = 0; d < dim; ++d) {
        const float zv = widen(zr[d]);
        ss = fmaf(__ldg(a_src + h * dim + d), zv, ss);
        sd = fmaf(__ldg(a_dst + h * dim + d), zv, sd);
    }
    s_src[idx] = ss;
    s_dst[idx] = sd;
}

// ------------------------------------------------------------------ fused aggregation

template <typename T, int VECN, int LPR, int EP>
__device__ __forceinline__ void gat_rows(const GatArgs& a, const Range& rg, int block_in_range, int col0, int chunk_end)
{
    constexpr int S = LPR * EP;
    constexpr int ROWS = kBlock / S;
    const int tid = threadIdx.x;
    const int slot = block_in_range * ROWS + tid / S;
    const int ls = tid % S;
    const int g = ls / LPR;
    const int j = col0 + (ls % LPR) * VECN;
    const bool col_ok = j < chunk_end;
    const bool active = slot < rg.item_count;
    const int h = col_ok ? j / a.dim : 0;      // all VECN columns of a lane lie in one head

    int32_t row = 0, b = 0, e = 0;
    if (active) {
        if (rg.hub) {
            row = a.seg_row[slot];
            b = a.seg_begin[slot];
            e = min(b + kHubSegment, a.row_ptr[row + 1]);
        } else {
            row = a.row_order[rg.item_begin + slot];
            b = a.row_ptr[row];
            e = a.row_ptr[row + 1];
        }
    }
    const float sd = active ? a.s_dst[(int64_t)row * a.heads + h] : 0.f;
    const float* ssrc = a.s_src + h;
    const T* zj = static_cast<const T*>(a.z) + j;

    float m = -CUDART_INF_F, l = 0.f;
    float acc[VECN];
#pragma unroll
    for (int i = 0; i < VECN; ++i) acc[i] = 0.f;

    for (int32_t k = b + g; k < e; k += EP * kUnroll) {
        int32_t u[kUnroll];
#pragma unroll
        for (int t = 0; t < kUnroll; ++t) {
            const int32_t kk = k + t * EP;
            u[t] = kk < e ? __ldcs(a.col_idx + kk) : -1;
        }
        float logit[kUnroll];
        ZVec<T, VECN> v[kUnroll];
#pragma unroll
        for (int t = 0; t < kUnroll; ++t) {
            if (u[t] >= 0) {
                logit[t] = __ldg(ssrc + (int64_t)u[t] * a.heads);
                if (col_ok) v[t].load(zj + (int64_t)u[t] * a.ldz); else v[t].zero();
            } else {
                logit[t] = 0.f;
                v[t].zero();
            }
        }
        float mx = m;
#pragma unroll
        for (int t = 0; t < kUnroll; ++t) {
            logit[t] = leaky(logit[t] + sd, a.slope);
            if (u[t] >= 0) mx = fmaxf(mx, logit[t]);
        }
        const float rescale = merge_scale(m, mx);     // the first edge of the step is valid, so mx is finite
        m = mx;
        l *= rescale;
#pragma unroll
        for (int i = 0; i < VECN; ++i) acc[i] *= rescale;
#pragma unroll
        for (int t = 0; t < kUnroll; ++t) {
            const float p = u[t] >= 0 ? expf(logit[t] - m) : 0.f;
            l += p;
#pragma unroll
            for (int i = 0; i < VECN; ++i) acc[i] = fmaf(p, v[t].get(i), acc[i]);
        }
    }

    // merge the EP groups of the row, fixed tree
#pragma unroll
    for (int o = S / 2; o >= LPR; o >>= 1) {
        const float m2 = __shfl_down_sync(0xffffffffu, m, o, S);
        const float l2 = __shfl_down_sync(0xffffffffu, l, o, S);
        const float mn = fmaxf(m, m2);
        const float sa = merge_scale(m, mn), sb = merge_scale(m2, mn);
        l = l * sa + l2 * sb;
#pragma unroll
        for (int i = 0; i < VECN; ++i) {
            const float a2 = __shfl_down_sync(0xffffffffu, acc[i], o, S);
            acc[i] = acc[i] * sa + a2 * sb;
        }
        m = mn;
    }

    if (!active || g != 0 || !col_ok) return;
    if (rg.hub) {
        float* p = a.partial + (int64_t)slot * a.fpad + j;
#pragma unroll
        for (int i = 0; i < VECN; ++i)
            if (j + i < chunk_end) p[i] = acc[i];
        // every lane of a head holds the same (m, l); the first lane of each head inside this column tile stores
        // it (sweeps that share a head store identical values)
        if (j % a.dim == 0 || ls % LPR == 0) {
            float* ml = a.partial_ml + ((int64_t)slot * a.heads + h) * 2;
            ml[0] = m;
            ml[1] = l;
        }
        return;
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int64_t o = (int64_t)row * a.ldo + j;
#pragma unroll
    for (int i = 0; i < VECN; ++i)
        if (j + i < chunk_end) store_out(a.out, a.out_bf16, o + i, acc[i] * inv);
}

template <typename T, int VECN, int LPR>
__global__ void __launch_bounds__(kBlock) gat_aggregate(const __grid_constant__ GatArgs a)
{
    const int64_t per_chunk = (int64_t)a.blocks_per_tile * a.n_ctiles;
    const int chunk = (int)(blockIdx.x / per_chunk);
    const int rem = (int)(blockIdx.x % per_chunk);
    const int rb = rem / a.n_ctiles;
    const int ctile = rem % a.n_ctiles;
    const int chunk_begin = chunk * a.chunk_width;
    const int chunk_end = min(a.f, chunk_begin + a.chunk_width);
    const int col0 = chunk_begin + ctile * (LPR * VECN);
    if (col0 >= chunk_end) return;
    int r = 0;
#pragma unroll
    for (int i = 1; i < kMaxRanges; ++i)
        if (i < a.n_ranges && rb >= a.range[i].first_block) r = i;
    const Range rg = a.range[r];
    const int bir = rb - rg.first_block;
    switch (rg.ep_log2) {
        case 0: gat_rows<T, VECN, LPR, 1>(a, rg, bir, col0, chunk_end); break;
        case 1: if constexpr (LPR * 2 <= 32) gat_rows<T, VECN, LPR, 2>(a, rg, bir, col0, chunk_end); break;
        case 2: if constexpr (LPR * 4 <= 32) gat_rows<T, VECN, LPR, 4>(a, rg, bir, col0, chunk_end); break;
        case 3: if constexpr (LPR * 8 <= 32) gat_rows<T, VECN, LPR, 8>(a, rg, bir, col0, chunk_end); break;
        case 4: if constexpr (LPR * 16 <= 32) gat_rows<T, VECN, LPR, 16>(a, rg, bir, col0, chunk_end); break;
        default: if constexpr (LPR == 1) gat_rows<T, VECN, LPR, 32>(a, rg, bir, col0, chunk_end); break;
    }
}

// out[row, j] = sum_s partial[s, j] e^(m_s - M) / sum_s l_s e^(m_s - M), segments in ascending order
__global__ void __launch_bounds__(kBlock)
gat_hub_reduce(const int32_t* __restrict__ row_order, const int32_t* __restrict__ hub_seg_ptr,
               const float* __restrict__ partial, const float* __restrict__ partial_ml, int64_t hub_begin, int32_t n_hub,
               int32_t f, int32_t fpad, int32_t heads, int32_t dim, void* __restrict__ out, int64_t ldo, int out_bf16)
{
    const int i = blockIdx.x;
    const int j = blockIdx.y * kBlock + threadIdx.x;
    if (i >= n_hub || j >= f) return;
    const int h = j / dim;
    const int32_t row = row_order[hub_begin + i];
    const int32_t s0 = hub_seg_ptr[i], s1 = hub_seg_ptr[i + 1];
    float mx = -CUDART_INF_F;
    for (int32_t s = s0; s < s1; ++s) mx = fmaxf(mx, partial_ml[((int64_t)s * heads + h) * 2]);
    float num = 0.f, den = 0.f;
    for (int32_t s = s0; s < s1; ++s) {
        const float* ml = partial_ml + ((int64_t)s * heads + h) * 2;
        const float w = merge_scale(ml[0], mx);
        den = fmaf(ml[1], w, den);
        num = fmaf(partial[(int64_t)s * fpad + j], w, num);
    }
    store_out(out, out_bf16, (int64_t)row * ldo + j, den > 0.f ? num / den : 0.f);
}

// ------------------------------------------------------------------ edge softmax
//
// GROUP threads (a warp, or a whole block for hub rows) share a row.  When heads is a power of two
// <= 32 a thread owns head t % heads and every (32 / heads)-th ... edge, so that alpha is written
// with consecutive threads on consecutive addresses; otherwise the heads are taken one at a time.

template <int GROUP>
__device__ __forceinline__ float group_max(float v, int lanes_per_value, float* smem)
{
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1)
        if (o >= lanes_per_value) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (GROUP > 32) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        __syncthreads();
        smem[warp * 32 + lane] = v;
        __syncthreads();
        v = smem[lane];
#pragma unroll
        for (int w = 1; w < GROUP / 32; ++w) v = fmaxf(v, smem[w * 32 + lane]);
    }
    return v;
}

template <int GROUP>
__device__ __forceinline__ float group_sum(float v, int lanes_per_value, float* smem)
{
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1)
        if (o >= lanes_per_value) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (GROUP > 32) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        __syncthreads();
        smem[warp * 32 + lane] = v;
        __syncthreads();
        v = smem[lane];
#pragma unroll
        for (int w = 1; w < GROUP / 32; ++w) v += smem[w * 32 + lane];
    }
    return v;
}

template <int GROUP>
__device__ __forceinline__ void softmax_row(const int32_t* __restrict__ col_idx, const float* __restrict__ s_src,
                                            const float* __restrict__ s_dst, int32_t row, int32_t b, int32_t e, int heads,
                                            float slope, float* __restrict__ alpha, float* smem)
{
    const int t = threadIdx.x % GROUP;
    const bool packed = heads <= 32 && (heads & (heads - 1)) == 0;
    const int hh = packed ? heads : 1;           // heads handled together
    const int step = GROUP / hh;                 // edges handled together
    for (int h0 = 0; h0 < heads; h0 += hh) {
        const int h = h0 + (t % hh);
        const float sd = s_dst[(int64_t)row * heads + h];
        float m = -CUDART_INF_F;
        for (int32_t k = b + t / hh; k < e; k += step)
            m = fmaxf(m, leaky(__ldg(s_src + (int64_t)col_idx[k] * heads + h) + sd, slope));
        m = group_max<GROUP>(m, hh, smem);
        float l = 0.f;
        for (int32_t k = b + t / hh; k < e; k += step)
            l += expf(leaky(__ldg(s_src + (int64_t)col_idx[k] * heads + h) + sd, slope) - m);
        l = group_sum<GROUP>(l, hh, smem);
        const float inv = 1.f / l;
        for (int32_t k = b + t / hh; k < e; k += step)
            __stcs(alpha + (int64_t)k * heads + h,
                   expf(leaky(__ldg(s_src + (int64_t)col_idx[k] * heads + h) + sd, slope) - m) * inv);
    }
}

__global__ void __launch_bounds__(kBlock)
edge_softmax_rows(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                  const int32_t* __restrict__ row_order, int64_t n_rows, const float* __restrict__ s_src,
                  const float* __restrict__ s_dst, int heads, float slope, float* __restrict__ alpha)
{
    const int64_t slot = (int64_t)blockIdx.x * (kBlock / 32) + (threadIdx.x >> 5);
    if (slot >= n_rows) return;               // whole warps leave together
    const int32_t row = row_order[slot];
    softmax_row<32>(col_idx, s_src, s_dst, row, row_ptr[row], row_ptr[row + 1], heads, slope, alpha, nullptr);
}

__global__ void __launch_bounds__(kBlock)
edge_softmax_hubs(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                  const int32_t* __restrict__ hub_rows, const float* __restrict__ s_src, const float* __restrict__ s_dst,
                  int heads, float slope, float* __restrict__ alpha)
{
    __shared__ float smem[kBlock];
    const int32_t row = hub_rows[blockIdx.x];
    softmax_row<kBlock>(col_idx, s_src, s_dst, row, row_ptr[row], row_ptr[row + 1], heads, slope, alpha, smem);
}

// ------------------------------------------------------------------ host side

typedef void (*GatKernel)(const GatArgs);

template <typename T, int VECN>
static GatKernel pick_lpr(int lpr)
{
    switch (lpr) {
        case 1: return gat_aggregate<T, VECN, 1>;
        case 2: return gat_aggregate<T, VECN, 2>;
        case 4: return gat_aggregate<T, VECN, 4>;
        case 8: return gat_aggregate<T, VECN, 8>;
        case 16: return gat_aggregate<T, VECN, 16>;
        default: return gat_aggregate<T, VECN, 32>;
    }
}

struct GatScratch {
    float *s_src, *s_dst, *partial, *partial_ml;
};

static void carve_gat(Carver& c, const gnnfd_csr_t* csr, int32_t heads, int32_t dim, GatScratch* g)
{
    const size_t fpad = align_up((size_t)heads * dim, 4);
    g->s_src = c.take<float>((size_t)csr->n * heads);
    g->s_dst = c.take<float>((size_t)csr->n * heads);
    g->partial = c.take<float>((size_t)csr->n_segments * fpad);
    g->partial_ml = c.take<float>((size_t)csr->n_segments * heads * 2);
}

static int launch_scores(int64_t n, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src,
                         const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst, cudaStream_t s)
{
    const int64_t total = n * heads;
    const unsigned grid = (unsigned)((total + kBlock - 1) / kBlock);
    if (zdt == GNNFD_F32)
        GNNFD_LAUNCH("gat_scores", s, gat_scores<float>, grid, kBlock, 0, static_cast<const float*>(d_z), ldz, d_a_src,
                     d_a_dst, n, heads, dim, d_s_src, d_s_dst);
    else
        GNNFD_LAUNCH("gat_scores", s, gat_scores<__nv_bfloat16>, grid, kBlock, 0, static_cast<const __nv_bfloat16*>(d_z),
                     ldz, d_a_src, d_a_dst, n, heads, dim, d_s_src, d_s_dst);
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" {

int gnnfd_gat_scores(int64_t n, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src, const float* d_a_dst,
                     int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst, void* stream)
{
    if (n <= 0 || !d_z || !d_a_src || !d_a_dst || !d_s_src || !d_s_dst || heads <= 0 || dim <= 0 ||
        ldz < (int64_t)heads * dim)
        return GNNFD_INVALID_ARG;
    if (zdt != GNNFD_F32 && zdt != GNNFD_BF16) return GNNFD_UNSUPPORTED;
    if (n * heads > 0x7fffffffll * gnnfd::kBlock) return GNNFD_TOO_LARGE;
    return gnnfd::launch_scores(n, d_z, ldz, zdt, d_a_src, d_a_dst, heads, dim, d_s_src, d_s_dst,
                                static_cast<cudaStream_t>(stream));
}

int gnnfd_gat_workspace_bytes(const gnnfd_csr_t* csr, int32_t heads, int32_t dim, size_t* scratch_bytes)
{
    if (!csr || heads <= 0 || dim <= 0 || !scratch_bytes) return GNNFD_INVALID_ARG;
    gnnfd::Carver c(nullptr, ~size_t(0));
    gnnfd::GatScratch g;
    gnnfd::carve_gat(c, csr, heads, dim, &g);
    *scratch_bytes = c.off;
    return GNNFD_OK;
}

int gnnfd_aggregate_gat(const gnnfd_csr_t* csr, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src,
                        const float* d_a_dst, int32_t heads, int32_t dim, float negative_slope, void* d_out, int64_t ldo,
                        gnnfd_dtype_t odt, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream)
{
    using namespace gnnfd;
    if (!csr || !d_z || !d_a_src || !d_a_dst || !d_out || heads <= 0 || dim <= 0 || chunk_width <= 0) return GNNFD_INVALID_ARG;
    const int64_t f64 = (int64_t)heads * dim;
    if (f64 > 0x7fffffffll || ldz < f64 || ldo < f64) return GNNFD_INVALID_ARG;
    if ((zdt != GNNFD_F32 && zdt != GNNFD_BF16) || (odt != GNNFD_F32 && odt != GNNFD_BF16)) return GNNFD_UNSUPPORTED;
    if (!d_scratch || ((uintptr_t)d_scratch & 255u)) return GNNFD_INVALID_ARG;
    const int32_t f = (int32_t)f64;
    Carver c(d_scratch, scratch_bytes);
    GatScratch g;
    carve_gat(c, csr, heads, dim, &g);
    if (!c.ok) return GNNFD_WORKSPACE_TOO_SMALL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    int rc = launch_scores(csr->n, d_z, ldz, zdt, d_a_src, d_a_dst, heads, dim, g.s_src, g.s_dst, s);
    if (rc) return rc;

    const int cw = chunk_width < f ? chunk_width : f;
    const int n_chunks = (f + cw - 1) / cw;
    const int zsize = zdt == GNNFD_F32 ? 4 : 2;
    const int vecn = 16 / zsize;
    // a lane's vector must start 16-byte aligned and stay inside one head
    const bool vec = ((uintptr_t)d_z % 16 == 0) && ((ldz * zsize) % 16 == 0) && (n_chunks == 1 || cw % vecn == 0) &&
                     (dim % vecn == 0);
    const int elems = vec ? vecn : 1;
    const int lanes = (cw + elems - 1) / elems;
    int lpr = 1;
    while (lpr < lanes && lpr < 32) lpr <<= 1;

    GatArgs a;
    a.row_ptr = csr->row_ptr; a.col_idx = csr->col_idx; a.row_order = csr->row_order;
    a.seg_row = csr->seg_row; a.seg_begin = csr->seg_begin;
    a.s_src = g.s_src; a.s_dst = g.s_dst; a.z = d_z; a.out = d_out;
    a.partial = g.partial; a.partial_ml = g.partial_ml;
    a.ldz = ldz; a.ldo = ldo; a.slope = negative_slope;
    a.f = f; a.heads = heads; a.dim = dim; a.chunk_width = cw;
    a.n_ctiles = (cw + lpr * elems - 1) / (lpr * elems);
    a.fpad = (int32_t)align_up((size_t)f, 4);
    a.out_bf16 = odt == GNNFD_BF16;

    const int64_t blocks = plan_ranges(csr, lpr, a.range, &a.n_ranges);
    a.blocks_per_tile = (int32_t)blocks;
    const int64_t grid = blocks * a.n_ctiles * n_chunks;
    if (grid > 0x7fffffffll || blocks > 0x7fffffffll) return GNNFD_TOO_LARGE;
    if (grid > 0) {
        GatKernel kernel;
        if (zdt == GNNFD_F32) kernel = vec ? pick_lpr<float, 4>(lpr) : pick_lpr<float, 1>(lpr);
        else kernel = vec ? pick_lpr<__nv_bfloat16, 8>(lpr) : pick_lpr<__nv_bfloat16, 1>(lpr);
        GNNFD_LAUNCH("gat_aggregate", s, kernel, (unsigned)grid, kBlock, 0, a);
    }
    const int64_t n_hub = csr->bin_count[4];
    if (n_hub > 0) {
        dim3 gr((unsigned)n_hub, (unsigned)((f + kBlock - 1) / kBlock));
        GNNFD_LAUNCH("gat_hub_reduce", s, gat_hub_reduce, gr, kBlock, 0, csr->row_order, csr->hub_seg_ptr, g.partial,
                     g.partial_ml, csr->bin_start[4], (int32_t)n_hub, f, a.fpad, heads, dim, d_out, ldo, a.out_bf16);
    }
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

int gnnfd_edge_softmax(const gnnfd_csr_t* csr, const float* d_s_src, const float* d_s_dst, int32_t heads,
                       float negative_slope, float* d_alpha, void* stream)
{
    using namespace gnnfd;
    if (!csr || !d_s_src || !d_s_dst || !d_alpha || heads <= 0) return GNNFD_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t n_hub = csr->bin_count[4];
    const int64_t n_rows = csr->n - n_hub;      // the hub rows are the tail of row_order
    if (n_rows > 0) {
        const unsigned grid = (unsigned)((n_rows + kBlock / 32 - 1) / (kBlock / 32));
        GNNFD_LAUNCH("edge_softmax_rows", s, edge_softmax_rows, grid, kBlock, 0, csr->row_ptr, csr->col_idx, csr->row_order,
                     n_rows, d_s_src, d_s_dst, heads, negative_slope, d_alpha);
    }
    if (n_hub > 0)
        GNNFD_LAUNCH("edge_softmax_hubs", s, edge_softmax_hubs, (unsigned)n_hub, kBlock, 0, csr->row_ptr, csr->col_idx,
                     csr->row_order + csr->bin_start[4], d_s_src, d_s_dst, heads, negative_slope, d_alpha);
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // extern "C"
