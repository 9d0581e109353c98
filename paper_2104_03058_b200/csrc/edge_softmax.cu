// Materialised edge softmax: alpha[k, h] for every CSR slot k from caller-supplied scores.
//
// Logit of slot k of row v, head h: LeakyReLU(s_src[col_idx[k], h] + s_dst[v, h]); alpha is the softmax
// over the slots of the row.  A row is shared by S threads.  When heads is a power of two <= 32 a
// thread owns head t % heads and every (S / heads)-th slot, so consecutive threads write
// consecutive addresses of alpha; otherwise the heads are taken one at a time.  S grows with the
// degree class of the row (the rows come sorted by degree, so a warp's rows have similar lengths).
// Rows of the top degree bin get a block each and hub rows a whole thread-block cluster: the per-head
// maxima and sums of the member blocks are exchanged through distributed shared memory.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace gnnfd {

constexpr int kRowBlock = 256;          // threads per block, ordinary rows
constexpr int kBigBlock = 256;          // threads per block, rows of 129 .. GNNFD_HUB_DEGREE entries (one block each)
constexpr int kHubBlock = 1024;         // threads per block, hub rows
constexpr int kHubCluster = 8;          // blocks per hub row

__device__ __forceinline__ float leaky_relu(float x, float slope) { return x >= 0.f ? x : slope * x; }

struct RowView {
    const int32_t* col_idx;
    const float* s_src;
    float* alpha;
    int32_t b, e;
    int heads;
    float slope;
};

// logit of slot k, head h
__device__ __forceinline__ float logit(const RowView& r, int32_t k, int h, float sd)
{
    return leaky_relu(__ldg(r.s_src + (int64_t)__ldg(r.col_idx + k) * r.heads + h) + sd, r.slope);
}

// Running maximum and denominator over slots first, first + step, ... (kInFlight logits in flight).
constexpr int kInFlight = 8;
__device__ __forceinline__ void online_max_sum(const RowView& r, int32_t first, int step, int h, float sd, float* m_out,
                                               float* l_out)
{
    float m = -CUDART_INF_F, l = 0.f;
    for (int32_t k = first; k < r.e; k += kInFlight * step) {
        float t[kInFlight];
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) t[i] = k + i * step < r.e ? logit(r, k + i * step, h, sd) : -CUDART_INF_F;
        float mx = m;                                                               // t[0] is valid, so mx ends finite
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) mx = fmaxf(mx, t[i]);
        l *= expf(m - mx);
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) l += expf(t[i] - mx);                   // exp(-inf) = 0 for the missing ones
        m = mx;
    }
    *m_out = m;
    *l_out = l;
}

__device__ __forceinline__ void write_alpha(const RowView& r, int32_t first, int step, int h, float sd, float m, float inv)
{
    for (int32_t k = first; k < r.e; k += kInFlight * step) {
        float t[kInFlight];
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) t[i] = k + i * step < r.e ? logit(r, k + i * step, h, sd) : 0.f;
#pragma unroll
        for (int i = 0; i < kInFlight; ++i)
            if (k + i * step < r.e) __stcs(r.alpha + (int64_t)(k + i * step) * r.heads + h, expf(t[i] - m) * inv);
    }
}

// ---- ordinary rows: S lanes of a warp per row

template <int S>
__global__ void __launch_bounds__(kRowBlock)
edge_softmax_rows(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                  const int32_t* __restrict__ rows, int64_t n_rows, const float* __restrict__ s_src,
                  const float* __restrict__ s_dst, int heads, int hh, float slope, float* __restrict__ alpha)
{
    const int64_t slot = (int64_t)blockIdx.x * (kRowBlock / S) + threadIdx.x / S;
    const int sl = threadIdx.x % S;
    const bool active = slot < n_rows;
    const int32_t row = active ? rows[slot] : 0;
    RowView r{col_idx, s_src, alpha, active ? row_ptr[row] : 0, active ? row_ptr[row + 1] : 0, heads, slope};
    const int step = S / hh;
    for (int h0 = 0; h0 < heads; h0 += hh) {
        const int h = h0 + sl % hh;
        const float sd = active ? s_dst[(int64_t)row * heads + h] : 0.f;
        const int32_t first = r.b + sl / hh;
        if (__all_sync(0xffffffffu, r.e - r.b <= kInFlight * step)) {
            // every row of this warp fits one round: the logits stay in registers between the two phases
            float t[kInFlight];
            float m = -CUDART_INF_F;
#pragma unroll
            for (int i = 0; i < kInFlight; ++i) {
                t[i] = first + i * step < r.e ? logit(r, first + i * step, h, sd) : -CUDART_INF_F;
                m = fmaxf(m, t[i]);
            }
#pragma unroll
            for (int o = S / 2; o >= 1; o >>= 1)
                if (o >= hh) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float l = 0.f;
#pragma unroll
            for (int i = 0; i < kInFlight; ++i) {
                t[i] = first + i * step < r.e ? expf(t[i] - m) : 0.f;
                l += t[i];
            }
#pragma unroll
            for (int o = S / 2; o >= 1; o >>= 1)
                if (o >= hh) l += __shfl_xor_sync(0xffffffffu, l, o);
            const float inv = 1.f / l;
#pragma unroll
            for (int i = 0; i < kInFlight; ++i)
                if (first + i * step < r.e) __stcs(alpha + (int64_t)(first + i * step) * heads + h, t[i] * inv);
            continue;
        }
        float m, l;
        online_max_sum(r, first, step, h, sd, &m, &l);
        float mall = m;
#pragma unroll
        for (int o = S / 2; o >= 1; o >>= 1)
            if (o >= hh) mall = fmaxf(mall, __shfl_xor_sync(0xffffffffu, mall, o));
        l = m == -CUDART_INF_F ? 0.f : l * expf(m - mall);
#pragma unroll
        for (int o = S / 2; o >= 1; o >>= 1)
            if (o >= hh) l += __shfl_xor_sync(0xffffffffu, l, o);
        write_alpha(r, first, step, h, sd, mall, 1.f / l);
    }
}

// ---- long rows: one block, hub rows: one cluster of blocks per row

// Combines one value per thread over all threads of the cluster that own the same head (threads with
// equal t % hh; hh divides 32).  `mine` is this block's exchange buffer of 32 floats.
template <bool IS_MAX, int THREADS, int CLUSTER>
__device__ __forceinline__ float cluster_combine(float v, int hh, float* warp_buf, float* mine, cg::cluster_group& cluster)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1)
        if (o >= hh) {
            const float other = __shfl_xor_sync(0xffffffffu, v, o);
            v = IS_MAX ? fmaxf(v, other) : v + other;
        }
    __syncthreads();                                  // the previous combine's readers are done
    warp_buf[warp * 32 + lane] = v;
    __syncthreads();
    float acc = warp_buf[lane];
#pragma unroll
    for (int w = 1; w < THREADS / 32; ++w) {
        const float other = warp_buf[w * 32 + lane];
        acc = IS_MAX ? fmaxf(acc, other) : acc + other;
    }
    if (CLUSTER == 1) return acc;
    if (warp == 0) mine[lane] = acc;
    cluster.sync();                                   // every block's `mine` is complete
    acc = IS_MAX ? -CUDART_INF_F : 0.f;
#pragma unroll
    for (int rk = 0; rk < CLUSTER; ++rk) {
        const float other = cluster.map_shared_rank(mine, rk)[lane];
        acc = IS_MAX ? fmaxf(acc, other) : acc + other;
    }
    cluster.sync();                                   // all reads done before the buffers are reused
    return acc;
}

template <int THREADS, int CLUSTER>
__global__ void __cluster_dims__(CLUSTER, 1, 1) __launch_bounds__(THREADS)
edge_softmax_big(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                 const int32_t* __restrict__ rows, const float* __restrict__ s_src, const float* __restrict__ s_dst,
                 int heads, int hh, float slope, int32_t min_len, int32_t max_len, float* __restrict__ alpha)
{
    __shared__ float warp_buf[THREADS];
    __shared__ float mine[32];
    cg::cluster_group cluster = cg::this_cluster();
    const int32_t row = rows[blockIdx.x / CLUSTER];
    {   // rows outside [min_len, max_len] belong to another launch; the whole cluster leaves together
        const int32_t len = row_ptr[row + 1] - row_ptr[row];
        if (len < min_len || len > max_len) return;
    }
    const int t = (CLUSTER == 1 ? 0 : (int)cluster.block_rank() * THREADS) + threadIdx.x;
    RowView r{col_idx, s_src, alpha, row_ptr[row], row_ptr[row + 1], heads, slope};
    const int step = THREADS * CLUSTER / hh;
    for (int h0 = 0; h0 < heads; h0 += hh) {
        const int h = h0 + t % hh;
        const float sd = s_dst[(int64_t)row * heads + h];
        float m, l;
        online_max_sum(r, r.b + t / hh, step, h, sd, &m, &l);
        const float mall = cluster_combine<true, THREADS, CLUSTER>(m, hh, warp_buf, mine, cluster);
        l = m == -CUDART_INF_F ? 0.f : l * expf(m - mall);
        l = cluster_combine<false, THREADS, CLUSTER>(l, hh, warp_buf, mine, cluster);
        write_alpha(r, r.b + t / hh, step, h, sd, mall, 1.f / l);
    }
}

typedef void (*RowKernel)(const int32_t*, const int32_t*, const int32_t*, int64_t, const float*, const float*, int, int,
                          float, float*);

static RowKernel pick_rows(int s)
{
    switch (s) {
        case 1: return edge_softmax_rows<1>;
        case 2: return edge_softmax_rows<2>;
        case 4: return edge_softmax_rows<4>;
        case 8: return edge_softmax_rows<8>;
        case 16: return edge_softmax_rows<16>;
        default: return edge_softmax_rows<32>;
    }
}

}  // namespace gnnfd

extern "C" int gnnfd_edge_softmax(const gnnfd_csr_t* csr, const float* d_s_src, const float* d_s_dst, int32_t heads,
                                  float negative_slope, float* d_alpha, void* stream)
{
    using namespace gnnfd;
    if (!csr || !d_s_src || !d_s_dst || heads <= 0 || (!d_alpha && csr->nnz > 0)) return GNNFD_INVALID_ARG;
    if (csr->nnz == 0) return GNNFD_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int hh = (heads <= 32 && (heads & (heads - 1)) == 0) ? heads : 1;   // heads handled together
    static const int slots_in_parallel[3] = {2, 8, 32};                       // per degree bin of the row
    for (int bin = 0; bin < 3; ++bin) {
        const int64_t rows = csr->bin_count[bin];
        if (rows == 0) continue;
        int lanes = hh * slots_in_parallel[bin];
        if (lanes > 32) lanes = 32;
        const int rows_per_block = kRowBlock / lanes;
        const unsigned grid = (unsigned)((rows + rows_per_block - 1) / rows_per_block);
        GNNFD_LAUNCH("edge_softmax_rows", s, pick_rows(lanes), grid, kRowBlock, 0, csr->row_ptr, csr->col_idx,
                     csr->row_order + csr->bin_start[bin], rows, d_s_src, d_s_dst, heads, hh, negative_slope, d_alpha);
    }
    if (csr->bin_count[3] > 0)
        GNNFD_LAUNCH("edge_softmax_long_rows", s, (edge_softmax_big<kBigBlock, 1>), (unsigned)csr->bin_count[3], kBigBlock, 0,
                     csr->row_ptr, csr->col_idx, csr->row_order + csr->bin_start[3], d_s_src, d_s_dst, heads, hh,
                     negative_slope, 0, 0x7fffffff, d_alpha);
    const int64_t n_hub = csr->bin_count[4];
    if (n_hub > 0)
        GNNFD_LAUNCH("edge_softmax_hubs", s, (edge_softmax_big<kHubBlock, kHubCluster>), (unsigned)(n_hub * kHubCluster),
                     kHubBlock, 0, csr->row_ptr, csr->col_idx, csr->row_order + csr->bin_start[4], d_s_src, d_s_dst, heads,
                     hh, negative_slope, 0, 0x7fffffff, d_alpha);
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}
