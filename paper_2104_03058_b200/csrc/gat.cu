// GAT: attention scores and the fused logit + online-softmax + weighted-sum aggregation.
//
// The attention logits always use the full head width (scores are computed once from all of z);
// feature decomposition only cuts the weighted sum into column chunks, so the chunked result equals
// the undecomposed one.  The fused kernel walks a row once, keeping a running maximum m, a running
// denominator l and the un-normalised weighted sum per lane; edge-parallel groups and hub segments
// are merged by the usual log-sum-exp rule in a fixed order.
#include <math_constants.h>

#include <type_traits>

#include "schedule.cuh"
#include "vec.cuh"

namespace gnnfd {

struct GatArgs {
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* row_order;
    const int32_t* seg_row;
    const int32_t* seg_begin;
    const int32_t* seg_end;
    const int32_t* seg_slot;
    const float* s_src;
    const float* s_dst;
    const void* z;
    void* out;
    float* partial;      // [n_segments, fpad] un-normalised sums of hub segments
    float* partial_ml;   // [n_segments, heads, 2] running max and denominator of hub segments
    int64_t ldz, ldo;
    float slope;
    int32_t f, heads, dim, chunk_width, n_ctiles, blocks_per_tile, fpad, out_bf16, wide_ok;
    int32_t chunk_base;      // first chunk of this launch (a launch covers at most 65,535 chunks)
    int32_t n_ranges;
    Range range[kMaxRanges];
};

__device__ __forceinline__ float widen(float x) { return x; }
__device__ __forceinline__ float widen(__nv_bfloat16 x) { return __bfloat162float(x); }


constexpr float kLog2e = 1.4426950408889634f;

// 2^x by the hardware approximation (2 ulp; results below 2^-126 become 0, 2^-inf = 0)
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// weight of a partial result with running maximum m (a base-2 logit) when merged under the maximum m_new
__device__ __forceinline__ float merge_scale(float m, float m_new)
{
    return m == -CUDART_INF_F ? 0.f : exp2f(m - m_new);
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

constexpr int kLoads = 8;      // 16-byte feature loads kept in flight per lane

constexpr int kStageSlots = kLoads * 32;      // column indices a warp stages per batch, at most

// One row (or hub segment) per S = LPR * EP lanes, same batching as the GCN / SAGE gather: the S lanes
// fetch S column indices per round with one coalesced load and stage them in shared memory.  A lane
// covers VPL adjacent vectors, all inside one head, so it needs one logit per entry.
template <typename T, int VECN, int LPR, int VPL, int EP>
__device__ __forceinline__ void gat_rows(const GatArgs& a, const Range& rg, int block_in_range, int col0, int chunk_end,
                                         int32_t (*stage_col)[kBlock / 32][kStageSlots], float (*tot_s)[kBlock])
{
    constexpr int S = LPR * EP;
    constexpr int ROWS = kBlock / S;
    constexpr int UB = kLoads / VPL;
    constexpr int R = UB > LPR ? UB / LPR : 1;
    constexpr int SPB = R * LPR;
    constexpr int EPB = R * S;
    constexpr unsigned kFull = 0xffffffffu;
    const int tid = threadIdx.x;
    const int slot = block_in_range * ROWS + tid / S;
    const int sl = tid % S;
    const int g = sl / LPR;
    const int c = sl % LPR;
    const int j0 = col0 + c * (VPL * VECN);
    const int warp = tid >> 5, lane = tid & 31;
    const int seg = lane - sl;                   // first lane of this row's segment inside the warp
    const bool active = slot < rg.item_count;
    const bool lane_ok = j0 < chunk_end;
    const int h = (lane_ok ? j0 : col0) / a.dim;

    bool okq[VPL];
    const T* zq[VPL];
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
        okq[q] = j0 + q * VECN < chunk_end;
        zq[q] = static_cast<const T*>(a.z) + (okq[q] ? j0 + q * VECN : col0);
    }

    int32_t row = 0, b = 0, e = 0;
    if (active) {
        if (rg.hub) {
            row = a.seg_row[slot];
            b = a.seg_begin[slot];
            e = a.seg_end[slot];
        } else {
            row = a.row_order[rg.item_begin + slot];
            b = a.row_ptr[row];
            e = a.row_ptr[row + 1];
        }
    }
    // one 32-byte load per entry when both vectors of the lane exist and every row start allows it
    const bool wide = a.wide_ok && okq[VPL - 1];
    const float sd = active ? a.s_dst[(int64_t)row * a.heads + h] : 0.f;
    const float* ssrc = a.s_src + h;
    // logits are kept in base 2: LeakyReLU(x) * log2 e = c1 * x + c2 * |x|
    const float c1 = 0.5f * kLog2e * (1.f + a.slope), c2 = 0.5f * kLog2e * (1.f - a.slope);
    auto leaky2 = [c1, c2](float x) { return fmaf(fabsf(x), c2, x * c1); };
    const uint32_t ld = (uint32_t)a.ldz;
    const uint32_t heads = (uint32_t)a.heads;

    // Two levels of accumulation (as in the GCN / SAGE gather): `acc` and `l` take at most kChain terms in a
    // row, then move into the thread's second-level sums in shared memory (slot VPL * VECN holds the
    // denominator).  The second level is expressed under its own maximum m_tot and is brought to the
    // current one only when something is added to it.
    constexpr int kChain = 64;
    constexpr int FLUSH = SPB >= kChain ? 1 : kChain / SPB;
    float m = -CUDART_INF_F, l = 0.f, m_tot = -CUDART_INF_F;
    float acc[VPL][VECN];
#pragma unroll
    for (int q = 0; q < VPL; ++q)
#pragma unroll
        for (int i = 0; i < VECN; ++i) acc[q][i] = 0.f;
    auto move_to_second_level = [&]() {
        const float sc = m_tot == -CUDART_INF_F ? 0.f : ex2(m_tot - m);     // m >= m_tot; both -inf before any entry
        m_tot = m;
        tot_s[VPL * VECN][tid] = fmaf(tot_s[VPL * VECN][tid], sc, l);
        l = 0.f;
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int i = 0; i < VECN; ++i) {
                tot_s[q * VECN + i][tid] = fmaf(tot_s[q * VECN + i][tid], sc, acc[q][i]);
                acc[q][i] = 0.f;
            }
    };

    const int n_batches = __reduce_max_sync(kFull, (e - b + EPB - 1) / EPB);
    const bool two_level = n_batches > FLUSH;          // short rows never leave the first level
    if (two_level) {
#pragma unroll
        for (int k = 0; k <= VPL * VECN; ++k) tot_s[k][tid] = 0.f;
    }
    int32_t ucur[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int32_t kk = b + r * S + sl;
        ucur[r] = kk < e ? __ldcs(a.col_idx + kk) : -1;
    }

    for (int ib = 0; ib < n_batches; ++ib) {
        const int32_t kb = b + ib * EPB;
        int32_t unext[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int32_t kk = kb + EPB + r * S + sl;
            unext[r] = kk < e ? __ldcs(a.col_idx + kk) : -1;
        }
        const int buf = ib & 1;
#pragma unroll
        for (int r = 0; r < R; ++r) stage_col[buf][warp][r * 32 + lane] = ucur[r];
        __syncwarp();
        // one group of UB entries: gathers issued together, then one update of the running softmax
        auto steps = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            // in a ragged batch step s works on entries s * EP .. of a row's batch: the steps past the longest
            // remainder in the warp have nothing to do for any lane
            const int rem = FULL ? EPB : __reduce_max_sync(kFull, e - kb);
#pragma unroll
            for (int s0 = 0; s0 < SPB; s0 += UB) {
                if (!FULL && s0 > 0 && s0 * EP >= rem) break;
                Vec<T, VECN> v[UB][VPL];
                float lg[UB];
                bool valid[UB];
#pragma unroll
                for (int i = 0; i < UB; ++i) {
                    const int r = (s0 + i) / LPR, t = (s0 + i) % LPR;
                    const int32_t u = stage_col[buf][warp][r * 32 + seg + t * EP + g];
                    valid[i] = FULL || u >= 0;
                    const uint32_t uu = FULL ? (uint32_t)u : (uint32_t)max(u, 0);
                    lg[i] = valid[i] ? __ldg(ssrc + (size_t)uu * heads) : 0.f;
                    const size_t off = (size_t)uu * ld;
                    if (VPL == 2 && VECN * sizeof(T) == 16 && wide) {
                        if (valid[i]) load_pair(v[i][0], v[i][VPL - 1], zq[0] + off);     // the lane's two vectors are adjacent
                        else { v[i][0].zero(); v[i][VPL - 1].zero(); }
                    } else {
#pragma unroll
                        for (int q = 0; q < VPL; ++q) {
                            if (valid[i]) v[i][q].load(zq[q] + off);
                            else v[i][q].zero();
                        }
                    }
                }
                float mx = m;
#pragma unroll
                for (int i = 0; i < UB; ++i) {
                    lg[i] = leaky2(lg[i] + sd);
                    if (valid[i]) mx = fmaxf(mx, lg[i]);
                }
                if (FULL || mx != -CUDART_INF_F) {      // a group with no entry at all leaves the state alone
                    const float rescale = ex2(m - mx);  // 2^-inf = 0 on the first group
                    m = mx;
                    l *= rescale;
#pragma unroll
                    for (int q = 0; q < VPL; ++q)
#pragma unroll
                        for (int i = 0; i < VECN; ++i) acc[q][i] *= rescale;
                }
#pragma unroll
                for (int i = 0; i < UB; ++i) {
                    // hardware 2^x: the argument is <= 0 and its error (about 2 ulp + |x| * 2^-23 relative) stays
                    // two orders below the 1e-5 bound on the weighted sum
                    const float p = valid[i] ? ex2(lg[i] - m) : 0.f;
                    l += p;
#pragma unroll
                    for (int q = 0; q < VPL; ++q)
#pragma unroll
                        for (int k = 0; k < VECN; ++k) acc[q][k] = fmaf(p, v[i][q].get(k), acc[q][k]);
                }
            }
        };
        if (__all_sync(kFull, kb + EPB <= e)) steps(std::true_type{});
        else steps(std::false_type{});
#pragma unroll
        for (int r = 0; r < R; ++r) ucur[r] = unext[r];
        if (two_level && (ib + 1) % FLUSH == 0) move_to_second_level();
    }
    if (two_level) {
        move_to_second_level();
        l = tot_s[VPL * VECN][tid];
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int i = 0; i < VECN; ++i) acc[q][i] = tot_s[q * VECN + i][tid];
    }

    // merge the EP groups of the row, fixed tree
#pragma unroll
    for (int o = S / 2; o >= LPR; o >>= 1) {
        const float m2 = __shfl_down_sync(kFull, m, o, S);
        const float l2 = __shfl_down_sync(kFull, l, o, S);
        const float mn = fmaxf(m, m2);
        const float sa = merge_scale(m, mn), sb = merge_scale(m2, mn);
        l = l * sa + l2 * sb;
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int i = 0; i < VECN; ++i) {
                const float a2 = __shfl_down_sync(kFull, acc[q][i], o, S);
                acc[q][i] = acc[q][i] * sa + a2 * sb;
            }
        m = mn;
    }

    if (!active || g != 0 || !lane_ok) return;
    // where a hub segment's partial results go (read here, at the end, so that it occupies no register during the walk)
    const int32_t part = rg.hub ? a.seg_slot[slot] : 0;
    if (rg.hub) {
        // every lane of a head holds the same (m, l); the first lane of each head inside this column tile stores
        // it (sweeps that share a head store identical values)
        if (j0 % a.dim == 0 || c == 0) {
            float* ml = a.partial_ml + ((int64_t)part * a.heads + h) * 2;
            ml[0] = m;
            ml[1] = l;
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
        if (!okq[q]) continue;
        const int j = j0 + q * VECN;
        if (rg.hub) {
            float* p = a.partial + (int64_t)part * a.fpad + j;
#pragma unroll
            for (int i = 0; i < VECN; ++i)
                if (j + i < chunk_end) p[i] = acc[q][i];
        } else {
            const int64_t o = (int64_t)row * a.ldo + j;
#pragma unroll
            for (int i = 0; i < VECN; ++i)
                if (j + i < chunk_end) store_elem(a.out, a.out_bf16, o + i, acc[q][i] * inv);
        }
    }
}

template <typename T, int VECN, int LPR, int VPL>
// Register budget: left to itself the compiler gives the wide instantiations anything between 80 and 126
// registers from one build to the next (two blocks per SM instead of three, 20 % slower); three blocks per SM for
// the vector-pair forms and four for the others is what the measured-good builds had.
__global__ void __launch_bounds__(kBlock, (VPL == 2 && VECN > 1) ? 3 : 4) gat_aggregate(const __grid_constant__ GatArgs a)
{
    __shared__ int32_t stage_col[2][kBlock / 32][kStageSlots];
    __shared__ float tot_s[VPL * VECN + 1][kBlock];        // second-level sums and denominator, one column per thread
    // grid: x = (block of the sweep, column tile), y = chunk; blocks are issued x first, so the sweeps follow each
    // other chunk by chunk.  (The chunk used to be divided out of a linear 64-bit block number: two 64-bit
    // divisions per thread, more instructions than a short row's whole walk.)
    const int chunk = a.chunk_base + (int)blockIdx.y;
    const unsigned n_ct = (unsigned)a.n_ctiles;
    const int rb = n_ct == 1 ? (int)blockIdx.x : (int)(blockIdx.x / n_ct);
    const int ctile = n_ct == 1 ? 0 : (int)(blockIdx.x % n_ct);
    const int chunk_begin = chunk * a.chunk_width;
    const int chunk_end = min(a.f, chunk_begin + a.chunk_width);
    const int col0 = chunk_begin + ctile * (LPR * VPL * VECN);
    if (col0 >= chunk_end) return;
    int r = 0;
#pragma unroll
    for (int i = 1; i < kMaxRanges; ++i)
        if (i < a.n_ranges && rb >= a.range[i].first_block) r = i;
    const Range rg = a.range[r];
    const int bir = rb - rg.first_block;
    switch (rg.ep_log2) {
        case 0: gat_rows<T, VECN, LPR, VPL, 1>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
        case 1: if constexpr (LPR * 2 <= 32) gat_rows<T, VECN, LPR, VPL, 2>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
        case 2: if constexpr (LPR * 4 <= 32) gat_rows<T, VECN, LPR, VPL, 4>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
        case 3: if constexpr (LPR * 8 <= 32) gat_rows<T, VECN, LPR, VPL, 8>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
        case 4: if constexpr (LPR * 16 <= 32) gat_rows<T, VECN, LPR, VPL, 16>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
        default: if constexpr (LPR == 1) gat_rows<T, VECN, LPR, VPL, 32>(a, rg, bir, col0, chunk_end, stage_col, tot_s); break;
    }
}

// out[row, j] = sum_s partial[s, j] e^(m_s - M) / sum_s l_s e^(m_s - M) over the segments s of a hub row.
// A block covers kReduceCols columns of one row; kReduceWays threads per column walk interleaved
// segments and their results are combined in a fixed order through shared memory.
constexpr int kReduceCols = 64;
constexpr int kReduceWays = kBlock / kReduceCols;

__global__ void __launch_bounds__(kBlock)
gat_hub_reduce(const int32_t* __restrict__ row_order, const int32_t* __restrict__ hub_seg_ptr,
               const float* __restrict__ partial, const float* __restrict__ partial_ml, int64_t hub_begin, int32_t n_hub,
               int32_t f, int32_t fpad, int32_t heads, int32_t dim, void* __restrict__ out, int64_t ldo, int out_bf16)
{
    __shared__ float s_max[kReduceWays][kReduceCols], s_num[kReduceWays][kReduceCols], s_den[kReduceWays][kReduceCols];
    const int i = blockIdx.x;
    const int c = threadIdx.x % kReduceCols, q = threadIdx.x / kReduceCols;
    const int j = blockIdx.y * kReduceCols + c;
    const bool ok = j < f;
    const int h = ok ? j / dim : 0;
    const int32_t row = row_order[hub_begin + i];
    const int32_t s0 = hub_seg_ptr[i], s1 = hub_seg_ptr[i + 1];
    float mx = -CUDART_INF_F;
    if (ok)
        for (int32_t s = s0 + q; s < s1; s += kReduceWays) mx = fmaxf(mx, partial_ml[((int64_t)s * heads + h) * 2]);
    s_max[q][c] = mx;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kReduceWays; ++w) mx = fmaxf(mx, s_max[w][c]);
    float num = 0.f, den = 0.f;
    if (ok) {
        float num_run = 0.f, den_run = 0.f;
        int in_run = 0;
        for (int32_t s = s0 + q; s < s1; s += kReduceWays) {
            const float* ml = partial_ml + ((int64_t)s * heads + h) * 2;
            const float w = merge_scale(ml[0], mx);
            den_run = fmaf(ml[1], w, den_run);
            num_run = fmaf(partial[(int64_t)s * fpad + j], w, num_run);
            if (++in_run == 32) { num += num_run; den += den_run; num_run = den_run = 0.f; in_run = 0; }   // short chains
        }
        num += num_run;
        den += den_run;
    }
    s_num[q][c] = num;
    s_den[q][c] = den;
    __syncthreads();
    if (q != 0 || !ok) return;
    num = 0.f;
    den = 0.f;
#pragma unroll
    for (int w = 0; w < kReduceWays; ++w) { num += s_num[w][c]; den += s_den[w][c]; }
    store_elem(out, out_bf16, (int64_t)row * ldo + j, den > 0.f ? num / den : 0.f);
}

// ------------------------------------------------------------------ host side

typedef void (*GatKernel)(const GatArgs);

template <typename T, int VECN, int VPL>
static GatKernel pick_lpr(int lpr)
{
    switch (lpr) {
        case 1: return gat_aggregate<T, VECN, 1, VPL>;
        case 2: return gat_aggregate<T, VECN, 2, VPL>;
        case 4: return gat_aggregate<T, VECN, 4, VPL>;
        case 8: return gat_aggregate<T, VECN, 8, VPL>;
        case 16: return gat_aggregate<T, VECN, 16, VPL>;
        default: return gat_aggregate<T, VECN, 32, VPL>;
    }
}

template <typename T, int VECN>
static GatKernel pick_vpl(int lpr, int vpl)
{
    return vpl == 2 ? pick_lpr<T, VECN, 2>(lpr) : pick_lpr<T, VECN, 1>(lpr);
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

// scores_ready: the two score arrays at the head of the scratch buffer (see gat_scratch_scores) already hold the
// scores of d_z (the dense transform's epilogue wrote them), so the scores pass is left out.
int gat_aggregate_impl(const gnnfd_csr_t* csr, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src,
                       const float* d_a_dst, int32_t heads, int32_t dim, float negative_slope, void* d_out, int64_t ldo,
                       gnnfd_dtype_t odt, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, bool scores_ready,
                       cudaStream_t s)
{
    if (!csr || !d_z || !d_out || heads <= 0 || dim <= 0 || chunk_width <= 0) return GNNFD_INVALID_ARG;
    if (!scores_ready && (!d_a_src || !d_a_dst)) return GNNFD_INVALID_ARG;
    const int64_t f64 = (int64_t)heads * dim;
    if (f64 > 0x7fffffffll || ldz < f64 || ldo < f64 || ldz > 0x7fffffffll) return GNNFD_INVALID_ARG;
    if ((zdt != GNNFD_F32 && zdt != GNNFD_BF16) || (odt != GNNFD_F32 && odt != GNNFD_BF16)) return GNNFD_UNSUPPORTED;
    if (!d_scratch || ((uintptr_t)d_scratch & 255u)) return GNNFD_INVALID_ARG;
    const int32_t f = (int32_t)f64;
    Carver c(d_scratch, scratch_bytes);
    GatScratch g;
    carve_gat(c, csr, heads, dim, &g);
    if (!c.ok) return GNNFD_WORKSPACE_TOO_SMALL;
    if (!scores_ready) {
        int rc = launch_scores(csr->n, d_z, ldz, zdt, d_a_src, d_a_dst, heads, dim, g.s_src, g.s_dst, s);
        if (rc) return rc;
    }

    const int cw = chunk_width < f ? chunk_width : f;
    const int n_chunks = (f + cw - 1) / cw;
    const int zsize = zdt == GNNFD_F32 ? 4 : 2;
    const int vecn = 16 / zsize;
    // a lane's vector must start 16-byte aligned and stay inside one head
    const bool vec = ((uintptr_t)d_z % 16 == 0) && ((ldz * zsize) % 16 == 0) && (n_chunks == 1 || cw % vecn == 0) &&
                     (dim % vecn == 0);
    const int elems = vec ? vecn : 1;
    // a lane covers two adjacent vectors when both stay inside one head and chunks start on such pairs
    const int vectors = (cw + elems - 1) / elems;
    const int vpl = (vectors > 1 && dim % (2 * elems) == 0 && (n_chunks == 1 || cw % (2 * elems) == 0)) ? 2 : 1;
    int lpr = 1;
    while (lpr * vpl < vectors && lpr < 32) lpr <<= 1;

    GatArgs a;
    a.row_ptr = csr->row_ptr; a.col_idx = csr->col_idx; a.row_order = csr->row_order;
    a.seg_row = csr->seg_row; a.seg_begin = csr->seg_begin; a.seg_end = csr->seg_end; a.seg_slot = csr->seg_slot;
    a.s_src = g.s_src; a.s_dst = g.s_dst; a.z = d_z; a.out = d_out;
    a.partial = g.partial; a.partial_ml = g.partial_ml;
    a.ldz = ldz; a.ldo = ldo; a.slope = negative_slope;
    a.f = f; a.heads = heads; a.dim = dim; a.chunk_width = cw;
    a.n_ctiles = (cw + lpr * vpl * elems - 1) / (lpr * vpl * elems);
    a.fpad = (int32_t)align_up((size_t)f, 4);
    a.out_bf16 = odt == GNNFD_BF16;
    // 32-byte loads of a lane's vector pair need every pair to start on a 32-byte boundary
    a.wide_ok = vec && vpl == 2 && ((uintptr_t)d_z % 32 == 0) && ((ldz * zsize) % 32 == 0) &&
                (n_chunks == 1 || (cw * zsize) % 32 == 0);

    const int64_t blocks = plan_ranges(csr, lpr, a.range, &a.n_ranges);
    a.blocks_per_tile = (int32_t)blocks;
    const int64_t grid_x = blocks * a.n_ctiles;
    if (grid_x > 0x7fffffffll) return GNNFD_TOO_LARGE;
    if (grid_x > 0) {
        GatKernel kernel;
        if (zdt == GNNFD_F32) kernel = vec ? pick_vpl<float, 4>(lpr, vpl) : pick_vpl<float, 1>(lpr, vpl);
        else kernel = vec ? pick_vpl<__nv_bfloat16, 8>(lpr, vpl) : pick_vpl<__nv_bfloat16, 1>(lpr, vpl);
        for (int c0 = 0; c0 < n_chunks; c0 += kMaxGridY) {
            a.chunk_base = c0;
            const dim3 grid((unsigned)grid_x, (unsigned)(n_chunks - c0 < kMaxGridY ? n_chunks - c0 : kMaxGridY));
            GNNFD_LAUNCH("gat_aggregate", s, kernel, grid, kBlock, 0, a);
        }
    }
    const int64_t n_hub = csr->bin_count[4];
    if (n_hub > 0) {
        dim3 gr((unsigned)n_hub, (unsigned)((f + kReduceCols - 1) / kReduceCols));
        GNNFD_LAUNCH("gat_hub_reduce", s, gat_hub_reduce, gr, kBlock, 0, csr->row_order, csr->hub_seg_ptr, g.partial,
                     g.partial_ml, csr->bin_start[4], (int32_t)n_hub, f, a.fpad, heads, dim, d_out, ldo, a.out_bf16);
    }
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

// where gnnfd_aggregate_gat keeps the two [n, heads] score arrays inside its scratch buffer
int gat_scratch_scores(const gnnfd_csr_t* csr, int32_t heads, int32_t dim, void* d_scratch, size_t scratch_bytes,
                       float** s_src, float** s_dst)
{
    if (!csr || heads <= 0 || dim <= 0 || !d_scratch || ((uintptr_t)d_scratch & 255u)) return GNNFD_INVALID_ARG;
    Carver c(d_scratch, scratch_bytes);
    GatScratch g;
    carve_gat(c, csr, heads, dim, &g);
    if (!c.ok) return GNNFD_WORKSPACE_TOO_SMALL;
    *s_src = g.s_src;
    *s_dst = g.s_dst;
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
    return gnnfd::gat_aggregate_impl(csr, d_z, ldz, zdt, d_a_src, d_a_dst, heads, dim, negative_slope, d_out, ldo, odt,
                                     chunk_width, d_scratch, scratch_bytes, false, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
