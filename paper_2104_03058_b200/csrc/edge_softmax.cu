// Materialised edge softmax: alpha[k, h] for every CSR slot k from caller-supplied scores.
//
// Logit of slot k of row v, head h: LeakyReLU(s_src[col_idx[k], h] + s_dst[v, h]); alpha is the softmax
// over the slots of the row.  The work is cut exactly as in the gather kernels: rows come sorted by
// degree class and a row is shared by more lanes the longer its class; a hub row is cut into segments
// of GNNFD_HUB_SEGMENT slots, one warp each, so that no unit of work is longer than a segment.  The
// heads of a slot are spread over LPS adjacent lanes, four heads (one 16-byte access) each, and SP
// slots are worked on side by side, so the lanes of a row read the scores of a slot and write its
// alphas as one contiguous piece, and consecutive slots follow each other in memory.
//
// An ordinary row is done by its lanes in one go: a running (max, sum) over the row, a fixed
// butterfly merge across the lanes, then the write pass (the logits stay in registers when the row
// fits one batch, otherwise they are gathered again: the row's indices and scores are cache hits).
// Hub rows take three launches: per-segment (max, sum), a merge per row in ascending segment order,
// and the write pass per segment.  Nothing waits on another block and nothing is accumulated
// atomically, so the result is the same bit for bit from run to run.
//
// The exponentials are base-2 (logits pre-multiplied by log2 e): the argument is rounded once more
// than with expf, which moves a result by about |logit| * 6e-8 relative (the fp32 sum s_src + s_dst
// already carries an error of that size).
#include <math_constants.h>

#include "schedule.cuh"

namespace gnnfd {

#ifndef GNNFD_SOFTMAX_IN_FLIGHT
#define GNNFD_SOFTMAX_IN_FLIGHT 4
#endif
#ifndef GNNFD_SOFTMAX_MIN_BLOCKS
#define GNNFD_SOFTMAX_MIN_BLOCKS 4
#endif
// slots a lane has in flight when it holds HB heads of a slot: GNNFD_SOFTMAX_IN_FLIGHT 16-byte loads' worth, at most 16
template <int HB> constexpr int slots_in_flight()
{
    return GNNFD_SOFTMAX_IN_FLIGHT * 4 / HB > 16 ? 16 : GNNFD_SOFTMAX_IN_FLIGHT * 4 / HB < 2 ? 2 : GNNFD_SOFTMAX_IN_FLIGHT * 4 / HB;
}
constexpr float kLog2e = 1.4426950408889634f;

struct SoftmaxArgs {
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* row_order;
    const int32_t* seg_row;
    const int32_t* seg_begin;
    const int32_t* seg_end;
    const int32_t* seg_slot;
    const int32_t* hub_seg_ptr;
    const float* s_src;
    const float* s_dst;
    float* alpha;
    float2* seg_stats;       // [n_segments, heads]: (max, sum) of a segment, later (max, 1 / sum) of its row
    float slope;
    int32_t heads;
    int32_t n_hub;
    int32_t n_ranges;
    Range range[kMaxRanges];
};

enum { kModeRows = 0, kModeHubStats = 1, kModeHubWrite = 2 };

template <int HB>
__device__ __forceinline__ void load_heads(const float* p, float (&v)[HB])
{
    if constexpr (HB % 4 == 0) {
#pragma unroll
        for (int i = 0; i < HB; i += 4) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(p + i));
            v[i] = q.x; v[i + 1] = q.y; v[i + 2] = q.z; v[i + 3] = q.w;
        }
    } else if constexpr (HB == 2) {
        const float2 q = __ldg(reinterpret_cast<const float2*>(p));
        v[0] = q.x; v[1] = q.y;
    } else {
        v[0] = __ldg(p);
    }
}

template <int HB>
__device__ __forceinline__ void store_heads(float* p, const float (&v)[HB])
{
    if constexpr (HB % 4 == 0) {
#pragma unroll
        for (int i = 0; i < HB; i += 4) __stcs(reinterpret_cast<float4*>(p + i), make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]));
    } else if constexpr (HB == 2) {
        __stcs(reinterpret_cast<float2*>(p), make_float2(v[0], v[1]));
    } else {
        __stcs(p, v[0]);
    }
}

// 2^x by the hardware approximation (2 ulp; results below 2^-126 become 0, 2^-inf = 0)
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// share of a partial result with maximum m under the merged maximum mx (both may be -inf)
__device__ __forceinline__ float rescale(float m, float mx) { return m == -CUDART_INF_F ? 0.f : ex2(m - mx); }

// LeakyReLU(x) * log2 e written as c1 * x + c2 * |x| with c1 = log2 e * (1 + slope) / 2 and
// c2 = log2 e * (1 - slope) / 2: two instructions per logit and no branch, for any slope.
struct Leaky {
    float c1, c2;
    __device__ __forceinline__ explicit Leaky(float slope) : c1(0.5f * kLog2e * (1.f + slope)), c2(0.5f * kLog2e * (1.f - slope)) {}
    __device__ __forceinline__ float operator()(float x) const { return fmaf(fabsf(x), c2, x * c1); }
};

// column indices of slots k, k + SP, ... of one row (-1 past the end of the row)
template <int SP, int NF>
__device__ __forceinline__ void load_cols(const SoftmaxArgs& a, int32_t k, int32_t e, int32_t (&u)[NF])
{
#pragma unroll
    for (int i = 0; i < NF; ++i) u[i] = k + i * SP < e ? __ldg(a.col_idx + k + i * SP) : -1;
}

// base-2 logits of the slots whose column indices are u[].  FULL: all of them exist; otherwise the
// missing ones (u < 0) get -inf.
template <int HB, bool FULL, int NF>
__device__ __forceinline__ void load_logits(const SoftmaxArgs& a, const Leaky& leaky, const float* ssrc, const float (&sd)[HB],
                                            const int32_t (&u)[NF], float (&t)[NF][HB])
{
#pragma unroll
    for (int i = 0; i < NF; ++i) {
        if (FULL || u[i] >= 0) {
            load_heads<HB>(ssrc + (int64_t)u[i] * a.heads, t[i]);
        } else {
#pragma unroll
            for (int h = 0; h < HB; ++h) t[i][h] = 0.f;
        }
    }
#pragma unroll
    for (int i = 0; i < NF; ++i)
#pragma unroll
        for (int h = 0; h < HB; ++h) {
            const float y = leaky(t[i][h] + sd[h]);
            t[i][h] = (FULL || u[i] >= 0) ? y : -CUDART_INF_F;
        }
}

// running (max, sum) of one head over a batch of logits
template <int HB, int NF>
__device__ __forceinline__ void online_update(const float (&t)[NF][HB], float (&m)[HB], float (&l)[HB])
{
#pragma unroll
    for (int h = 0; h < HB; ++h) {
        float mx = m[h];                                               // t[0] is a real slot, so mx ends finite
#pragma unroll
        for (int i = 0; i < NF; ++i) mx = fmaxf(mx, t[i][h]);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < NF; ++i) sum += ex2(t[i][h] - mx);                  // 2^-inf = 0
        l[h] = l[h] * ex2(m[h] - mx) + sum;
        m[h] = mx;
    }
}

// One row (or hub segment) per S = LPS * SP lanes: SP slots are worked on side by side, and the heads
// of a slot are spread over LPS lanes holding HB heads each (LPS * HB heads per round; more heads take
// more rounds over the row).
template <int HB, int LPS, int SP, int MODE>
__device__ __forceinline__ void softmax_items(const SoftmaxArgs& a, const Range& rg, int block_in_range)
{
    constexpr int S = LPS * SP;
    constexpr int NF = slots_in_flight<HB>();
    constexpr unsigned kFull = 0xffffffffu;
    const int tid = threadIdx.x;
    const int slot = block_in_range * (kBlock / S) + tid / S;
    const int sl = tid % S;
    const int hb = sl % LPS;             // which block of HB heads of a slot
    const int sp = sl / LPS;             // which of the SP slots of a step
    const bool active = slot < rg.item_count;
    int32_t row = 0, b = 0, e = 0, part = 0;      // part: where a hub segment's (max, sum) lives
    if (active) {
        if (rg.hub) {
            row = a.seg_row[slot];
            b = a.seg_begin[slot];
            e = a.seg_end[slot];
            part = a.seg_slot[slot];
        } else {
            row = a.row_order[rg.item_begin + slot];
            b = a.row_ptr[row];
            e = a.row_ptr[row + 1];
        }
    }
    // every row of the warp fits one batch: the write pass reuses the logits of the first pass
    const bool fits = MODE == kModeRows && __all_sync(kFull, e - b <= SP * NF);
    const Leaky leaky(a.slope);

    for (int hh = 0; hh < a.heads; hh += LPS * HB) {
        const int h0 = hh + hb * HB;
        const bool head_ok = h0 < a.heads;
        float sd[HB];
#pragma unroll
        for (int h = 0; h < HB; ++h) sd[h] = 0.f;
        if (active && head_ok) load_heads<HB>(a.s_dst + (int64_t)row * a.heads + h0, sd);
        const float* ssrc = a.s_src + h0;
        float m[HB], inv[HB];
        float t[NF][HB];

        if (MODE != kModeHubWrite) {
            float l[HB];
#pragma unroll
            for (int h = 0; h < HB; ++h) { m[h] = -CUDART_INF_F; l[h] = 0.f; }
            if (head_ok) {
                int32_t u[NF], un[NF];
                load_cols<SP, NF>(a, b + sp, e, u);
                for (int32_t kb = b; kb < e; kb += SP * NF) {
                    // the next batch's indices are on their way while this batch is gathered and reduced
                    load_cols<SP, NF>(a, kb + SP * NF + sp, e, un);
                    if (kb + SP * NF <= e) {               // the same for all lanes of the row
                        load_logits<HB, true, NF>(a, leaky, ssrc, sd, u, t);
                        online_update<HB, NF>(t, m, l);
                    } else if (u[0] >= 0) {
                        load_logits<HB, false, NF>(a, leaky, ssrc, sd, u, t);
                        online_update<HB, NF>(t, m, l);
                    }
#pragma unroll
                    for (int i = 0; i < NF; ++i) u[i] = un[i];
                }
            }
            // butterfly over the SP lanes that hold the same heads; both partners evaluate the same commutative expression
            if constexpr (SP > 1) {
#pragma unroll
                for (int o = S / 2; o >= LPS; o >>= 1)
#pragma unroll
                    for (int h = 0; h < HB; ++h) {
                        const float mo = __shfl_xor_sync(kFull, m[h], o);
                        const float lo = __shfl_xor_sync(kFull, l[h], o);
                        const float mx = fmaxf(m[h], mo);
                        l[h] = __fadd_rn(__fmul_rn(l[h], rescale(m[h], mx)), __fmul_rn(lo, rescale(mo, mx)));
                        m[h] = mx;
                    }
            }
            if constexpr (MODE == kModeHubStats) {
                if (active && head_ok && sp == 0) {
#pragma unroll
                    for (int h = 0; h < HB; ++h) a.seg_stats[(int64_t)part * a.heads + h0 + h] = make_float2(m[h], l[h]);
                }
            }
#pragma unroll
            for (int h = 0; h < HB; ++h) inv[h] = 1.f / l[h];          // unused (inf) for an empty row
        } else {
#pragma unroll
            for (int h = 0; h < HB; ++h) {
                const float2 st = (active && head_ok) ? a.seg_stats[(int64_t)part * a.heads + h0 + h] : make_float2(0.f, 0.f);
                m[h] = st.x;
                inv[h] = st.y;
            }
        }
        if (MODE == kModeHubStats || !head_ok) continue;

        if (fits) {
#pragma unroll
            for (int i = 0; i < NF; ++i) {
                const int32_t k = b + sp + i * SP;
                if (k < e) {
                    float w[HB];
#pragma unroll
                    for (int h = 0; h < HB; ++h) w[h] = ex2(t[i][h] - m[h]) * inv[h];
                    store_heads<HB>(a.alpha + (int64_t)k * a.heads + h0, w);
                }
            }
        } else {
            int32_t u[NF], un[NF];
            load_cols<SP, NF>(a, b + sp, e, u);
            for (int32_t kb = b; kb < e; kb += SP * NF) {
                const int32_t k = kb + sp;
                load_cols<SP, NF>(a, k + SP * NF, e, un);
                if (kb + SP * NF <= e) {
                    load_logits<HB, true, NF>(a, leaky, ssrc, sd, u, t);
#pragma unroll
                    for (int i = 0; i < NF; ++i) {
                        float w[HB];
#pragma unroll
                        for (int h = 0; h < HB; ++h) w[h] = ex2(t[i][h] - m[h]) * inv[h];
                        store_heads<HB>(a.alpha + (int64_t)(k + i * SP) * a.heads + h0, w);
                    }
                } else if (u[0] >= 0) {
                    load_logits<HB, false, NF>(a, leaky, ssrc, sd, u, t);
#pragma unroll
                    for (int i = 0; i < NF; ++i) {
                        if (u[i] >= 0) {
                            float w[HB];
#pragma unroll
                            for (int h = 0; h < HB; ++h) w[h] = ex2(t[i][h] - m[h]) * inv[h];
                            store_heads<HB>(a.alpha + (int64_t)(k + i * SP) * a.heads + h0, w);
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < NF; ++i) u[i] = un[i];
            }
        }
    }
}

// All ordinary rows (stats and write in one go) and, in the same grid, the write pass of the hub segments.
template <int HB, int LPS>
__global__ void __launch_bounds__(kBlock, GNNFD_SOFTMAX_MIN_BLOCKS) edge_softmax_rows(const __grid_constant__ SoftmaxArgs a)
{
    const int rb = blockIdx.x;
    int r = 0;
#pragma unroll
    for (int i = 1; i < kMaxRanges; ++i)
        if (i < a.n_ranges && rb >= a.range[i].first_block) r = i;
    const Range rg = a.range[r];
    const int bir = rb - rg.first_block;
    if (rg.hub) { softmax_items<HB, LPS, 32 / LPS, kModeHubWrite>(a, rg, bir); return; }
    switch (rg.ep_log2) {
        case 0: softmax_items<HB, LPS, 1, kModeRows>(a, rg, bir); break;
        case 1: if constexpr (LPS * 2 <= 32) softmax_items<HB, LPS, 2, kModeRows>(a, rg, bir); break;
        case 2: if constexpr (LPS * 4 <= 32) softmax_items<HB, LPS, 4, kModeRows>(a, rg, bir); break;
        case 3: if constexpr (LPS * 8 <= 32) softmax_items<HB, LPS, 8, kModeRows>(a, rg, bir); break;
        case 4: if constexpr (LPS * 16 <= 32) softmax_items<HB, LPS, 16, kModeRows>(a, rg, bir); break;
        default: if constexpr (LPS == 1) softmax_items<HB, LPS, 32, kModeRows>(a, rg, bir); break;
    }
}

// (max, sum) of every hub segment; range 0 of the plan is the hub range
template <int HB, int LPS>
__global__ void __launch_bounds__(kBlock, GNNFD_SOFTMAX_MIN_BLOCKS) edge_softmax_hub_stats(const __grid_constant__ SoftmaxArgs a)
{
    softmax_items<HB, LPS, 32 / LPS, kModeHubStats>(a, a.range[0], blockIdx.x);
}

// One thread per (hub row, head): merges the segment results in ascending segment order and leaves the
// row's (max, 1 / sum) in every segment's entry.
__global__ void __launch_bounds__(kBlock) edge_softmax_hub_merge(const __grid_constant__ SoftmaxArgs a)
{
    const int64_t idx = (int64_t)blockIdx.x * kBlock + threadIdx.x;
    if (idx >= (int64_t)a.n_hub * a.heads) return;
    const int i = (int)(idx / a.heads), h = (int)(idx % a.heads);
    const int32_t s0 = a.hub_seg_ptr[i], s1 = a.hub_seg_ptr[i + 1];
    float m = -CUDART_INF_F;
    for (int32_t s = s0; s < s1; ++s) m = fmaxf(m, a.seg_stats[(int64_t)s * a.heads + h].x);
    float l = 0.f, run = 0.f;                      // runs of 32 segments: a row of very many segments keeps short chains
    for (int32_t s = s0; s < s1; ++s) {
        const float2 st = a.seg_stats[(int64_t)s * a.heads + h];
        run += st.y * rescale(st.x, m);
        if (((s - s0) & 31) == 31) { l += run; run = 0.f; }
    }
    l += run;
    const float2 row_stats = make_float2(m, 1.f / l);
    for (int32_t s = s0; s < s1; ++s) a.seg_stats[(int64_t)s * a.heads + h] = row_stats;
}

static size_t softmax_scratch_bytes(const gnnfd_csr_t* csr, int32_t heads)
{
    return align_up((size_t)csr->n_segments * (size_t)heads * sizeof(float2), 256);
}

template <int HB, int LPS>
static int launch_softmax(const gnnfd_csr_t* csr, SoftmaxArgs& a, cudaStream_t s)
{
    const int64_t blocks = plan_ranges(csr, LPS, a.range, &a.n_ranges);
    if (blocks > 0x7fffffffll) return GNNFD_TOO_LARGE;
    if (blocks == 0) return GNNFD_OK;
    if (csr->n_segments > 0) {
        const unsigned hub_blocks = (unsigned)((csr->n_segments + kBlock / 32 - 1) / (kBlock / 32));
        GNNFD_LAUNCH("edge_softmax_hub_stats", s, (edge_softmax_hub_stats<HB, LPS>), hub_blocks, kBlock, 0, a);
        const int64_t pairs = (int64_t)a.n_hub * a.heads;
        GNNFD_LAUNCH("edge_softmax_hub_merge", s, edge_softmax_hub_merge, (unsigned)((pairs + kBlock - 1) / kBlock), kBlock,
                     0, a);
    }
    GNNFD_LAUNCH("edge_softmax_rows", s, (edge_softmax_rows<HB, LPS>), (unsigned)blocks, kBlock, 0, a);
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" {

int gnnfd_edge_softmax_workspace_bytes(const gnnfd_csr_t* csr, int32_t heads, size_t* scratch_bytes)
{
    if (!csr || heads <= 0 || !scratch_bytes) return GNNFD_INVALID_ARG;
    *scratch_bytes = gnnfd::softmax_scratch_bytes(csr, heads);
    return GNNFD_OK;
}

int gnnfd_edge_softmax(const gnnfd_csr_t* csr, const float* d_s_src, const float* d_s_dst, int32_t heads,
                       float negative_slope, float* d_alpha, void* d_scratch, size_t scratch_bytes, void* stream)
{
    using namespace gnnfd;
    if (!csr || !d_s_src || !d_s_dst || heads <= 0 || (!d_alpha && csr->nnz > 0)) return GNNFD_INVALID_ARG;
    if (csr->nnz == 0) return GNNFD_OK;
    const size_t need = softmax_scratch_bytes(csr, heads);
    if (need > 0 && (!d_scratch || scratch_bytes < need)) return GNNFD_WORKSPACE_TOO_SMALL;
    if (need > 0 && ((uintptr_t)d_scratch & 7u)) return GNNFD_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    SoftmaxArgs a;
    a.row_ptr = csr->row_ptr; a.col_idx = csr->col_idx; a.row_order = csr->row_order;
    a.seg_row = csr->seg_row; a.seg_begin = csr->seg_begin; a.seg_end = csr->seg_end; a.seg_slot = csr->seg_slot;
    a.hub_seg_ptr = csr->hub_seg_ptr;
    a.s_src = d_s_src; a.s_dst = d_s_dst; a.alpha = d_alpha; a.seg_stats = static_cast<float2*>(d_scratch);
    a.slope = negative_slope; a.heads = heads; a.n_hub = (int32_t)csr->bin_count[4];

    // heads per lane (HB) and lanes per slot (LPS): 16-byte accesses when heads is a multiple of 4 and the
    // pointers allow it, with the heads of a slot spread over up to 8 lanes so that a warp's accesses to
    // alpha are contiguous; otherwise one lane per slot with 8- or 4-byte accesses
    const uintptr_t ptrs = (uintptr_t)d_s_src | (uintptr_t)d_s_dst | (uintptr_t)d_alpha;
    if (heads % 4 == 0 && ptrs % 16 == 0) {
        const int blocks4 = heads / 4;
        if (blocks4 % 8 == 0) return launch_softmax<4, 8>(csr, a, s);
        if (blocks4 % 4 == 0) return launch_softmax<4, 4>(csr, a, s);
        if (blocks4 % 2 == 0) return launch_softmax<4, 2>(csr, a, s);
        return launch_softmax<4, 1>(csr, a, s);
    }
    if (heads % 2 == 0 && ptrs % 8 == 0) return launch_softmax<2, 1>(csr, a, s);
    return launch_softmax<1, 1>(csr, a, s);
}

}  // extern "C"
