// Chunked gather-aggregate for GCN and GraphSAGE (Algorithm 1: Message + Aggregate per decomposition
// layer, Concat by writing each chunk into its own output columns) and the second-level reduction
// of hub rows.
//
// Work decomposition.  One launch sweeps the chunks one after the other (the block index is
// chunk-major), so at any time the blocks in flight gather from one chunk's n x chunk_width slice of
// x, which is what keeps the gathered working set small enough for L2.  Inside a sweep the rows come
// grouped by degree class.  A row is owned by S = LPR * EP lanes: LPR lanes cover the chunk's columns
// with one or two 16-byte vectors each, and EP groups of LPR lanes walk interleaved entries of the
// row, each keeping 8 loads in flight; column indices and edge weights are staged per warp in shared memory.  The EP partial sums are combined by a fixed shuffle tree, hub rows
// (degree > GNNFD_HUB_DEGREE) by per-segment partial sums that a second kernel adds in ascending
// segment order: no atomics, bit-identical from run to run.
#include "schedule.cuh"
#include "vec.cuh"

namespace gnnfd {

struct GatherArgs {
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const float* edge_w;
    const float* rdeg;
    const int32_t* row_order;
    const int32_t* seg_row;
    const int32_t* seg_begin;
    const int32_t* seg_end;
    const int32_t* seg_slot;
    const void* x;
    void* out;
    float* partial;
    int64_t ldx, ldo;
    int32_t f, chunk_width, n_ctiles, blocks_per_tile, fpad, out_bf16, out_vec_ok, wide_ok;
    int32_t chunk_base;      // first chunk of this launch (a launch covers at most 65,535 chunks)
    int32_t n_ranges;
    Range range[kMaxRanges];
};

#ifndef GNNFD_GATHER_LOADS
#define GNNFD_GATHER_LOADS 8
#endif
#ifndef GNNFD_GATHER_MIN_BLOCKS
#define GNNFD_GATHER_MIN_BLOCKS 3
#endif
constexpr int kLoads = GNNFD_GATHER_LOADS;      // 16-byte feature loads kept in flight per lane

constexpr int kStageSlots = kLoads * 32;      // column indices (and weights) a warp stages per batch, at most

// One row (or hub segment) per S = LPR * EP lanes.  The S lanes fetch the row's indices and weights
// S at a time with one coalesced streaming load each (R rounds per batch) and stage them in the
// warp's shared-memory buffer (double-buffered; the next batch is already in registers, on its way
// from HBM, while this one is consumed).  In step s of a batch, group g works on entry
// r*S + t*EP + g (r = s / LPR, t = s % LPR), read back as a broadcast.  A lane covers VPL vectors of the
// chunk (columns c + q*LPR, q < VPL, in vector units) so that the index traffic, the address
// arithmetic and the shuffles are paid once per VPL * 16 gathered bytes.
// The thread's second-level sums live in shared memory as tot_s[k][thread]; with a multiple of four sums
// they are moved four at a time (tot_s is then indexed as float4 rows of the same array).
template <int NV, bool ZERO_ACC>
__device__ __forceinline__ void second_level(float (*tot_s)[kBlock], int tid, float* acc, int mode /*0 clear, 1 add acc, 2 fetch*/)
{
    if constexpr (NV % 4 == 0) {
        float4* t4 = reinterpret_cast<float4*>(&tot_s[0][0]) + tid;          // element k4 of the thread: t4[k4 * kBlock]
#pragma unroll
        for (int k4 = 0; k4 < NV / 4; ++k4) {
            float4& slot = t4[k4 * kBlock];
            if (mode == 0) {
                slot = make_float4(0.f, 0.f, 0.f, 0.f);
            } else if (mode == 1) {
                float4 v = slot;
                v.x += acc[4 * k4]; v.y += acc[4 * k4 + 1]; v.z += acc[4 * k4 + 2]; v.w += acc[4 * k4 + 3];
                slot = v;
                if (ZERO_ACC) acc[4 * k4] = acc[4 * k4 + 1] = acc[4 * k4 + 2] = acc[4 * k4 + 3] = 0.f;
            } else {
                const float4 v = slot;
                acc[4 * k4] += v.x; acc[4 * k4 + 1] += v.y; acc[4 * k4 + 2] += v.z; acc[4 * k4 + 3] += v.w;
            }
        }
    } else {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            if (mode == 0) tot_s[k][tid] = 0.f;
            else if (mode == 1) { tot_s[k][tid] += acc[k]; if (ZERO_ACC) acc[k] = 0.f; }
            else acc[k] += tot_s[k][tid];
        }
    }
}

template <typename T, int VECN, int LPR, int VPL, bool WEIGHTED, bool WIDE, int EP>
__device__ __forceinline__ void gather_rows(const GatherArgs& a, const Range& rg, int block_in_range, int col0,
                                            int chunk_end, int32_t (*stage_col)[kBlock / 32][kStageSlots],
                                            float (*stage_w)[kBlock / 32][kStageSlots], float (*tot_s)[kBlock])
{
    constexpr int S = LPR * EP;
    constexpr int ROWS = kBlock / S;
    constexpr int UB = kLoads / VPL;                      // steps whose loads are issued together
    constexpr int R = UB > LPR ? UB / LPR : 1;            // index registers per lane and batch
    constexpr int SPB = R * LPR;                          // steps per batch
    constexpr int EPB = R * S;                            // entries per batch
    constexpr unsigned kFull = 0xffffffffu;
    const int tid = threadIdx.x;
    const int group = tid / S;
    const int sl = tid % S;
    const int g = sl / LPR;
    const int c = sl % LPR;
    const int warp = tid >> 5, lane = tid & 31;
    const int seg = lane - sl;                   // first lane of this row's segment inside the warp

    int jq[VPL];
    bool okq[VPL];
    const T* xq[VPL];
#pragma unroll
    for (int q = 0; q < VPL; ++q) {
        // with 32-byte loads a lane's two vectors are neighbours, otherwise they lie LPR vectors apart
        jq[q] = col0 + (WIDE ? c * VPL + q : c + q * LPR) * VECN;
        okq[q] = jq[q] < chunk_end;
        xq[q] = static_cast<const T*>(a.x) + (okq[q] ? jq[q] : col0);   // out-of-chunk lanes re-read a valid column
    }
    const bool wide = WIDE && okq[VPL - 1];            // both vectors of the lane exist: one 32-byte load per entry
    const uint32_t ld = (uint32_t)a.ldx;

    const int slot = block_in_range * ROWS + group;
    const bool active = slot < rg.item_count;
    int32_t row = 0, b = 0, e = 0, part = 0;      // part: where a hub segment's partial sums go
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
    int32_t ucur[R];
    float wcur[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int32_t kk = b + r * S + sl;
        const bool ok = kk < e;
        ucur[r] = ok ? __ldcs(a.col_idx + kk) : -1;
        wcur[r] = (WEIGHTED && ok) ? __ldcs(a.edge_w + kk) : 0.f;
    }

    // Two levels of accumulation: `acc` takes at most kChain products in a row, then moves into the
    // thread's second-level sums (kept in shared memory, they cost no registers), so that no fp32 chain
    // of a lane is longer than kChain + (entries of the lane) / kChain terms.  Long runs of equal-sign
    // terms (a hub row fed by one source many times) otherwise drift by half an ulp per term.
    constexpr int kChain = 64;
    constexpr int FLUSH = SPB >= kChain ? 1 : kChain / SPB;      // batches between two moves
    float acc[VPL][VECN];
#pragma unroll
    for (int q = 0; q < VPL; ++q)
#pragma unroll
        for (int i = 0; i < VECN; ++i) acc[q][i] = 0.f;

    const int n_batches = __reduce_max_sync(kFull, (e - b + EPB - 1) / EPB);     // the warp loops together
    const bool two_level = n_batches > FLUSH;                                    // short rows never leave the first level
    if (two_level) second_level<VPL * VECN, true>(tot_s, tid, &acc[0][0], 0);

    for (int ib = 0; ib < n_batches; ++ib) {
        const int32_t kb = b + ib * EPB;
        // the next batch's indices are requested before this batch's gathers are consumed
        int32_t unext[R];
        float wnext[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int32_t kk = kb + EPB + r * S + sl;
            const bool ok = kk < e;
            unext[r] = ok ? __ldcs(a.col_idx + kk) : -1;
            wnext[r] = (WEIGHTED && ok) ? __ldcs(a.edge_w + kk) : 0.f;
        }
        const bool full = __all_sync(kFull, kb + EPB <= e);
        const int buf = ib & 1;
        if (LPR > 1) {      // with one lane per row every lane consumes exactly the entries it fetched
#pragma unroll
            for (int r = 0; r < R; ++r) {
                stage_col[buf][warp][r * 32 + lane] = ucur[r];
                if (WEIGHTED) stage_w[buf][warp][r * 32 + lane] = wcur[r];
            }
            __syncwarp();
        }
        auto consume = [&](const Vec<T, VECN> (&v)[UB][VPL], const float (&wv)[UB]) {
#pragma unroll
            for (int i = 0; i < UB; ++i)
#pragma unroll
                for (int q = 0; q < VPL; ++q)
#pragma unroll
                    for (int k = 0; k < VECN; ++k) {
                        if (WEIGHTED) acc[q][k] = fmaf(wv[i], v[i][q].get(k), acc[q][k]);
                        else acc[q][k] += v[i][q].get(k);
                    }
        };
        if (full) {
            // every lane has all of the batch's entries: straight-line code, no tests
#pragma unroll
            for (int s0 = 0; s0 < SPB; s0 += UB) {
                Vec<T, VECN> v[UB][VPL];
                float wv[UB];
#pragma unroll
                for (int i = 0; i < UB; ++i) {
                    const int r = (s0 + i) / LPR, tt = (s0 + i) % LPR;
                    const int32_t u = LPR > 1 ? stage_col[buf][warp][r * 32 + seg + tt * EP + g] : ucur[r];
                    if (WEIGHTED) wv[i] = LPR > 1 ? stage_w[buf][warp][r * 32 + seg + tt * EP + g] : wcur[r];
                    const size_t off = (size_t)(uint32_t)u * ld;
                    if (WIDE && wide) {
                        load_pair(v[i][0], v[i][VPL - 1], xq[0] + off);
                    } else {
#pragma unroll
                        for (int q = 0; q < VPL; ++q) v[i][q].load(xq[q] + off);
                    }
                }
                consume(v, wv);
            }
        } else {
            // A ragged batch.  Step s works on entries s * EP .. of a row's batch, so the steps past the longest
            // remainder in the warp have nothing to do for any lane (a row of 3 entries in a class whose batch
            // holds 16 would otherwise pay for 16).
            const int rem = __reduce_max_sync(kFull, e - kb);
#pragma unroll
            for (int s0 = 0; s0 < SPB; s0 += UB) {
                if (s0 > 0 && s0 * EP >= rem) break;
                Vec<T, VECN> v[UB][VPL];
                float wv[UB];
#pragma unroll
                for (int i = 0; i < UB; ++i) {
                    const int r = (s0 + i) / LPR, tt = (s0 + i) % LPR;
                    const int32_t u = LPR > 1 ? stage_col[buf][warp][r * 32 + seg + tt * EP + g] : ucur[r];
                    if (WEIGHTED) wv[i] = LPR > 1 ? stage_w[buf][warp][r * 32 + seg + tt * EP + g] : wcur[r];
                    const size_t off = (size_t)(uint32_t)max(u, 0) * ld;
                    if (WIDE && wide) {
                        if (u >= 0) load_pair(v[i][0], v[i][VPL - 1], xq[0] + off);
                        else { v[i][0].zero(); v[i][VPL - 1].zero(); }
                    } else {
#pragma unroll
                        for (int q = 0; q < VPL; ++q) {
                            if (u >= 0) v[i][q].load(xq[q] + off);
                            else v[i][q].zero();
                        }
                    }
                }
                consume(v, wv);
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) { ucur[r] = unext[r]; wcur[r] = wnext[r]; }
        if (two_level && (ib + 1) % FLUSH == 0) second_level<VPL * VECN, true>(tot_s, tid, &acc[0][0], 1);
    }
    if (two_level) second_level<VPL * VECN, true>(tot_s, tid, &acc[0][0], 2);

    // fixed-order combination of the EP partial sums of the row
#pragma unroll
    for (int o = S / 2; o >= LPR; o >>= 1)
#pragma unroll
        for (int q = 0; q < VPL; ++q)
#pragma unroll
            for (int i = 0; i < VECN; ++i) acc[q][i] += __shfl_down_sync(kFull, acc[q][i], o, S);

    if (active && g == 0) {
        const float scale = (WEIGHTED || rg.hub) ? 1.f : a.rdeg[row];
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            if (!okq[q]) continue;
            const int j = jq[q];
            if (rg.hub) {
                float* p = a.partial + (int64_t)part * a.fpad + j;
#pragma unroll
                for (int i = 0; i < VECN; ++i)
                    if (j + i < chunk_end) p[i] = acc[q][i];
                continue;
            }
            const int64_t o = (int64_t)row * a.ldo + j;
            if (VECN % 4 == 0 && a.out_vec_ok && j + VECN <= chunk_end) {
#pragma unroll
                for (int i = 0; i < VECN; i += 4)
                    __stcs(reinterpret_cast<float4*>(static_cast<float*>(a.out) + o + i),
                           make_float4(acc[q][i] * scale, acc[q][i + 1] * scale, acc[q][i + 2] * scale, acc[q][i + 3] * scale));
            } else {
#pragma unroll
                for (int i = 0; i < VECN; ++i)
                    if (j + i < chunk_end) store_elem(a.out, a.out_bf16, o + i, acc[q][i] * scale);
            }
        }
    }
}

template <typename T, int VECN, int LPR, int VPL, bool WEIGHTED, bool WIDE = false>
__global__ void __launch_bounds__(kBlock, GNNFD_GATHER_MIN_BLOCKS) gather_aggregate(const __grid_constant__ GatherArgs a)
{
    __shared__ int32_t stage_col[2][kBlock / 32][kStageSlots];
    __shared__ float stage_w[2][kBlock / 32][kStageSlots];
    __shared__ __align__(16) float tot_s[VPL * VECN][kBlock];   // second-level sums of every thread
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
        case 0: gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 1>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
        case 1: if constexpr (LPR * 2 <= 32) gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 2>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
        case 2: if constexpr (LPR * 4 <= 32) gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 4>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
        case 3: if constexpr (LPR * 8 <= 32) gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 8>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
        case 4: if constexpr (LPR * 16 <= 32) gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 16>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
        default: if constexpr (LPR == 1) gather_rows<T, VECN, LPR, VPL, WEIGHTED, WIDE, 32>(a, rg, bir, col0, chunk_end, stage_col, stage_w, tot_s); break;
    }
}

// out[row, j] = scale * sum over the row's segments, ascending, of partial[segment, j]
__global__ void __launch_bounds__(kBlock)
hub_reduce(const int32_t* __restrict__ row_order, const int32_t* __restrict__ hub_seg_ptr, const float* __restrict__ rdeg,
           const float* __restrict__ partial, int64_t hub_begin, int32_t n_hub, int32_t f, int32_t fpad, int use_rdeg,
           void* __restrict__ out, int64_t ldo, int out_bf16)
{
    const int i = blockIdx.x;
    const int j = blockIdx.y * kBlock + threadIdx.x;
    if (i >= n_hub || j >= f) return;
    const int32_t row = row_order[hub_begin + i];
    const int32_t s0 = hub_seg_ptr[i], s1 = hub_seg_ptr[i + 1];
    // segment sums in ascending order, in runs of 32 so that a row of very many segments keeps short chains
    float acc = 0.f, run = 0.f;
    for (int32_t s = s0; s < s1; ++s) {
        run += partial[(int64_t)s * fpad + j];
        if (((s - s0) & 31) == 31) { acc += run; run = 0.f; }
    }
    acc += run;
    if (use_rdeg) acc *= rdeg[row];
    store_elem(out, out_bf16, (int64_t)row * ldo + j, acc);
}

// ------------------------------------------------------------------ host side

typedef void (*GatherKernel)(const GatherArgs);

template <typename T, int VECN, bool WEIGHTED>
static GatherKernel pick_lpr(int lpr, int vpl, bool wide)
{
    if (vpl == 1) return gather_aggregate<T, VECN, 1, 1, WEIGHTED>;
    if constexpr (VECN * sizeof(T) == 16) {
        if (wide) {          // narrow chunks whose vector pairs start on 32-byte boundaries
            switch (lpr) {
                case 1: return gather_aggregate<T, VECN, 1, 2, WEIGHTED, true>;
                case 2: return gather_aggregate<T, VECN, 2, 2, WEIGHTED, true>;
                default: return gather_aggregate<T, VECN, 4, 2, WEIGHTED, true>;
            }
        }
    }
    switch (lpr) {
        case 1: return gather_aggregate<T, VECN, 1, 2, WEIGHTED>;
        case 2: return gather_aggregate<T, VECN, 2, 2, WEIGHTED>;
        case 4: return gather_aggregate<T, VECN, 4, 2, WEIGHTED>;
        case 8: return gather_aggregate<T, VECN, 8, 2, WEIGHTED>;
        case 16: return gather_aggregate<T, VECN, 16, 2, WEIGHTED>;
        default: return gather_aggregate<T, VECN, 32, 2, WEIGHTED>;
    }
}

template <bool WEIGHTED>
static GatherKernel pick_kernel(gnnfd_dtype_t xdt, bool vec, int lpr, int vpl, bool wide)
{
    if (xdt == GNNFD_F32)
        return vec ? pick_lpr<float, 4, WEIGHTED>(lpr, vpl, wide) : pick_lpr<float, 1, WEIGHTED>(lpr, vpl, false);
    return vec ? pick_lpr<__nv_bfloat16, 8, WEIGHTED>(lpr, vpl, wide) : pick_lpr<__nv_bfloat16, 1, WEIGHTED>(lpr, vpl, false);
}

static size_t partial_bytes(const gnnfd_csr_t* csr, int32_t f)
{
    const size_t fpad = align_up((size_t)f, 4);
    return align_up((size_t)csr->n_segments * fpad * sizeof(float), 256);
}

static int aggregate(bool weighted, const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out,
                     int64_t ldo, gnnfd_dtype_t odt, int32_t f, int32_t chunk_width, void* d_scratch,
                     size_t scratch_bytes, cudaStream_t s)
{
    if (!csr || !d_x || !d_out || f <= 0 || chunk_width <= 0 || ldx < f || ldo < f || ldx > 0x7fffffffll)
        return GNNFD_INVALID_ARG;
    if ((xdt != GNNFD_F32 && xdt != GNNFD_BF16) || (odt != GNNFD_F32 && odt != GNNFD_BF16)) return GNNFD_UNSUPPORTED;
    const size_t need = partial_bytes(csr, f);
    if (need > 0 && (!d_scratch || scratch_bytes < need)) return GNNFD_WORKSPACE_TOO_SMALL;
    if (need > 0 && ((uintptr_t)d_scratch & 15u)) return GNNFD_INVALID_ARG;

    const int cw = chunk_width < f ? chunk_width : f;
    const int n_chunks = (f + cw - 1) / cw;
    const int xsize = xdt == GNNFD_F32 ? 4 : 2;
    const int vecn = 16 / xsize;
    // 128-bit loads need 16-byte aligned row starts and chunk starts
    const bool vec = ((uintptr_t)d_x % 16 == 0) && ((ldx * xsize) % 16 == 0) && (n_chunks == 1 || cw % vecn == 0);
    const int elems = vec ? vecn : 1;
    // a lane covers two vectors of the chunk unless the chunk is a single vector wide
    const int vectors = (cw + elems - 1) / elems;
    const int vpl = vectors > 1 ? 2 : 1;
    int lpr = 1;
    while (lpr * vpl < vectors && lpr < 32) lpr <<= 1;

    GatherArgs a;
    a.row_ptr = csr->row_ptr; a.col_idx = csr->col_idx; a.edge_w = csr->edge_w; a.rdeg = csr->rdeg;
    a.row_order = csr->row_order; a.seg_row = csr->seg_row; a.seg_begin = csr->seg_begin;
    a.seg_end = csr->seg_end; a.seg_slot = csr->seg_slot;
    a.x = d_x; a.out = d_out; a.partial = static_cast<float*>(d_scratch);
    a.ldx = ldx; a.ldo = ldo; a.f = f; a.chunk_width = cw;
    a.n_ctiles = (cw + lpr * vpl * elems - 1) / (lpr * vpl * elems);
    a.fpad = (int32_t)align_up((size_t)f, 4);
    a.out_bf16 = odt == GNNFD_BF16;
    // 32-byte loads of a lane's vector pair: every pair must start on a 32-byte boundary, and the chunk must
    // be narrow (up to 128 bytes, four lanes per row).  There the pair load halves the cache lines an
    // instruction touches (hidden width 8 / 16 / 32 on the config-4 graph: 0.84 / 1.04 / 1.28 -> 0.61 / 0.77 /
    // 0.99 ms); with eight or more lanes per row the strided single vectors already cover whole lines and
    // the pair form is slower (config 4 at 64 columns 16.2 -> 18.4 ms).
    a.wide_ok = vec && vpl == 2 && lpr <= 4 && ((uintptr_t)d_x % 32 == 0) && ((ldx * xsize) % 32 == 0) &&
                (n_chunks == 1 || (cw * xsize) % 32 == 0);
    a.out_vec_ok = odt == GNNFD_F32 && ((uintptr_t)d_out % 16 == 0) && (ldo % 4 == 0) && (n_chunks == 1 || cw % 4 == 0);

    const int64_t blocks = plan_ranges(csr, lpr, a.range, &a.n_ranges);
    a.blocks_per_tile = (int32_t)blocks;
    const int64_t grid_x = blocks * a.n_ctiles;
    if (grid_x > 0x7fffffffll) return GNNFD_TOO_LARGE;

    if (grid_x > 0) {
        GatherKernel kernel = weighted ? pick_kernel<true>(xdt, vec, lpr, vpl, a.wide_ok != 0) : pick_kernel<false>(xdt, vec, lpr, vpl, a.wide_ok != 0);
        for (int c0 = 0; c0 < n_chunks; c0 += kMaxGridY) {
            a.chunk_base = c0;
            const dim3 grid((unsigned)grid_x, (unsigned)(n_chunks - c0 < kMaxGridY ? n_chunks - c0 : kMaxGridY));
            GNNFD_LAUNCH(weighted ? "gather_aggregate_gcn" : "gather_aggregate_sage", s, kernel, grid, kBlock, 0, a);
        }
    }
    const int64_t n_hub = csr->bin_count[4];
    if (n_hub > 0) {
        dim3 g((unsigned)n_hub, (unsigned)((f + kBlock - 1) / kBlock));
        GNNFD_LAUNCH("hub_reduce", s, hub_reduce, g, kBlock, 0, csr->row_order, csr->hub_seg_ptr, csr->rdeg, a.partial,
                     csr->bin_start[4], (int32_t)n_hub, f, a.fpad, weighted ? 0 : 1, d_out, ldo, a.out_bf16);
    }
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" {

int gnnfd_aggregate_workspace_bytes(const gnnfd_csr_t* csr, int32_t f, size_t* scratch_bytes)
{
    if (!csr || f <= 0 || !scratch_bytes) return GNNFD_INVALID_ARG;
    *scratch_bytes = gnnfd::partial_bytes(csr, f);
    return GNNFD_OK;
}

int gnnfd_aggregate_gcn(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo,
                        gnnfd_dtype_t odt, int32_t f, int32_t chunk_width, void* d_scratch, size_t scratch_bytes,
                        void* stream)
{
    return gnnfd::aggregate(true, csr, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, d_scratch, scratch_bytes,
                            static_cast<cudaStream_t>(stream));
}

int gnnfd_aggregate_sage(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo,
                         gnnfd_dtype_t odt, int32_t f, int32_t chunk_width, void* d_scratch, size_t scratch_bytes,
                         void* stream)
{
    return gnnfd::aggregate(false, csr, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, d_scratch, scratch_bytes,
                            static_cast<cudaStream_t>(stream));
}

}  // extern "C"
