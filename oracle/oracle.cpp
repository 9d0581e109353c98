// CPU oracle for feature-decomposed GNN aggregation.
//
// TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 restatement of what the
// aggregation phase computes (Algorithm 1, the Message / Aggregate / Concat
// steps inside the loop over decomposition layers p), used to check the CUDA
// library and as the timed CPU baseline.  It shares no code with the CUDA
// path and nothing in the product may call it.
//
// The paper names its three aggregators (GCN, GraphSAGE, GAT; Section II-A,
// Section III) by citation only, so the formulas are the cited models'
// standard ones, as PyG (the paper's framework, Section II-C) evaluates them
// on a destination-indexed edge list:
//   GCN   out[v] = sum_{u->v} deg(u)^-1/2 deg(v)^-1/2 x[u]
//   SAGE  out[v] = (1/deg(v)) sum_{u->v} x[u]
//   GAT   out[v,h] = sum_{u->v} softmax_u(LeakyReLU(a_src[h].z[u,h] + a_dst[h].z[v,h])) z[u,h]
// with deg = number of CSR entries in the row (in-degree, multi-edges counted)
// and deg^-1/2, 1/deg := 0 for empty rows.
//
// Parity pins: every function here is pinned by tests that do not go through
// it (dense adjacency products, closed forms on star / regular graphs, the
// hand-computed Fig. 2 example, invariants); none is "parity unpinned".
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum : uint32_t { ADD_SELF_LOOPS = 1, DEDUP = 2, SYMMETRIZE = 4 };
enum : int { ERR_INVALID = -1, ERR_BAD_INDEX = -2, ERR_TOO_LARGE = -3 };
enum : int { DT_F32 = 0, DT_BF16 = 1 };

struct Edge { int64_t dst, src, id; };

inline double load_x(const void* x, int dt, int64_t i)
{
    if (dt == DT_F32) return (double)static_cast<const float*>(x)[i];
    uint32_t bits = (uint32_t)static_cast<const uint16_t*>(x)[i] << 16;  // bf16 widens exactly
    float f; std::memcpy(&f, &bits, 4);
    return (double)f;
}

inline int64_t load_id(const void* p, int itype, int64_t i)
{
    return itype == 0 ? (int64_t)static_cast<const int32_t*>(p)[i] : static_cast<const int64_t*>(p)[i];
}

}  // namespace

extern "C" {

// CSR by destination from a COO edge list (Section II-C: the input is the edge
// set in COO form).  Steps, in order: reject ids outside [0,n); SYMMETRIZE
// appends the reverse of every non-loop edge with id e+i; ADD_SELF_LOOPS drops
// every loop and appends one (v,v) per vertex with id -1; order by (dst, src),
// ties by id; DEDUP keeps the first of each run of equal (dst, src).
// row_ptr has n+1 entries; col_idx / perm must hold orc_csr_capacity entries.
// Returns nnz or a negative error.
int64_t orc_csr_capacity(int64_t n, int64_t e, uint32_t flags)
{
    int64_t m = e;
    if (flags & SYMMETRIZE) m += e;
    if (flags & ADD_SELF_LOOPS) m += n;
    return m;
}

int64_t orc_build_csr(int64_t n, int64_t e, const void* src, const void* dst, int itype, uint32_t flags,
                      int32_t* row_ptr, int32_t* col_idx, int32_t* perm)
{
    if (n <= 0 || e < 0) return ERR_INVALID;
    std::vector<Edge> edges;
    edges.reserve((size_t)orc_csr_capacity(n, e, flags));
    for (int64_t i = 0; i < e; ++i) {
        int64_t s = load_id(src, itype, i), d = load_id(dst, itype, i);
        if (s < 0 || s >= n || d < 0 || d >= n) return ERR_BAD_INDEX;
        edges.push_back({d, s, i});
    }
    if (flags & SYMMETRIZE)
        for (int64_t i = 0; i < e; ++i)
            if (edges[i].src != edges[i].dst) edges.push_back({edges[i].src, edges[i].dst, e + i});
    if (flags & ADD_SELF_LOOPS) {
        edges.erase(std::remove_if(edges.begin(), edges.end(), [](const Edge& x) { return x.src == x.dst; }),
                    edges.end());
        for (int64_t v = 0; v < n; ++v) edges.push_back({v, v, -1});
    }
    std::stable_sort(edges.begin(), edges.end(), [](const Edge& a, const Edge& b) {
        if (a.dst != b.dst) return a.dst < b.dst;
        if (a.src != b.src) return a.src < b.src;
        return a.id < b.id;
    });
    if (flags & DEDUP)
        edges.erase(std::unique(edges.begin(), edges.end(),
                                [](const Edge& a, const Edge& b) { return a.dst == b.dst && a.src == b.src; }),
                    edges.end());
    const int64_t nnz = (int64_t)edges.size();
    if (nnz >= (int64_t(1) << 31)) return ERR_TOO_LARGE;
    for (int64_t v = 0; v <= n; ++v) row_ptr[v] = 0;
    for (int64_t k = 0; k < nnz; ++k) row_ptr[edges[k].dst + 1] += 1;
    for (int64_t v = 0; v < n; ++v) row_ptr[v + 1] += row_ptr[v];
    for (int64_t k = 0; k < nnz; ++k) {
        col_idx[k] = (int32_t)edges[k].src;
        perm[k] = (int32_t)edges[k].id;
    }
    return nnz;
}

// deg(v) = entries in row v; dinv = deg^-1/2, rdeg = 1/deg, both 0 for empty rows.
void orc_degree_norm(int64_t n, const int32_t* row_ptr, int32_t* deg, double* dinv, double* rdeg)
{
    for (int64_t v = 0; v < n; ++v) {
        int32_t d = row_ptr[v + 1] - row_ptr[v];
        deg[v] = d;
        dinv[v] = d > 0 ? 1.0 / std::sqrt((double)d) : 0.0;
        rdeg[v] = d > 0 ? 1.0 / (double)d : 0.0;
    }
}

// GCN (model 0) and SAGE mean (model 1) aggregation, Algorithm 1's loop over
// decomposition layers p written out: the feature columns are cut into chunks
// of chunk_width (the last one narrower, as torch.chunk does), each chunk is
// aggregated over all vertices, and chunk p's result lands in its own columns
// of out (the Concat step).  rows == nullptr: all vertices, out is [n, f];
// otherwise only the n_rows listed vertices, out is [n_rows, f].
// abs_out (optional) receives sum |w * x| per element, the tolerance scale.
int orc_aggregate(int model, int64_t n, const int32_t* row_ptr, const int32_t* col_idx,
                  const void* x, int64_t ldx, int xdt, int32_t f, int32_t chunk_width,
                  const int64_t* rows, int64_t n_rows, double* out, double* abs_out, int threads)
{
    if (n <= 0 || f <= 0 || chunk_width <= 0 || ldx < f || (model != 0 && model != 1)) return ERR_INVALID;
    std::vector<double> dinv(n);
    for (int64_t v = 0; v < n; ++v) {
        int32_t d = row_ptr[v + 1] - row_ptr[v];
        dinv[v] = d > 0 ? 1.0 / std::sqrt((double)d) : 0.0;
    }
    const int64_t count = rows ? n_rows : n;
    const int32_t n_chunks = (f + chunk_width - 1) / chunk_width;
    (void)threads;
    for (int32_t p = 0; p < n_chunks; ++p) {
        const int32_t j0 = p * chunk_width, j1 = std::min(f, j0 + chunk_width);
#pragma omp parallel for schedule(dynamic, 64) num_threads(threads > 1 ? threads : 1) if (threads > 1)
        for (int64_t r = 0; r < count; ++r) {
            const int64_t v = rows ? rows[r] : r;
            const int32_t b = row_ptr[v], e = row_ptr[v + 1];
            const double rdeg = e > b ? 1.0 / (double)(e - b) : 0.0;
            for (int32_t j = j0; j < j1; ++j) {
                double acc = 0.0, aabs = 0.0;
                for (int32_t k = b; k < e; ++k) {
                    const int64_t u = col_idx[k];
                    const double w = model == 0 ? dinv[u] * dinv[v] : rdeg;
                    const double m = w * load_x(x, xdt, u * ldx + j);   // Message
                    acc += m;                                           // Aggregate
                    aabs += std::fabs(m);
                }
                out[r * f + j] = acc;
                if (abs_out) abs_out[r * f + j] = aabs;
            }
        }
    }
    return 0;
}

// GAT attention scores: s_src[u,h] = sum_d a_src[h,d] z[u,h,d], likewise s_dst.
int orc_gat_scores(int64_t n, const void* z, int64_t ldz, int zdt, const float* a_src, const float* a_dst,
                   int32_t heads, int32_t dim, double* s_src, double* s_dst)
{
    if (n <= 0 || heads <= 0 || dim <= 0 || ldz < (int64_t)heads * dim) return ERR_INVALID;
    for (int64_t v = 0; v < n; ++v)
        for (int32_t h = 0; h < heads; ++h) {
            double ss = 0.0, sd = 0.0;
            for (int32_t d = 0; d < dim; ++d) {
                const double zv = load_x(z, zdt, v * ldz + h * dim + d);
                ss += (double)a_src[h * dim + d] * zv;
                sd += (double)a_dst[h * dim + d] * zv;
            }
            s_src[v * heads + h] = ss;
            s_dst[v * heads + h] = sd;
        }
    return 0;
}

// Edge softmax: alpha[k,h] over the entries k of each CSR row, logits
// LeakyReLU(s_src[col[k],h] + s_dst[v,h]); alpha is [nnz, heads] in CSR order.
int orc_edge_softmax(int64_t n, const int32_t* row_ptr, const int32_t* col_idx, const double* s_src,
                     const double* s_dst, int32_t heads, double slope, double* alpha)
{
    if (n <= 0 || heads <= 0) return ERR_INVALID;
    for (int64_t v = 0; v < n; ++v) {
        const int32_t b = row_ptr[v], e = row_ptr[v + 1];
        for (int32_t h = 0; h < heads; ++h) {
            double mx = -INFINITY;
            for (int32_t k = b; k < e; ++k) {
                double t = s_src[(int64_t)col_idx[k] * heads + h] + s_dst[v * heads + h];
                t = t >= 0.0 ? t : slope * t;
                alpha[(int64_t)k * heads + h] = t;
                mx = std::max(mx, t);
            }
            double sum = 0.0;
            for (int32_t k = b; k < e; ++k) {
                double p = std::exp(alpha[(int64_t)k * heads + h] - mx);
                alpha[(int64_t)k * heads + h] = p;
                sum += p;
            }
            for (int32_t k = b; k < e; ++k) alpha[(int64_t)k * heads + h] /= sum;
        }
    }
    return 0;
}

// Same as orc_edge_softmax with fp32 scores as the caller of the library's
// edge-softmax entry point supplies them (widened exactly).
int orc_edge_softmax_f32(int64_t n, const int32_t* row_ptr, const int32_t* col_idx, const float* s_src,
                         const float* s_dst, int32_t heads, double slope, double* alpha)
{
    std::vector<double> a((size_t)n * heads), b((size_t)n * heads);
    for (size_t i = 0; i < a.size(); ++i) { a[i] = s_src[i]; b[i] = s_dst[i]; }
    return orc_edge_softmax(n, row_ptr, col_idx, a.data(), b.data(), heads, slope, alpha);
}

// GAT aggregation with feature decomposition.  The attention logits use the
// full head width (scores are computed once from all of z); only the weighted
// sum runs chunk by chunk over the flattened heads*dim columns, column j
// belonging to head j / dim.  rows / abs_out as in orc_aggregate.
int orc_aggregate_gat(int64_t n, const int32_t* row_ptr, const int32_t* col_idx, const void* z, int64_t ldz,
                      int zdt, const float* a_src, const float* a_dst, int32_t heads, int32_t dim,
                      double slope, int32_t chunk_width, const int64_t* rows, int64_t n_rows,
                      double* out, double* abs_out, int threads)
{
    const int32_t f = heads * dim;
    if (n <= 0 || heads <= 0 || dim <= 0 || chunk_width <= 0 || ldz < f) return ERR_INVALID;
    std::vector<double> s_src((size_t)n * heads), s_dst((size_t)n * heads);
    orc_gat_scores(n, z, ldz, zdt, a_src, a_dst, heads, dim, s_src.data(), s_dst.data());
    const int64_t count = rows ? n_rows : n;
    const int32_t n_chunks = (f + chunk_width - 1) / chunk_width;
    (void)threads;
    for (int32_t p = 0; p < n_chunks; ++p) {
        const int32_t j0 = p * chunk_width, j1 = std::min(f, j0 + chunk_width);
#pragma omp parallel for schedule(dynamic, 64) num_threads(threads > 1 ? threads : 1) if (threads > 1)
        for (int64_t r = 0; r < count; ++r) {
            const int64_t v = rows ? rows[r] : r;
            const int32_t b = row_ptr[v], e = row_ptr[v + 1];
            std::vector<double> a((size_t)(e - b));
            int32_t a_head = -1;
            for (int32_t j = j0; j < j1; ++j) {
                const int32_t h = j / dim;
                if (h != a_head) {   // softmax over the row for head h
                    double mx = -INFINITY, sum = 0.0;
                    for (int32_t k = b; k < e; ++k) {
                        double t = s_src[(int64_t)col_idx[k] * heads + h] + s_dst[v * heads + h];
                        a[k - b] = t >= 0.0 ? t : slope * t;
                        mx = std::max(mx, a[k - b]);
                    }
                    for (int32_t k = b; k < e; ++k) { a[k - b] = std::exp(a[k - b] - mx); sum += a[k - b]; }
                    for (int32_t k = b; k < e; ++k) a[k - b] /= sum;
                    a_head = h;
                }
                double acc = 0.0, aabs = 0.0;
                for (int32_t k = b; k < e; ++k) {
                    const double m = a[k - b] * load_x(z, zdt, (int64_t)col_idx[k] * ldz + j);
                    acc += m;
                    aabs += std::fabs(m);
                }
                out[r * f + j] = acc;
                if (abs_out) abs_out[r * f + j] = aabs;
            }
        }
    }
    return 0;
}

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
