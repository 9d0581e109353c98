// One-shot aggregation of a COO edge list: for a graph that is aggregated once, at a narrow width, the full
// conversion costs several times the aggregation it serves (the paper's point about format-conversion latency,
// Section III).  This path does the light build (destination-only sort, rows in edge-id order) and the
// aggregation in one call out of one caller buffer, and keeps no handle.
#include "common.cuh"

namespace gnnfd {

struct OneshotLayout {
    size_t persistent, build_scratch, aggregate;
};

static uint32_t oneshot_flags(uint32_t flags)
{
    // duplicate removal needs the fully ordered build; everything else takes the light one
    return (flags & GNNFD_CSR_DEDUP) ? flags : (flags | GNNFD_CSR_INPUT_ORDER);
}

// heads > 0: the GAT aggregation's workspace (two [n, heads] score arrays, per-segment sums, maxima and denominators)
static int oneshot_layout(int64_t n, int64_t e, uint32_t flags, int32_t f, int32_t heads, OneshotLayout* L)
{
    if (f <= 0 || heads < 0) return GNNFD_INVALID_ARG;
    int rc = gnnfd_csr_workspace_bytes(n, e, oneshot_flags(flags), &L->persistent, &L->build_scratch);
    if (rc) return rc;
    const int64_t segs = segment_capacity(n, e, oneshot_flags(flags));
    if (segs < 0) return GNNFD_INVALID_ARG;
    L->aggregate = align_up((size_t)segs * align_up((size_t)f, 4) * sizeof(float), 256);
    if (heads > 0)
        L->aggregate += 2 * align_up((size_t)n * heads * sizeof(float), 256) +
                        align_up((size_t)segs * heads * 2 * sizeof(float), 256);
    return GNNFD_OK;
}

static int oneshot(bool weighted, int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype,
                   uint32_t flags, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                   int32_t f, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream)
{
    if (!d_scratch || ((uintptr_t)d_scratch & 255u)) return GNNFD_INVALID_ARG;
    OneshotLayout L;
    int rc = oneshot_layout(n, e, flags, f, 0, &L);
    if (rc) return rc;
    if (scratch_bytes < L.persistent + L.build_scratch + L.aggregate) return GNNFD_WORKSPACE_TOO_SMALL;
    char* base = static_cast<char*>(d_scratch);
    gnnfd_csr_t* csr = nullptr;
    rc = gnnfd_build_csr(n, e, d_src, d_dst, itype, oneshot_flags(flags), base, L.persistent, base + L.persistent,
                         L.build_scratch, stream, &csr);
    if (rc) return rc;
    void* agg = base + L.persistent + L.build_scratch;
    rc = weighted ? gnnfd_aggregate_gcn(csr, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, agg, L.aggregate, stream)
                  : gnnfd_aggregate_sage(csr, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, agg, L.aggregate, stream);
    gnnfd_csr_destroy(csr);       // the enqueued kernels hold device pointers only
    return rc;
}

}  // namespace gnnfd

extern "C" {

int gnnfd_oneshot_workspace_bytes(int64_t n, int64_t e, uint32_t flags, int32_t f, size_t* scratch_bytes)
{
    if (!scratch_bytes) return GNNFD_INVALID_ARG;
    gnnfd::OneshotLayout L;
    int rc = gnnfd::oneshot_layout(n, e, flags, f, 0, &L);
    if (rc) return rc;
    *scratch_bytes = L.persistent + L.build_scratch + L.aggregate;
    return GNNFD_OK;
}

int gnnfd_oneshot_gat_workspace_bytes(int64_t n, int64_t e, uint32_t flags, int32_t heads, int32_t dim, size_t* scratch_bytes)
{
    if (!scratch_bytes || heads <= 0 || dim <= 0 || (int64_t)heads * dim > 0x7fffffffll) return GNNFD_INVALID_ARG;
    gnnfd::OneshotLayout L;
    int rc = gnnfd::oneshot_layout(n, e, flags, heads * dim, heads, &L);
    if (rc) return rc;
    *scratch_bytes = L.persistent + L.build_scratch + L.aggregate;
    return GNNFD_OK;
}

int gnnfd_oneshot_gat(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                      const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src, const float* d_a_dst, int32_t heads,
                      int32_t dim, float negative_slope, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t chunk_width,
                      void* d_scratch, size_t scratch_bytes, void* stream)
{
    using namespace gnnfd;
    if (!d_scratch || ((uintptr_t)d_scratch & 255u) || heads <= 0 || dim <= 0 || (int64_t)heads * dim > 0x7fffffffll)
        return GNNFD_INVALID_ARG;
    OneshotLayout L;
    int rc = oneshot_layout(n, e, flags, heads * dim, heads, &L);
    if (rc) return rc;
    if (scratch_bytes < L.persistent + L.build_scratch + L.aggregate) return GNNFD_WORKSPACE_TOO_SMALL;
    char* base = static_cast<char*>(d_scratch);
    gnnfd_csr_t* csr = nullptr;
    rc = gnnfd_build_csr(n, e, d_src, d_dst, itype, oneshot_flags(flags), base, L.persistent, base + L.persistent,
                         L.build_scratch, stream, &csr);
    if (rc) return rc;
    rc = gnnfd_aggregate_gat(csr, d_z, ldz, zdt, d_a_src, d_a_dst, heads, dim, negative_slope, d_out, ldo, odt, chunk_width,
                             base + L.persistent + L.build_scratch, L.aggregate, stream);
    gnnfd_csr_destroy(csr);
    return rc;
}

int gnnfd_oneshot_gcn(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                      const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f,
                      int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream)
{
    return gnnfd::oneshot(true, n, e, d_src, d_dst, itype, flags, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, d_scratch,
                          scratch_bytes, stream);
}

int gnnfd_oneshot_sage(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                       const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f,
                       int32_t chunk_width, void* d_scratch, size_t scratch_bytes, void* stream)
{
    return gnnfd::oneshot(false, n, e, d_src, d_dst, itype, flags, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, d_scratch,
                          scratch_bytes, stream);
}

}  // extern "C"
