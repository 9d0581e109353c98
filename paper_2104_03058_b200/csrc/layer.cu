// A whole layer on a built CSR: the dense transform first, then the aggregation of the transformed features
// (Section III runs the Combination phase ahead of the Aggregation phase).  Only plumbing lives here: the
// transform is combine.cu's kernel, the aggregation the gather kernels; for GAT the transform's epilogue writes
// the attention scores straight into the place where the fused aggregation expects them.
#include "common.cuh"

namespace gnnfd {

static int32_t z_pitch(int32_t f_out) { return (int32_t)align_up((size_t)f_out, 8); }      // 16-byte rows for fp32 and bf16

static size_t z_bytes(const gnnfd_csr_t* csr, int32_t f_out, gnnfd_dtype_t xdt)
{
    return align_up((size_t)csr->n * z_pitch(f_out) * (xdt == GNNFD_BF16 ? 2 : 4), 256);
}

static int layer_sum(bool weighted, const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in,
                     const void* d_w_t, int64_t ldw, int32_t f_out, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt,
                     int32_t chunk_width, void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream)
{
    if (!csr || f_out <= 0 || !d_scratch || ((uintptr_t)d_scratch & 255u)) return GNNFD_INVALID_ARG;
    if (xdt != GNNFD_F32 && xdt != GNNFD_BF16) return GNNFD_UNSUPPORTED;
    const size_t zb = z_bytes(csr, f_out, xdt);
    if (scratch_bytes < zb) return GNNFD_WORKSPACE_TOO_SMALL;
    void* z = d_scratch;
    int rc = combine_impl(csr->n, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, z, z_pitch(f_out), xdt, mode, nullptr, nullptr, 0, 0,
                          nullptr, nullptr, d_status, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    void* rest = static_cast<char*>(d_scratch) + zb;
    return weighted ? gnnfd_aggregate_gcn(csr, z, z_pitch(f_out), xdt, d_out, ldo, odt, f_out, chunk_width, rest,
                                          scratch_bytes - zb, stream)
                    : gnnfd_aggregate_sage(csr, z, z_pitch(f_out), xdt, d_out, ldo, odt, f_out, chunk_width, rest,
                                           scratch_bytes - zb, stream);
}

}  // namespace gnnfd

extern "C" {

int gnnfd_layer_workspace_bytes(const gnnfd_csr_t* csr, int model, int32_t f_out, int32_t heads, int32_t dim,
                                gnnfd_dtype_t xdt, size_t* scratch_bytes)
{
    using namespace gnnfd;
    if (!csr || !scratch_bytes || model < 0 || model > 2) return GNNFD_INVALID_ARG;
    if (xdt != GNNFD_F32 && xdt != GNNFD_BF16) return GNNFD_UNSUPPORTED;
    size_t rest = 0;
    int rc;
    if (model == 2) {
        if (heads <= 0 || dim <= 0 || (int64_t)heads * dim > 0x7fffffffll) return GNNFD_INVALID_ARG;
        f_out = heads * dim;
        rc = gnnfd_gat_workspace_bytes(csr, heads, dim, &rest);
    } else {
        if (f_out <= 0) return GNNFD_INVALID_ARG;
        rc = gnnfd_aggregate_workspace_bytes(csr, f_out, &rest);
    }
    if (rc) return rc;
    *scratch_bytes = z_bytes(csr, f_out, xdt) + align_up(rest, 256);
    return GNNFD_OK;
}

int gnnfd_layer_gcn(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t,
                    int64_t ldw, int32_t f_out, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t chunk_width,
                    void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream)
{
    return gnnfd::layer_sum(true, csr, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, mode, d_out, ldo, odt, chunk_width, d_scratch,
                            scratch_bytes, d_status, stream);
}

int gnnfd_layer_sage(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t,
                     int64_t ldw, int32_t f_out, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t chunk_width,
                     void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream)
{
    return gnnfd::layer_sum(false, csr, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, mode, d_out, ldo, odt, chunk_width, d_scratch,
                            scratch_bytes, d_status, stream);
}

int gnnfd_layer_gat(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t,
                    int64_t ldw, int32_t heads, int32_t dim, const float* d_a_src, const float* d_a_dst,
                    float negative_slope, int mode, void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t chunk_width,
                    void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream)
{
    using namespace gnnfd;
    if (!csr || heads <= 0 || dim <= 0 || (int64_t)heads * dim > 0x7fffffffll || !d_a_src || !d_a_dst || !d_scratch ||
        ((uintptr_t)d_scratch & 255u))
        return GNNFD_INVALID_ARG;
    if (xdt != GNNFD_F32 && xdt != GNNFD_BF16) return GNNFD_UNSUPPORTED;
    const int32_t f_out = heads * dim;
    const size_t zb = z_bytes(csr, f_out, xdt);
    if (scratch_bytes < zb) return GNNFD_WORKSPACE_TOO_SMALL;
    void* z = d_scratch;
    void* rest = static_cast<char*>(d_scratch) + zb;
    float *s_src = nullptr, *s_dst = nullptr;
    int rc = gat_scratch_scores(csr, heads, dim, rest, scratch_bytes - zb, &s_src, &s_dst);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = combine_impl(csr->n, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, z, z_pitch(f_out), xdt, mode, d_a_src, d_a_dst, heads, dim,
                      s_src, s_dst, d_status, s);
    bool scores_ready = rc == GNNFD_OK;
    if (rc == GNNFD_UNSUPPORTED)      // heads that straddle the transform's column tiles: plain transform, separate scores pass
        rc = combine_impl(csr->n, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, z, z_pitch(f_out), xdt, mode, nullptr, nullptr, 0, 0,
                          nullptr, nullptr, d_status, s);
    if (rc) return rc;
    return gat_aggregate_impl(csr, z, z_pitch(f_out), xdt, d_a_src, d_a_dst, heads, dim, negative_slope, d_out, ldo, odt,
                              chunk_width, rest, scratch_bytes - zb, scores_ready, s);
}

}  // extern "C"
