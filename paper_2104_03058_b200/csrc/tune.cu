// Chunk-width selection by measurement.  The paper leaves the number of decomposition layers to the
// user, to be set from the device's memory and the dataset at hand (Section II-B); the best width depends on how the graph's gathers hit the caches, which a size
// formula does not capture (an RMAT graph with 2 M vertices runs fastest undecomposed, the
// Reddit-shaped graph at 64 columns), so the candidates are simply timed on the caller's data.
#include "common.cuh"

extern "C" {

int gnnfd_default_chunk_candidates(int32_t f, gnnfd_dtype_t xdt, int32_t* candidates, int capacity)
{
    if (f <= 0 || !candidates || capacity <= 0) return GNNFD_INVALID_ARG;
    if (xdt != GNNFD_F32 && xdt != GNNFD_BF16) return GNNFD_UNSUPPORTED;
    const int vec = xdt == GNNFD_F32 ? 4 : 8;          // elements per 16-byte vector
    int count = 0;
    candidates[count++] = f;                           // no decomposition
    for (int w = 256; w >= 2 * vec && count < capacity; w >>= 1)
        if (w < f) candidates[count++] = w;
    return count;
}

int gnnfd_tune_chunk_width(const gnnfd_csr_t* csr, int model, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                           void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, const int32_t* candidates,
                           int n_candidates, void* d_scratch, size_t scratch_bytes, void* stream, int32_t* best_width,
                           float* best_ms)
{
    if (!candidates || n_candidates <= 0 || !best_width || (model != 0 && model != 1)) return GNNFD_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t t0 = nullptr, t1 = nullptr;
    GNNFD_CUDA_CHECK(cudaEventCreate(&t0));
    cudaError_t e = cudaEventCreate(&t1);
    if (e != cudaSuccess) { cudaEventDestroy(t0); gnnfd::set_cuda_error(e); return GNNFD_CUDA_ERROR; }
    int status = GNNFD_OK;
    float best = -1.f;
    for (int i = 0; i < n_candidates && status == GNNFD_OK; ++i) {
        const int32_t w = candidates[i];
        for (int rep = 0; rep < 2 && status == GNNFD_OK; ++rep) {      // the second call is the timed one
            if (rep == 1) cudaEventRecord(t0, s);
            status = model == 0
                ? gnnfd_aggregate_gcn(csr, d_x, ldx, xdt, d_out, ldo, odt, f, w, d_scratch, scratch_bytes, stream)
                : gnnfd_aggregate_sage(csr, d_x, ldx, xdt, d_out, ldo, odt, f, w, d_scratch, scratch_bytes, stream);
        }
        if (status != GNNFD_OK) break;
        cudaEventRecord(t1, s);
        e = cudaEventSynchronize(t1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t0, t1);
        if (e != cudaSuccess) { gnnfd::set_cuda_error(e); status = GNNFD_CUDA_ERROR; break; }
        if (best < 0.f || ms < best) { best = ms; *best_width = w; }
    }
    cudaEventDestroy(t0);
    cudaEventDestroy(t1);
    if (status == GNNFD_OK && best_ms) *best_ms = best;
    return status;
}

}  // extern "C"
