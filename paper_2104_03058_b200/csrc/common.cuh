// Shared host-side plumbing of the gnnfd library: handle layout, launch bookkeeping, error capture.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gnnfd.h"

namespace gnnfd {

constexpr int kNumBins = 5;                 // four degree classes + hub rows
constexpr int kBinDeg0 = 8, kBinDeg1 = 32, kBinDeg2 = 128, kBinDeg3 = GNNFD_HUB_DEGREE;   // upper degree of each class
constexpr int kHubSegment = GNNFD_HUB_SEGMENT;

// Device-side counters filled during the build and copied to the host once.
struct BuildCounts {
    int32_t bad_index;       // ids outside [0, n)
    int32_t n_valid;         // candidate edges that survive the self-loop / reverse-edge rules
    int32_t nnz;             // entries after dedup
    int32_t max_degree;
    int32_t n_segments;      // hub segments
    int32_t bin_count[kNumBins];
    int32_t pad[6];
};

}  // namespace gnnfd

struct gnnfd_csr {
    int64_t n, nnz;
    int32_t max_degree;
    int64_t bin_count[gnnfd::kNumBins];
    int64_t bin_start[gnnfd::kNumBins];
    int64_t n_segments;
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* perm;
    const float* dinv;
    const float* rdeg;
    const float* edge_w;
    const int32_t* row_order;
    const int32_t* seg_row;
    const int32_t* seg_begin;
    const int32_t* seg_end;
    const int32_t* seg_slot;
    const int32_t* hub_seg_ptr;
};

namespace gnnfd {

void set_cuda_error(cudaError_t e);

// Records the launch (count, optional event bracket).  Use through GNNFD_LAUNCH.
struct LaunchScope {
    LaunchScope(const char* name, cudaStream_t s);
    ~LaunchScope();
    const char* name;
    cudaStream_t stream;
    void* rec;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Bump allocator over a caller-provided device buffer.
struct Carver {
    char* base;
    size_t off, cap;
    bool ok;
    Carver(void* p, size_t bytes) : base(static_cast<char*>(p)), off(0), cap(bytes), ok(true) {}
    template <typename T>
    T* take(size_t count)
    {
        size_t bytes = align_up(count * sizeof(T), 256);
        if (off + bytes > cap) { ok = false; off += bytes; return nullptr; }
        T* r = reinterpret_cast<T*>(base + off);
        off += bytes;
        return r;
    }
};

// Exclusive prefix sum of `count` int32 values (in -> out, may alias), temp from scan_temp_ints().
size_t scan_temp_ints(size_t count);
int exclusive_scan_i32(const int32_t* d_in, int32_t* d_out, size_t count, int32_t* d_temp, cudaStream_t s);

// ---- pieces of one translation unit that the layer entry points (layer.cu) put together

int64_t segment_capacity(int64_t n, int64_t e, uint32_t flags);      // csr_build.cu; -1 for sizes the build rejects

int combine_impl(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t, int64_t ldw,
                 int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int mode, const float* d_a_src,
                 const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst, int32_t* d_status,
                 cudaStream_t s);
int gat_aggregate_impl(const gnnfd_csr_t* csr, const void* d_z, int64_t ldz, gnnfd_dtype_t zdt, const float* d_a_src,
                       const float* d_a_dst, int32_t heads, int32_t dim, float negative_slope, void* d_out, int64_t ldo,
                       gnnfd_dtype_t odt, int32_t chunk_width, void* d_scratch, size_t scratch_bytes, bool scores_ready,
                       cudaStream_t s);
int gat_scratch_scores(const gnnfd_csr_t* csr, int32_t heads, int32_t dim, void* d_scratch, size_t scratch_bytes,
                       float** s_src, float** s_dst);

}  // namespace gnnfd

#define GNNFD_LAUNCH(name, stream, kernel, grid, block, smem, ...)                   \
    do {                                                                             \
        ::gnnfd::LaunchScope scope_(name, stream);                                   \
        kernel<<<grid, block, smem, stream>>>(__VA_ARGS__);                          \
    } while (0)

#define GNNFD_CUDA_CHECK(expr)                                                       \
    do {                                                                             \
        cudaError_t err_ = (expr);                                                   \
        if (err_ != cudaSuccess) { ::gnnfd::set_cuda_error(err_); return GNNFD_CUDA_ERROR; } \
    } while (0)
