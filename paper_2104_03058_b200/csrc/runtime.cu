// Diagnostics, launch bookkeeping, handle accessors and the device prefix sum used by the build.
#include <atomic>
#include <cstring>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace gnnfd {

static thread_local int g_last_cuda_error = 0;
static std::atomic<int64_t> g_launches{0};
static std::atomic<int> g_timing{0};

struct TimedLaunch { const char* name; cudaEvent_t start, stop; };
static std::mutex g_timing_mutex;
static std::vector<TimedLaunch> g_timed;

void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

LaunchScope::LaunchScope(const char* name_, cudaStream_t s) : name(name_), stream(s), rec(nullptr)
{
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (g_timing.load(std::memory_order_relaxed)) {
        TimedLaunch* t = new TimedLaunch{name_, nullptr, nullptr};
        if (cudaEventCreate(&t->start) == cudaSuccess && cudaEventCreate(&t->stop) == cudaSuccess) {
            cudaEventRecord(t->start, s);
            rec = t;
        } else {
            if (t->start) cudaEventDestroy(t->start);
            delete t;
        }
    }
}

LaunchScope::~LaunchScope()
{
    if (rec) {
        TimedLaunch* t = static_cast<TimedLaunch*>(rec);
        cudaEventRecord(t->stop, stream);
        std::lock_guard<std::mutex> lock(g_timing_mutex);
        g_timed.push_back(*t);
        delete t;
    }
}

// ------------------------------------------------------------------ exclusive scan (int32)
//
// Three-phase scan without inter-block waiting: per-tile sums, a recursive scan of those sums,
// then a per-tile scan seeded with its offset.  Tile = 256 threads x 8 items.

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

__device__ __forceinline__ int32_t block_exclusive_scan(int32_t v, int32_t* total, int32_t* smem /*[8]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    int32_t warp_off = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kScanThreads / 32; ++w) {
        int32_t s = smem[w];
        if (w < warp) warp_off += s;
        all += s;
    }
    __syncthreads();
    *total = all;
    return warp_off + inc - v;
}

// the kScanItems values of one thread, with two 16-byte loads when the whole group exists and is aligned
__device__ __forceinline__ void load_scan_items(const int32_t* in, size_t base, size_t count, bool vec, int32_t (&item)[kScanItems])
{
    static_assert(kScanItems == 8, "two 16-byte vectors per thread");
    if (vec && base + kScanItems <= count) {
        const int4 a = *reinterpret_cast<const int4*>(in + base), b = *reinterpret_cast<const int4*>(in + base + 4);
        item[0] = a.x; item[1] = a.y; item[2] = a.z; item[3] = a.w;
        item[4] = b.x; item[5] = b.y; item[6] = b.z; item[7] = b.w;
    } else {
#pragma unroll
        for (int i = 0; i < kScanItems; ++i) item[i] = base + i < count ? in[base + i] : 0;
    }
}

__global__ void __launch_bounds__(kScanThreads) scan_tile_sums(const int32_t* __restrict__ in, size_t count,
                                                             int32_t* __restrict__ sums)
{
    __shared__ int32_t smem[8];
    const size_t base = (size_t)blockIdx.x * kScanTile + (size_t)threadIdx.x * kScanItems;
    const bool vec = (reinterpret_cast<uintptr_t>(in) & 15u) == 0;
    int32_t item[kScanItems];
    load_scan_items(in, base, count, vec, item);
    int32_t v = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) v += item[i];
    int32_t total;
    block_exclusive_scan(v, &total, smem);
    if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kScanThreads) scan_tiles(const int32_t* in, int32_t* out, size_t count,
                                                         const int32_t* offsets)
{
    __shared__ int32_t smem[8];
    const size_t base = (size_t)blockIdx.x * kScanTile + (size_t)threadIdx.x * kScanItems;
    const bool vec = ((reinterpret_cast<uintptr_t>(in) | reinterpret_cast<uintptr_t>(out)) & 15u) == 0;
    int32_t item[kScanItems];
    load_scan_items(in, base, count, vec, item);
    int32_t v = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) v += item[i];
    int32_t total;
    int32_t run = block_exclusive_scan(v, &total, smem) + (offsets ? offsets[blockIdx.x] : 0);
    int32_t res[kScanItems];
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        res[i] = run;
        run += item[i];
    }
    if (vec && base + kScanItems <= count) {
        *reinterpret_cast<int4*>(out + base) = make_int4(res[0], res[1], res[2], res[3]);
        *reinterpret_cast<int4*>(out + base + 4) = make_int4(res[4], res[5], res[6], res[7]);
    } else {
#pragma unroll
        for (int i = 0; i < kScanItems; ++i)
            if (base + i < count) out[base + i] = res[i];
    }
}

size_t scan_temp_ints(size_t count)
{
    size_t total = 0;
    while (count > (size_t)kScanTile) {
        size_t tiles = (count + kScanTile - 1) / kScanTile;
        total += align_up(tiles, 64);
        count = tiles;
    }
    return total + 64;
}

int exclusive_scan_i32(const int32_t* d_in, int32_t* d_out, size_t count, int32_t* d_temp, cudaStream_t s)
{
    if (count == 0) return GNNFD_OK;
    const size_t tiles = (count + kScanTile - 1) / kScanTile;
    if (tiles == 1) {
        GNNFD_LAUNCH("scan_tiles", s, scan_tiles, 1, kScanThreads, 0, d_in, d_out, count, nullptr);
    } else {
        int32_t* sums = d_temp;
        GNNFD_LAUNCH("scan_tile_sums", s, scan_tile_sums, (unsigned)tiles, kScanThreads, 0, d_in, count, sums);
        int rc = exclusive_scan_i32(sums, sums, tiles, d_temp + align_up(tiles, 64), s);
        if (rc) return rc;
        GNNFD_LAUNCH("scan_tiles", s, scan_tiles, (unsigned)tiles, kScanThreads, 0, d_in, d_out, count, sums);
    }
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" {

const char* gnnfd_status_string(int status)
{
    switch (status) {
        case GNNFD_OK: return "ok";
        case GNNFD_INVALID_ARG: return "invalid argument";
        case GNNFD_BAD_INDEX: return "vertex id out of range in the edge list";
        case GNNFD_TOO_LARGE: return "graph too large for the int32 structure";
        case GNNFD_WORKSPACE_TOO_SMALL: return "workspace buffer too small";
        case GNNFD_UNSUPPORTED: return "unsupported dtype or index type";
        case GNNFD_CUDA_ERROR: return "CUDA runtime error";
        case GNNFD_STATIC_SCRATCH_EXCEEDED: return "built-in workspace too small for this call";
        default: return "unknown status";
    }
}

int gnnfd_last_cuda_error(void) { return gnnfd::g_last_cuda_error; }

int64_t gnnfd_launch_count(void) { return gnnfd::g_launches.load(); }

int gnnfd_kernel_timing_enable(int on)
{
    gnnfd::g_timing.store(on ? 1 : 0);
    return GNNFD_OK;
}

int gnnfd_kernel_timing_read(const char** names, double* ms, int64_t* launches, int capacity)
{
    using namespace gnnfd;
    std::vector<TimedLaunch> taken;
    {
        std::lock_guard<std::mutex> lock(g_timing_mutex);
        taken.swap(g_timed);
    }
    std::vector<const char*> seen;
    std::vector<double> total;
    std::vector<int64_t> count;
    int status = GNNFD_OK;
    for (TimedLaunch& t : taken) {
        float dt = 0.f;
        cudaError_t e = cudaEventSynchronize(t.stop);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&dt, t.start, t.stop);
        if (e != cudaSuccess) { set_cuda_error(e); status = GNNFD_CUDA_ERROR; }
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
        size_t i = 0;
        for (; i < seen.size(); ++i)
            if (std::strcmp(seen[i], t.name) == 0) break;
        if (i == seen.size()) { seen.push_back(t.name); total.push_back(0.0); count.push_back(0); }
        total[i] += dt;
        count[i] += 1;
    }
    if (status != GNNFD_OK) return status;
    for (size_t i = 0; i < seen.size() && (int)i < capacity; ++i) {
        if (names) names[i] = seen[i];
        if (ms) ms[i] = total[i];
        if (launches) launches[i] = count[i];
    }
    return (int)seen.size();
}

int gnnfd_csr_info(const gnnfd_csr_t* csr, int64_t* n, int64_t* nnz, const int32_t** d_row_ptr,
                   const int32_t** d_col_idx, const int32_t** d_perm, const float** d_dinv_sqrt,
                   const float** d_rdeg, const float** d_edge_weight, int32_t* max_degree)
{
    if (!csr) return GNNFD_INVALID_ARG;
    if (n) *n = csr->n;
    if (nnz) *nnz = csr->nnz;
    if (d_row_ptr) *d_row_ptr = csr->row_ptr;
    if (d_col_idx) *d_col_idx = csr->col_idx;
    if (d_perm) *d_perm = csr->perm;
    if (d_dinv_sqrt) *d_dinv_sqrt = csr->dinv;
    if (d_rdeg) *d_rdeg = csr->rdeg;
    if (d_edge_weight) *d_edge_weight = csr->edge_w;
    if (max_degree) *max_degree = csr->max_degree;
    return GNNFD_OK;
}

int gnnfd_csr_schedule(const gnnfd_csr_t* csr, int64_t bin_count[5], const int32_t** d_row_order,
                       int64_t* n_segments, const int32_t** d_seg_row, const int32_t** d_seg_begin,
                       const int32_t** d_seg_end, const int32_t** d_seg_slot, const int32_t** d_hub_seg_ptr)
{
    if (!csr) return GNNFD_INVALID_ARG;
    if (bin_count)
        for (int b = 0; b < gnnfd::kNumBins; ++b) bin_count[b] = csr->bin_count[b];
    if (d_row_order) *d_row_order = csr->row_order;
    if (n_segments) *n_segments = csr->n_segments;
    if (d_seg_row) *d_seg_row = csr->seg_row;
    if (d_seg_begin) *d_seg_begin = csr->seg_begin;
    if (d_seg_end) *d_seg_end = csr->seg_end;
    if (d_seg_slot) *d_seg_slot = csr->seg_slot;
    if (d_hub_seg_ptr) *d_hub_seg_ptr = csr->hub_seg_ptr;
    return GNNFD_OK;
}

void gnnfd_csr_destroy(gnnfd_csr_t* csr) { delete csr; }

}  // extern "C"
