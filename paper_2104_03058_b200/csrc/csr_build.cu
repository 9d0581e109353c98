// Device CSR-by-destination builder: key generation, stable LSD radix sort of (dst, src) keys,
// duplicate removal, row pointers, degree normalisers, GCN edge weights and the launch schedule
// (degree bins, hub segments).  Integer work throughout; the only host synchronisation is the
// final read of the counters.
#include <cstddef>
#include <cstring>
#include <new>

#include "common.cuh"

namespace gnnfd {

using u64 = unsigned long long;

constexpr int kThreads = 256;
constexpr int kMaxDigitBits = 9;
constexpr int kRadix = 1 << kMaxDigitBits;           // histogram bins (a pass may use fewer)
constexpr int kSortTile = 4096;                      // keys per block of a sort pass
#ifndef GNNFD_SCATTER_THREADS
#define GNNFD_SCATTER_THREADS 256
#endif
constexpr int kHistItems = kSortTile / kThreads;     // keys per thread of the histogram kernel
constexpr int kScatterThreads = GNNFD_SCATTER_THREADS;
constexpr int kSortItems = kSortTile / kScatterThreads;   // keys per thread of the scatter kernel
constexpr int kSortWarps = kScatterThreads / 32;
constexpr int kWarpItems = 32 * kSortItems;
constexpr int kOwnDigits = kRadix / kScatterThreads; // digit values a scatter thread looks after
static_assert(kRadix % kScatterThreads == 0 && kOwnDigits >= 1, "a scatter block must cover the digit values evenly");

static inline unsigned blocks_for(size_t count, int per_block)
{
    size_t b = (count + per_block - 1) / per_block;
    return (unsigned)(b ? b : 1);
}

// ------------------------------------------------------------------ keys

// Candidate i < e: input edge i.  e <= i < 2e (symmetrise): reverse of edge i - e.  Then one
// self-loop per vertex (value -1).  key = (dst << src_bits) | src; dropped candidates get the
// destination n, above every valid key, so the sort moves them behind the kept ones.  When key and
// value fit one 64-bit word together (vals == nullptr) the word is key << val_bits | (value + 1) and
// every later kernel reads the key as word >> val_bits.
constexpr int kKeyItems = 4;                          // candidates per thread of make_keys / entries per thread of finalize_entries

template <typename IdT>
__global__ void __launch_bounds__(kThreads)
make_keys(const IdT* __restrict__ src, const IdT* __restrict__ dst, int64_t n, int64_t e, int64_t m, uint32_t flags,
          int src_bits, int val_bits, u64* __restrict__ keys, int32_t* __restrict__ vals,
          BuildCounts* __restrict__ counts)
{
    const int64_t base = (int64_t)blockIdx.x * (kThreads * kKeyItems) + threadIdx.x;
    const u64 invalid = (u64)n << src_bits;
    const int64_t n_rev = (flags & GNNFD_CSR_SYMMETRIZE) ? e : 0;
    int kept = 0, bads = 0;
    auto emit = [&](int64_t i, int64_t sv, int64_t dv, int32_t val, bool keep) {
        const u64 key = keep ? (((u64)dv << src_bits) | (u64)sv) : invalid;
        if (vals) {
            __stcs(keys + i, key);
            __stcs(vals + i, val);
        } else {
            __stcs(keys + i, (key << val_bits) | (u64)(uint32_t)(val + 1));   // value travels in the low bits
        }
        kept += keep ? 1 : 0;
    };
    if ((int64_t)(blockIdx.x + 1) * (kThreads * kKeyItems) <= e) {
        // the block lies inside the plain input edges: all loads are issued before the first store
        IdT sv[kKeyItems], dv[kKeyItems];
#pragma unroll
        for (int j = 0; j < kKeyItems; ++j) {
            sv[j] = __ldcs(src + base + j * kThreads);
            dv[j] = __ldcs(dst + base + j * kThreads);
        }
#pragma unroll
        for (int j = 0; j < kKeyItems; ++j) {
            const int64_t s64 = (int64_t)sv[j], d64 = (int64_t)dv[j];
            const bool bad = s64 < 0 || s64 >= n || d64 < 0 || d64 >= n;
            bads += bad ? 1 : 0;
            emit(base + j * kThreads, s64, d64, (int32_t)(base + j * kThreads),
                 !bad && !((flags & GNNFD_CSR_ADD_SELF_LOOPS) && s64 == d64));
        }
    } else {
        for (int j = 0; j < kKeyItems; ++j) {
            const int64_t i = base + j * kThreads;
            if (i >= m) break;
            if (i < e) {
                const int64_t s64 = (int64_t)src[i], d64 = (int64_t)dst[i];
                const bool bad = s64 < 0 || s64 >= n || d64 < 0 || d64 >= n;
                bads += bad ? 1 : 0;
                emit(i, s64, d64, (int32_t)i, !bad && !((flags & GNNFD_CSR_ADD_SELF_LOOPS) && s64 == d64));
            } else if (i < e + n_rev) {
                const int64_t s64 = (int64_t)dst[i - e], d64 = (int64_t)src[i - e];
                emit(i, s64, d64, (int32_t)i, !(s64 < 0 || s64 >= n || d64 < 0 || d64 >= n) && s64 != d64);
            } else {
                emit(i, i - e - n_rev, i - e - n_rev, -1, true);
            }
        }
    }
    // one atomic per block and counter: all blocks add to the same two words
    __shared__ int warp_kept[kThreads / 32], warp_bads[kThreads / 32];
    const int kept_warp = __reduce_add_sync(0xffffffffu, kept), bads_warp = __reduce_add_sync(0xffffffffu, bads);
    if ((threadIdx.x & 31) == 0) {
        warp_kept[threadIdx.x >> 5] = kept_warp;
        warp_bads[threadIdx.x >> 5] = bads_warp;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int kept_all = 0, bads_all = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) { kept_all += warp_kept[w]; bads_all += warp_bads[w]; }
        if (kept_all) atomicAdd(&counts->n_valid, kept_all);
        if (bads_all) atomicAdd(&counts->bad_index, bads_all);
    }
}

// ------------------------------------------------------------------ radix sort (one digit of up to 9 bits per pass)

__global__ void __launch_bounds__(kThreads)
radix_histogram(const u64* __restrict__ keys, int64_t m, int shift, int mask, int64_t n_tiles, int32_t* __restrict__ hist)
{
    __shared__ int32_t h[kRadix];
    h[threadIdx.x] = 0;
    h[threadIdx.x + kThreads] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
    if (base + kSortTile <= m) {
        // full tile: 16-byte loads, all of them issued before the first shared-memory atomic
        const ulonglong2* k2 = reinterpret_cast<const ulonglong2*>(keys + base);
        ulonglong2 v[kHistItems / 2];
#pragma unroll
        for (int i = 0; i < kHistItems / 2; ++i) v[i] = __ldcs(k2 + i * kThreads + threadIdx.x);
#pragma unroll
        for (int i = 0; i < kHistItems / 2; ++i) {
            atomicAdd(&h[(int)(v[i].x >> shift) & mask], 1);
            atomicAdd(&h[(int)(v[i].y >> shift) & mask], 1);
        }
    } else {
#pragma unroll
        for (int i = 0; i < kHistItems; ++i) {
            const int64_t idx = base + i * kThreads + threadIdx.x;
            if (idx < m) atomicAdd(&h[(int)(keys[idx] >> shift) & mask], 1);
        }
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
    hist[(int64_t)(threadIdx.x + kThreads) * n_tiles + blockIdx.x] = h[threadIdx.x + kThreads];
}

struct ScatterSmem {
    u64 keys[kSortTile];
    int32_t warp_count[kSortWarps][kRadix];
    int32_t digit_base[kRadix];     // first slot of each digit inside the sorted tile
    int32_t to_global[kRadix];      // global position of tile slot i holding digit d: to_global[d] + i
    int32_t scan[kSortWarps];
    int32_t vals[kSortTile];        // last: not allocated when the values travel inside the keys
};

// exclusive scan of one value per thread over a scatter block; *total receives the block sum
__device__ __forceinline__ int32_t block_scan(int32_t v, int32_t* total, int32_t* smem)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    int32_t off = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
        const int32_t s = smem[w];
        if (w < warp) off += s;
        all += s;
    }
    *total = all;
    return off + inc - v;
}

// Lanes of the warp that hold the same digit value (among the valid ones): one ballot per digit bit.
// The match instruction gives the same mask, but measured on this part it occupies its pipe for about
// 56 cycles per warp, against about 21 ALU cycles for the nine ballots and their masking.  The two run
// on different pipes, so the scatter uses the match instruction for GNNFD_SCATTER_MATCH_ROUNDS of a
// warp's 16 rounds and ballots for the rest (config 4, per build: all match 3.59 ms, all ballots 3.09,
// 3 / 5 / 7 rounds of match 3.02 / 2.86 / 2.99).
__device__ __forceinline__ unsigned lanes_with_equal_digit(int digit, bool valid)
{
    unsigned peers = __ballot_sync(0xffffffffu, valid);
#pragma unroll
    for (int b = 0; b < kMaxDigitBits; ++b) {
        const bool bit = (digit >> b) & 1;
        const unsigned with_bit = __ballot_sync(0xffffffffu, bit);
        peers &= bit ? with_bit : ~with_bit;
    }
    return valid ? peers : 0u;
}

// Stable scatter of one tile.  A warp owns kWarpItems consecutive keys and walks them 32 at a time: keys
// with equal digits inside a round are ranked by lane (ballots over the digit's bits), across rounds by a per-warp running
// count, across warps by a prefix over the per-warp counts.  The tile is then laid out sorted by
// digit in shared memory and written out run by run, so that consecutive threads store to
// consecutive addresses; the run of digit d starts at the scanned histogram entry of (d, tile).
#ifndef GNNFD_SCATTER_MATCH_ROUNDS
#define GNNFD_SCATTER_MATCH_ROUNDS 5
#endif
#ifndef GNNFD_SCATTER_MIN_BLOCKS
#define GNNFD_SCATTER_MIN_BLOCKS 3
#endif
template <bool HAS_VALS>
__global__ void __launch_bounds__(kScatterThreads, GNNFD_SCATTER_MIN_BLOCKS)
radix_scatter(const u64* __restrict__ keys_in, const int32_t* __restrict__ vals_in, u64* __restrict__ keys_out,
              int32_t* __restrict__ vals_out, int64_t m, int shift, int mask, int64_t n_tiles,
              const int32_t* __restrict__ tile_offset)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ScatterSmem& sm = *reinterpret_cast<ScatterSmem*>(smem_raw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSortWarps * kRadix; i += kScatterThreads) (&sm.warp_count[0][0])[i] = 0;
    __syncthreads();

    const int64_t tile_base = (int64_t)blockIdx.x * kSortTile;
    const int64_t warp_base = tile_base + (int64_t)warp * kWarpItems;
    u64 key[kSortItems];
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
        const int64_t idx = warp_base + r * 32 + lane;
        key[r] = idx < m ? __ldcs(keys_in + idx) : 0ull;
    }
    int32_t rank[kSortItems];
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
        const bool valid = warp_base + r * 32 + lane < m;
        const int digit = (int)(key[r] >> shift) & mask;
        // some rounds use the match instruction, the others ballots: the two run on different pipes
        const unsigned peers = r < GNNFD_SCATTER_MATCH_ROUNDS ? __match_any_sync(0xffffffffu, valid ? digit : kRadix)
                                                              : lanes_with_equal_digit(digit, valid);
        const int leader = __ffs(peers) - 1;
        // the leader of each digit bumps the warp's running count; a warp's shared-memory atomics on one
        // address complete in program order, so the rounds need no barrier between them
        int32_t before = 0;
        if (lane == leader && valid) before = atomicAdd(&sm.warp_count[warp][digit], __popc(peers));
        before = __shfl_sync(0xffffffffu, before, leader);
        rank[r] = before + __popc(peers & ((1u << lane) - 1u));
    }
    __syncthreads();
    {
        // per-warp counts -> exclusive prefix over warps; thread t owns digit values t, t + blockDim, ...
        int32_t carry = 0;
#pragma unroll
        for (int q = 0; q < kOwnDigits; ++q) {
            const int d = threadIdx.x + q * kScatterThreads;
            int32_t run = 0;
#pragma unroll
            for (int w = 0; w < kSortWarps; ++w) {
                const int32_t c = sm.warp_count[w][d];
                sm.warp_count[w][d] = run;
                run += c;
            }
            int32_t total;
            const int32_t base = block_scan(run, &total, sm.scan) + carry;
            carry += total;
            sm.digit_base[d] = base;
            sm.to_global[d] = tile_offset[(int64_t)d * n_tiles + blockIdx.x] - base;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
        if (warp_base + r * 32 + lane < m) {
            const int digit = (int)(key[r] >> shift) & mask;
            const int slot = sm.digit_base[digit] + sm.warp_count[warp][digit] + rank[r];
            sm.keys[slot] = key[r];
            if (HAS_VALS) sm.vals[slot] = __ldcs(vals_in + warp_base + r * 32 + lane);
        }
    }
    __syncthreads();
    const int count = (int)min((int64_t)kSortTile, m - tile_base);
    for (int i = threadIdx.x; i < count; i += kScatterThreads) {
        const u64 k = sm.keys[i];
        const int64_t pos = (int64_t)sm.to_global[(int)(k >> shift) & mask] + i;
        keys_out[pos] = k;
        if (HAS_VALS) vals_out[pos] = sm.vals[i];
    }
}

// ------------------------------------------------------------------ after the sort

// Duplicate removal after the sort, in two sweeps with a scan of one count per tile between them: a
// sorted candidate is kept when it is valid and its key differs from its predecessor's.  A thread
// looks after kUniqueItems consecutive candidates, a block after kUniqueTile.
constexpr int kUniqueItems = 8;
constexpr int kUniqueTile = kThreads * kUniqueItems;

// bit j of the result: candidate first + j is the first of a run of equal keys among the n_valid kept ones
__device__ __forceinline__ uint32_t first_of_run_mask(const u64* __restrict__ keys, int64_t first, int64_t n_valid, int val_bits,
                                                      u64 (&word)[kUniqueItems])
{
    u64 prev = first > 0 && first <= n_valid ? (__ldg(keys + first - 1) >> val_bits) : 0ull;
    if (first + kUniqueItems <= n_valid) {            // whole group present: 16-byte loads (first is a multiple of 8)
        const ulonglong2* k2 = reinterpret_cast<const ulonglong2*>(keys + first);
#pragma unroll
        for (int j = 0; j < kUniqueItems; j += 2) {
            const ulonglong2 v = __ldcs(k2 + j / 2);
            word[j] = v.x;
            word[j + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int j = 0; j < kUniqueItems; ++j) word[j] = first + j < n_valid ? __ldcs(keys + first + j) : 0ull;
    }
    uint32_t mask = 0;
#pragma unroll
    for (int j = 0; j < kUniqueItems; ++j) {
        const int64_t i = first + j;
        const u64 key = word[j] >> val_bits;
        if (i < n_valid && (i == 0 || key != prev)) mask |= 1u << j;
        prev = key;
    }
    return mask;
}

// sum of one value per thread over the block, and the exclusive prefix of this thread's value
__device__ __forceinline__ int32_t block_prefix_256(int32_t v, int32_t* total, int32_t* smem /*[8]*/)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    int32_t off = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        const int32_t t = smem[w];
        if (w < warp) off += t;
        all += t;
    }
    *total = all;
    return off + inc - v;
}

__global__ void __launch_bounds__(kThreads)
unique_tile_counts(const u64* __restrict__ keys, int val_bits, const BuildCounts* __restrict__ counts,
                   int32_t* __restrict__ tile_count)
{
    __shared__ int32_t smem[kThreads / 32];
    u64 word[kUniqueItems];
    const int64_t first = (int64_t)blockIdx.x * kUniqueTile + (int64_t)threadIdx.x * kUniqueItems;
    const int32_t mine = __popc(first_of_run_mask(keys, first, counts->n_valid, val_bits, word));
    int32_t total;
    block_prefix_256(mine, &total, smem);
    if (threadIdx.x == 0) tile_count[blockIdx.x] = total;
}

// tile_first[t] = kept candidates in earlier tiles; the kept ones move to keys_out / perm in order
__global__ void __launch_bounds__(kThreads)
compact_unique(const u64* __restrict__ keys, const int32_t* __restrict__ vals, const int32_t* __restrict__ tile_first,
               int64_t m, int val_bits, u64* __restrict__ keys_out, int32_t* __restrict__ perm,
               BuildCounts* __restrict__ counts)
{
    __shared__ int32_t smem[kThreads / 32];
    __shared__ u64 kept_key[kUniqueTile];
    __shared__ int32_t kept_val[kUniqueTile];
    u64 word[kUniqueItems];
    const int64_t first = (int64_t)blockIdx.x * kUniqueTile + (int64_t)threadIdx.x * kUniqueItems;
    const uint32_t mask = first_of_run_mask(keys, first, counts->n_valid, val_bits, word);
    int32_t total;
    int32_t pos = block_prefix_256(__popc(mask), &total, smem);
    // the kept candidates of the tile are gathered in shared memory so that they leave as one contiguous piece
#pragma unroll
    for (int j = 0; j < kUniqueItems; ++j) {
        if (mask >> j & 1u) {
            kept_key[pos] = word[j];
            kept_val[pos] = vals ? vals[first + j] : (int32_t)(word[j] & ((1ull << val_bits) - 1ull)) - 1;
            ++pos;
        }
    }
    __syncthreads();
    const int32_t out0 = tile_first[blockIdx.x];
    for (int i = threadIdx.x; i < total; i += kThreads) {
        keys_out[out0 + i] = kept_key[i];
        perm[out0 + i] = kept_val[i];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) counts->nnz = tile_first[blockIdx.x] + total;
}

// row_ptr[v] = number of kept keys with dst < v (binary search in the sorted keys).  Without
// duplicate removal every kept candidate is an entry, which thread 0 records.
__global__ void __launch_bounds__(kThreads)
row_pointers(const u64* __restrict__ keys, BuildCounts* __restrict__ counts, int64_t n, int src_bits, int val_bits,
             int dedup, int32_t* __restrict__ row_ptr)
{
    const int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int32_t nnz = dedup ? counts->nnz : counts->n_valid;
    if (v == 0 && !dedup) counts->nnz = nnz;
    if (v > n) return;
    const u64 target = (u64)v << src_bits;
    int32_t lo = 0, hi = nnz;
    while (lo < hi) {
        const int32_t mid = lo + ((hi - lo) >> 1);
        if ((keys[mid] >> val_bits) < target) lo = mid + 1; else hi = mid;
    }
    row_ptr[v] = lo;
}

// Degree class of a row: exact degree up to 8, then quarter octaves of (deg - 1) up to the hub
// threshold, then one class for hub rows.  Classes are monotone in the degree, so each of the five
// launch bins (<= 8, <= 32, <= 128, <= hub threshold, hub) is a contiguous range of classes.
constexpr int kHubClass = 41;
__device__ __forceinline__ int degree_class(int32_t deg)
{
    if (deg <= kBinDeg0) return deg;
    if (deg > kBinDeg3) return kHubClass;
    const int t = deg - 1;
    const int o = 31 - __clz(t);                       // 3 .. 10
    return 9 + (o - 3) * 4 + ((t >> (o - 2)) & 3);
}
__device__ __forceinline__ int degree_bin(int32_t deg)
{
    return deg <= kBinDeg0 ? 0 : deg <= kBinDeg1 ? 1 : deg <= kBinDeg2 ? 2 : deg <= kBinDeg3 ? 3 : 4;
}

// degree normalisers (rounded once from fp64), the bin sizes, and the (class, row) sort keys
__global__ void __launch_bounds__(kThreads)
degrees_and_classes(const int32_t* __restrict__ row_ptr, int64_t n, float* __restrict__ dinv, float* __restrict__ rdeg,
                    u64* __restrict__ class_keys, int32_t* __restrict__ class_vals, BuildCounts* __restrict__ counts)
{
    const int64_t v = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    int32_t deg = 0;
    int bin = -1;
    if (v < n) {
        deg = row_ptr[v + 1] - row_ptr[v];
        dinv[v] = deg > 0 ? (float)(1.0 / sqrt((double)deg)) : 0.f;
        rdeg[v] = deg > 0 ? (float)(1.0 / (double)deg) : 0.f;
        bin = degree_bin(deg);
        class_keys[v] = ((u64)degree_class(deg) << 32) | (u64)v;
        class_vals[v] = (int32_t)v;
    }
#pragma unroll
    for (int b = 0; b < kNumBins; ++b) {
        const int c = __syncthreads_count(bin == b);
        if (threadIdx.x == 0 && c) atomicAdd(&counts->bin_count[b], c);
    }
    // block maximum, then one atomic per block (every block updates the same word)
    __shared__ int32_t warp_max[kThreads / 32];
    deg = __reduce_max_sync(0xffffffffu, deg);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = deg;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) deg = max(deg, warp_max[w]);
        if (deg > 0) atomicMax(&counts->max_degree, deg);
    }
}

// col_idx, the GCN weight and (unless the duplicate removal already wrote it) perm of every slot
__global__ void __launch_bounds__(kThreads)
finalize_entries(const u64* __restrict__ keys, const int32_t* __restrict__ vals, int write_perm,
                 const BuildCounts* __restrict__ counts, int src_bits, int val_bits, const float* __restrict__ dinv,
                 int32_t* __restrict__ col_idx, float* __restrict__ edge_w, int32_t* __restrict__ perm, int64_t m)
{
    const int64_t base = (int64_t)blockIdx.x * (kThreads * kKeyItems) + threadIdx.x;
    const int64_t nnz = counts->nnz;
    u64 word[kKeyItems];
#pragma unroll
    for (int j = 0; j < kKeyItems; ++j) {
        const int64_t k = base + j * kThreads;
        word[j] = (k < m && k < nnz) ? __ldcs(keys + k) : 0ull;
    }
    float ws[kKeyItems], wd[kKeyItems];
#pragma unroll
    for (int j = 0; j < kKeyItems; ++j) {
        const u64 key = word[j] >> val_bits;
        ws[j] = __ldg(dinv + (int32_t)(key & ((1ull << src_bits) - 1ull)));       // 0 for the padding words: in range
        wd[j] = __ldg(dinv + (int32_t)(key >> src_bits));
    }
#pragma unroll
    for (int j = 0; j < kKeyItems; ++j) {
        const int64_t k = base + j * kThreads;
        if (k >= m || k >= nnz) continue;
        const u64 key = word[j] >> val_bits;
        __stcs(col_idx + k, (int32_t)(key & ((1ull << src_bits) - 1ull)));
        __stcs(edge_w + k, ws[j] * wd[j]);
        if (write_perm) __stcs(perm + k, vals ? __ldcs(vals + k) : (int32_t)(word[j] & ((1ull << val_bits) - 1ull)) - 1);
    }
}

// Hub rows are cut twice: at the boundaries of source ranges of `range_rows` vertex ids (a row's sources are
// ascending, so a range is a contiguous piece of the row) and then into segments of at most GNNFD_HUB_SEGMENT
// entries.  Segments are scheduled range by range (all hub rows' pieces of source range 0, then range 1, ...),
// so the hub rows that are gathered at the same time read the same narrow band of x: a source that several
// hub rows share is fetched from HBM once per sweep instead of once per row.  A segment keeps a second number,
// its slot: slots count a row's segments in ascending source order, row after row, and index the partial
// results, so that the per-row reductions run over a contiguous, ordered slot range.

__device__ __forceinline__ int32_t lower_bound_col(const int32_t* __restrict__ col, int32_t lo, int32_t hi, int64_t bound)
{
    while (lo < hi) {
        const int32_t mid = lo + ((hi - lo) >> 1);
        if ((int64_t)col[mid] < bound) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// per hub row and source range: the number of segments (range-major: count[r * hub_cap + i]) and per hub row
// the total; entries past the last hub row are 0 so that the scans yield the totals
__global__ void __launch_bounds__(kThreads)
hub_segment_counts(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                   const int32_t* __restrict__ row_order, int64_t n, const BuildCounts* __restrict__ counts, int64_t hub_cap,
                   int32_t n_ranges, int64_t range_rows, int32_t* __restrict__ range_count, int32_t* __restrict__ seg_count)
{
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i > hub_cap) return;
    const int32_t n_hub = counts->bin_count[4];
    int32_t total = 0;
    if (i < n_hub) {
        const int32_t v = row_order[n - n_hub + i];
        int32_t pos = row_ptr[v];
        const int32_t e = row_ptr[v + 1];
        for (int32_t r = 0; r < n_ranges; ++r) {
            const int32_t nxt = r == n_ranges - 1 ? e : lower_bound_col(col_idx, pos, e, (int64_t)(r + 1) * range_rows);
            const int32_t c = (nxt - pos + kHubSegment - 1) / kHubSegment;
            range_count[(int64_t)r * hub_cap + i] = c;
            total += c;
            pos = nxt;
        }
    } else if (i < hub_cap) {
        for (int32_t r = 0; r < n_ranges; ++r) range_count[(int64_t)r * hub_cap + i] = 0;
    }
    seg_count[i] = total;
    if (i == 0) range_count[(int64_t)n_ranges * hub_cap] = 0;
}

// range_first: exclusive scan of range_count (the schedule position of a row's first segment in a range);
// hub_seg_ptr: exclusive scan of seg_count (the row's first slot)
__global__ void __launch_bounds__(kThreads)
fill_segments(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx, const int32_t* __restrict__ row_order,
              int64_t n, BuildCounts* __restrict__ counts, const int32_t* __restrict__ hub_seg_ptr,
              const int32_t* __restrict__ range_first, int64_t hub_cap, int32_t n_ranges, int64_t range_rows,
              int32_t* __restrict__ seg_row, int32_t* __restrict__ seg_begin, int32_t* __restrict__ seg_end,
              int32_t* __restrict__ seg_slot)
{
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int32_t n_hub = counts->bin_count[4];
    if (i == 0) counts->n_segments = hub_seg_ptr[n_hub];
    if (i >= hub_cap || i >= n_hub) return;
    const int32_t v = row_order[n - n_hub + i];
    int32_t pos = row_ptr[v];
    const int32_t e = row_ptr[v + 1];
    int32_t slot = hub_seg_ptr[i];
    for (int32_t r = 0; r < n_ranges; ++r) {
        const int32_t nxt = r == n_ranges - 1 ? e : lower_bound_col(col_idx, pos, e, (int64_t)(r + 1) * range_rows);
        int32_t p = range_first[(int64_t)r * hub_cap + i];
        for (int32_t x0 = pos; x0 < nxt; x0 += kHubSegment, ++p, ++slot) {
            seg_row[p] = v;
            seg_begin[p] = x0;
            seg_end[p] = min(x0 + kHubSegment, nxt);
            seg_slot[p] = slot;
        }
        pos = nxt;
    }
}

// ------------------------------------------------------------------ host side

struct BuildLayout {
    int64_t m;             // candidate edges
    int64_t n_tiles;       // sort tiles of the edge sort
    int64_t row_tiles;     // sort tiles of the row (degree class) sort
    int64_t hub_cap;       // upper bound on hub rows
    int64_t seg_cap;       // upper bound on hub segments
    int src_bits, key_bits, passes, digit_bits;
    int first_bit;         // lowest key bit the sort looks at (0; src_bits when rows keep their input order)
    int n_ranges;          // source ranges the hub rows are cut at (1: no cut)
    int64_t range_rows;    // vertex ids per source range
    int val_bits;          // > 0: keys and values share one 64-bit word (key << val_bits | value + 1)
};

static int make_layout(int64_t n, int64_t e, uint32_t flags, BuildLayout* L)
{
    if (n <= 0 || e < 0) return GNNFD_INVALID_ARG;
    if (flags & ~(uint32_t)(GNNFD_CSR_ADD_SELF_LOOPS | GNNFD_CSR_DEDUP | GNNFD_CSR_SYMMETRIZE | GNNFD_CSR_INPUT_ORDER))
        return GNNFD_INVALID_ARG;
    // duplicates are found as neighbours of the (dst, src) order, which the input-order build does not establish
    if ((flags & GNNFD_CSR_INPUT_ORDER) && (flags & GNNFD_CSR_DEDUP)) return GNNFD_INVALID_ARG;
    const int64_t limit = (int64_t(1) << 31) - 1;
    if (n > limit || e > limit) return GNNFD_TOO_LARGE;
    int64_t m = e;
    if (flags & GNNFD_CSR_SYMMETRIZE) m += e;
    if (flags & GNNFD_CSR_ADD_SELF_LOOPS) m += n;
    if (m > limit) return GNNFD_TOO_LARGE;
    L->m = m;
    L->n_tiles = (m + kSortTile - 1) / kSortTile;
    if (L->n_tiles == 0) L->n_tiles = 1;
    L->row_tiles = (n + kSortTile - 1) / kSortTile;
    L->hub_cap = m / (GNNFD_HUB_DEGREE + 1) + 1;
    // source ranges of GNNFD_HUB_RANGE_ROWS vertices, at most 64 of them (narrower ranges would keep a band of x
    // resident in L2, but on the RMAT workload the extra, shorter segments cost more than the saved traffic: 32
    // ranges cut the gather's DRAM bytes by 27 % and made it 13 % slower, 4 ranges are 3 % faster than none); a row
    // whose sources are not ascending (input-order build) cannot be cut by range
    L->range_rows = GNNFD_HUB_RANGE_ROWS;
    while ((n + L->range_rows - 1) / L->range_rows > 64) L->range_rows <<= 1;
    L->n_ranges = (flags & GNNFD_CSR_INPUT_ORDER) ? 1 : (int)((n + L->range_rows - 1) / L->range_rows);
    L->seg_cap = m / kHubSegment + L->hub_cap * L->n_ranges + 1;
    int bits = 1;
    while ((int64_t(1) << bits) < n) ++bits;
    int dst_bits = 1;
    while ((int64_t(1) << dst_bits) < n + 1) ++dst_bits;      // destination n marks dropped candidates
    L->src_bits = bits;
    L->key_bits = bits + dst_bits;
    // Rows in input order: the stable sort looks at the destination bits only, so entries of a row stay in the
    // order of their candidate numbers (input edges, then reverses, then the added loop).
    L->first_bit = (flags & GNNFD_CSR_INPUT_ORDER) ? bits : 0;
    const int sort_bits = L->key_bits - L->first_bit;
    L->passes = (sort_bits + kMaxDigitBits - 1) / kMaxDigitBits;
    L->digit_bits = (sort_bits + L->passes - 1) / L->passes;
    int vb = 1;
    while ((int64_t(1) << vb) < m + 2) ++vb;                  // values -1 .. m-1 stored as 0 .. m
    L->val_bits = L->key_bits + vb <= 64 ? vb : 0;
    return GNNFD_OK;
}

// upper bound on the hub segments of any graph with these sizes (what the persistent buffer reserves)
int64_t segment_capacity(int64_t n, int64_t e, uint32_t flags)
{
    BuildLayout L;
    return make_layout(n, e, flags, &L) == GNNFD_OK ? L.seg_cap : -1;
}

struct PersistentPtrs {
    int32_t *row_ptr, *col_idx, *perm, *row_order, *seg_row, *seg_begin, *seg_end, *seg_slot, *hub_seg_ptr;
    float *edge_w, *dinv, *rdeg;
    BuildCounts* counts;
};

static void carve_persistent(Carver& c, int64_t n, const BuildLayout& L, PersistentPtrs* p)
{
    const size_t cap = (size_t)(L.m > 0 ? L.m : 1);
    p->row_ptr = c.take<int32_t>((size_t)n + 1);
    p->col_idx = c.take<int32_t>(cap);
    p->perm = c.take<int32_t>(cap);
    p->edge_w = c.take<float>(cap);
    p->dinv = c.take<float>((size_t)n);
    p->rdeg = c.take<float>((size_t)n);
    p->row_order = c.take<int32_t>((size_t)n);
    p->seg_row = c.take<int32_t>((size_t)L.seg_cap);
    p->seg_begin = c.take<int32_t>((size_t)L.seg_cap);
    p->seg_end = c.take<int32_t>((size_t)L.seg_cap);
    p->seg_slot = c.take<int32_t>((size_t)L.seg_cap);
    p->hub_seg_ptr = c.take<int32_t>((size_t)L.hub_cap + 1);
    p->counts = c.take<BuildCounts>(1);
}

struct ScratchPtrs {
    u64 *keys_a, *keys_b;
    int32_t *vals_a, *vals_b, *hist, *flags, *scan_temp;
};

static size_t flag_ints(int64_t n, const BuildLayout& L)
{
    // one count per tile of the duplicate removal, a 64-bit dump for the row sort's keys (2 ints per row),
    // hub segment counts (per source range and hub row, then per hub row)
    size_t a = (size_t)L.m / kUniqueTile + 2, b = 2 * (size_t)n + 2, c = (size_t)L.hub_cap * (L.n_ranges + 1) + 4;
    size_t r = a > b ? a : b;
    return (r > c ? r : c) + 1;
}

static void carve_scratch(Carver& c, int64_t n, const BuildLayout& L, ScratchPtrs* p)
{
    const size_t cap = (size_t)(L.m > n ? L.m : n);      // the row sort reuses the edge sort's buffers
    p->keys_a = c.take<u64>(cap);
    p->keys_b = c.take<u64>(cap);
    // when the values travel inside the key words only the row sort needs value buffers
    const size_t val_cap = L.val_bits > 0 ? (size_t)n : cap;
    p->vals_a = c.take<int32_t>(val_cap);
    p->vals_b = c.take<int32_t>(val_cap);
    const size_t hist_ints = (size_t)kRadix * (size_t)(L.n_tiles > L.row_tiles ? L.n_tiles : L.row_tiles);
    p->hist = c.take<int32_t>(hist_ints);
    const size_t fl = flag_ints(n, L);
    p->flags = c.take<int32_t>(fl);
    const size_t biggest = hist_ints > fl ? hist_ints : fl;
    p->scan_temp = c.take<int32_t>(scan_temp_ints(biggest));
}

}  // namespace gnnfd

extern "C" {

int gnnfd_csr_workspace_bytes(int64_t n, int64_t e, uint32_t flags, size_t* persistent_bytes, size_t* scratch_bytes)
{
    using namespace gnnfd;
    BuildLayout L;
    int rc = make_layout(n, e, flags, &L);
    if (rc) return rc;
    if (persistent_bytes) {
        Carver c(nullptr, ~size_t(0));
        PersistentPtrs p;
        carve_persistent(c, n, L, &p);
        *persistent_bytes = c.off;
    }
    if (scratch_bytes) {
        Carver c(nullptr, ~size_t(0));
        ScratchPtrs s;
        carve_scratch(c, n, L, &s);
        *scratch_bytes = c.off;
    }
    return GNNFD_OK;
}

int gnnfd_build_csr(int64_t n, int64_t e, const void* d_src, const void* d_dst, gnnfd_itype_t itype, uint32_t flags,
                    void* d_persistent, size_t persistent_bytes, void* d_scratch, size_t scratch_bytes, void* stream,
                    gnnfd_csr_t** out)
{
    using namespace gnnfd;
    if (!out) return GNNFD_INVALID_ARG;
    *out = nullptr;
    BuildLayout L;
    int rc = make_layout(n, e, flags, &L);
    if (rc) return rc;
    if (itype != GNNFD_I32 && itype != GNNFD_I64) return GNNFD_UNSUPPORTED;
    if ((e > 0 && (!d_src || !d_dst)) || !d_persistent || !d_scratch) return GNNFD_INVALID_ARG;
    if (((uintptr_t)d_persistent | (uintptr_t)d_scratch) & 255u) return GNNFD_INVALID_ARG;

    Carver pc(d_persistent, persistent_bytes), sc(d_scratch, scratch_bytes);
    PersistentPtrs P;
    ScratchPtrs S;
    carve_persistent(pc, n, L, &P);
    carve_scratch(sc, n, L, &S);
    if (!pc.ok || !sc.ok) return GNNFD_WORKSPACE_TOO_SMALL;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t m = L.m;
    GNNFD_CUDA_CHECK(cudaMemsetAsync(P.counts, 0, sizeof(BuildCounts), s));

    BuildCounts host_counts;
    std::memset(&host_counts, 0, sizeof(host_counts));
    u64* keys = S.keys_a;
    u64* keys_alt = S.keys_b;
    int32_t* vals = S.vals_a;
    int32_t* vals_alt = S.vals_b;

    const bool dedup = (flags & GNNFD_CSR_DEDUP) != 0;
    const int vb = L.val_bits;
    const bool packed = vb > 0;                     // values ride in the low bits of the keys
    const size_t scatter_smem = packed ? offsetof(ScatterSmem, vals) : sizeof(ScatterSmem);
    GNNFD_CUDA_CHECK(cudaFuncSetAttribute(radix_scatter<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(ScatterSmem)));
    GNNFD_CUDA_CHECK(cudaFuncSetAttribute(radix_scatter<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)offsetof(ScatterSmem, vals)));
    if (m > 0) {
        int32_t* key_vals = packed ? nullptr : vals;
        if (itype == GNNFD_I32)
            GNNFD_LAUNCH("make_keys", s, make_keys<int32_t>, blocks_for(m, kThreads * kKeyItems), kThreads, 0,
                         static_cast<const int32_t*>(d_src), static_cast<const int32_t*>(d_dst), n, e, m, flags, L.src_bits,
                         vb, keys, key_vals, P.counts);
        else
            GNNFD_LAUNCH("make_keys", s, make_keys<long long>, blocks_for(m, kThreads * kKeyItems), kThreads, 0,
                         static_cast<const long long*>(d_src), static_cast<const long long*>(d_dst), n, e, m, flags,
                         L.src_bits, vb, keys, key_vals, P.counts);
        const int mask = (1 << L.digit_bits) - 1;
        for (int pass = 0; pass < L.passes; ++pass) {
            const int shift = L.first_bit + pass * L.digit_bits + vb;
            GNNFD_LAUNCH("radix_histogram", s, radix_histogram, (unsigned)L.n_tiles, kThreads, 0, keys, m, shift, mask,
                         L.n_tiles, S.hist);
            rc = exclusive_scan_i32(S.hist, S.hist, (size_t)kRadix * (size_t)L.n_tiles, S.scan_temp, s);
            if (rc) return rc;
            if (packed)
                GNNFD_LAUNCH("radix_scatter", s, radix_scatter<false>, (unsigned)L.n_tiles, kScatterThreads, scatter_smem, keys,
                             (const int32_t*)nullptr, keys_alt, (int32_t*)nullptr, m, shift, mask, L.n_tiles, S.hist);
            else
                GNNFD_LAUNCH("radix_scatter", s, radix_scatter<true>, (unsigned)L.n_tiles, kScatterThreads, scatter_smem, keys,
                             (const int32_t*)vals, keys_alt, vals_alt, m, shift, mask, L.n_tiles, S.hist);
            u64* tk = keys; keys = keys_alt; keys_alt = tk;
            int32_t* tv = vals; vals = vals_alt; vals_alt = tv;
        }
        if (dedup) {
            const unsigned unique_tiles = blocks_for(m, kUniqueTile);
            int32_t* tile_first = S.flags;
            GNNFD_LAUNCH("unique_tile_counts", s, unique_tile_counts, unique_tiles, kThreads, 0, keys, vb, P.counts, tile_first);
            rc = exclusive_scan_i32(tile_first, tile_first, (size_t)unique_tiles, S.scan_temp, s);
            if (rc) return rc;
            GNNFD_LAUNCH("compact_unique", s, compact_unique, unique_tiles, kThreads, 0, keys,
                         packed ? (const int32_t*)nullptr : (const int32_t*)vals, (const int32_t*)tile_first, m, vb, keys_alt,
                         P.perm, P.counts);
            u64* tk = keys; keys = keys_alt; keys_alt = tk;
        }
    }
    GNNFD_LAUNCH("row_pointers", s, row_pointers, blocks_for((size_t)n + 1, kThreads), kThreads, 0, keys, P.counts, n,
                 L.src_bits, vb, dedup ? 1 : 0, P.row_ptr);
    // keys_alt / vals_alt are free from here on: they take the (degree class, row) pairs
    GNNFD_LAUNCH("degrees_and_classes", s, degrees_and_classes, blocks_for((size_t)n, kThreads), kThreads, 0, P.row_ptr, n,
                 P.dinv, P.rdeg, keys_alt, vals_alt, P.counts);
    if (m > 0)
        GNNFD_LAUNCH("finalize_entries", s, finalize_entries, blocks_for(m, kThreads * kKeyItems), kThreads, 0, keys,
                     packed ? (const int32_t*)nullptr : (const int32_t*)vals, dedup ? 0 : 1, P.counts, L.src_bits, vb,
                     P.dinv, P.col_idx, P.edge_w, P.perm, m);
    // row_order = rows sorted by degree class, ascending row id inside a class: one stable radix pass
    {
        GNNFD_LAUNCH("radix_histogram", s, radix_histogram, (unsigned)L.row_tiles, kThreads, 0, keys_alt, n, 32, kRadix - 1,
                     L.row_tiles, S.hist);
        rc = exclusive_scan_i32(S.hist, S.hist, (size_t)kRadix * (size_t)L.row_tiles, S.scan_temp, s);
        if (rc) return rc;
        GNNFD_LAUNCH("radix_scatter", s, radix_scatter<true>, (unsigned)L.row_tiles, kScatterThreads, sizeof(ScatterSmem), keys_alt,
                     vals_alt, reinterpret_cast<u64*>(S.flags), P.row_order, n, 32, kRadix - 1, L.row_tiles, S.hist);
    }
    // the flag buffer is free again: segment counts per (source range, hub row), then per hub row
    int32_t* range_count = S.flags;
    int32_t* seg_count = S.flags + (size_t)L.hub_cap * L.n_ranges + 1;
    GNNFD_LAUNCH("hub_segment_counts", s, hub_segment_counts, blocks_for((size_t)L.hub_cap + 1, kThreads), kThreads, 0,
                 P.row_ptr, P.col_idx, P.row_order, n, P.counts, L.hub_cap, L.n_ranges, L.range_rows, range_count, seg_count);
    rc = exclusive_scan_i32(seg_count, P.hub_seg_ptr, (size_t)L.hub_cap + 1, S.scan_temp, s);
    if (rc) return rc;
    rc = exclusive_scan_i32(range_count, range_count, (size_t)L.hub_cap * L.n_ranges + 1, S.scan_temp, s);
    if (rc) return rc;
    GNNFD_LAUNCH("fill_segments", s, fill_segments, blocks_for((size_t)L.hub_cap, kThreads), kThreads, 0, P.row_ptr, P.col_idx,
                 P.row_order, n, P.counts, P.hub_seg_ptr, range_count, L.hub_cap, L.n_ranges, L.range_rows, P.seg_row,
                 P.seg_begin, P.seg_end, P.seg_slot);
    GNNFD_CUDA_CHECK(cudaGetLastError());
    GNNFD_CUDA_CHECK(cudaMemcpyAsync(&host_counts, P.counts, sizeof(BuildCounts), cudaMemcpyDeviceToHost, s));
    GNNFD_CUDA_CHECK(cudaStreamSynchronize(s));

    if (host_counts.bad_index > 0) return GNNFD_BAD_INDEX;

    gnnfd_csr_t* h = new (std::nothrow) gnnfd_csr_t;
    if (!h) return GNNFD_INVALID_ARG;
    h->n = n;
    h->nnz = host_counts.nnz;
    h->max_degree = host_counts.max_degree;
    int64_t start = 0;
    for (int b = 0; b < kNumBins; ++b) {
        h->bin_count[b] = host_counts.bin_count[b];
        h->bin_start[b] = start;
        start += host_counts.bin_count[b];
    }
    h->n_segments = host_counts.n_segments;
    h->row_ptr = P.row_ptr;
    h->col_idx = P.col_idx;
    h->perm = P.perm;
    h->dinv = P.dinv;
    h->rdeg = P.rdeg;
    h->edge_w = P.edge_w;
    h->row_order = P.row_order;
    h->seg_row = P.seg_row;
    h->seg_begin = P.seg_begin;
    h->seg_end = P.seg_end;
    h->seg_slot = P.seg_slot;
    h->hub_seg_ptr = P.hub_seg_ptr;
    *out = h;
    return GNNFD_OK;
}

}  // extern "C"
