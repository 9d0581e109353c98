// Launch schedule shared by the gather kernels: how a sweep over one column tile of one chunk is cut
// into block ranges (hub segments first, then the degree classes from high to low).
#pragma once

#include "common.cuh"

namespace gnnfd {

#ifndef GNNFD_GATHER_BLOCK
#define GNNFD_GATHER_BLOCK 256
#endif
constexpr int kBlock = GNNFD_GATHER_BLOCK;      // threads per block of the gather kernels
constexpr int kMaxRanges = 5;
constexpr int kMaxGridY = 65535;               // chunks one launch of a gather kernel covers (grid y)

struct Range {
    int32_t first_block;   // first block (within one column tile of one sweep) of this range
    int32_t item_begin;    // offset into row_order (rows) or 0 (hub segments)
    int32_t item_count;
    int32_t ep_log2;       // log2 of the edge-parallel groups per row
    int32_t hub;           // 1: items are hub segments writing partial results
};

inline int ilog2(int x) { int l = 0; while ((1 << l) < x) ++l; return l; }

// Edge-parallel groups per row for a degree class, limited by the lanes a row may use.  Rows of up to 32
// entries get one group, rows of up to 128 four: a short row is bound by its chain of dependent loads
// (row number -> row pointer -> indices -> features), so more rows in flight per block beat more lanes per
// row (config 2 at 64 columns 0.128 -> 0.115 ms, GAT on config 3 0.189 -> 0.167 ms, config 5 at 64 columns
// 1.81 -> 1.62 ms against 4 and 8 groups).
inline int ep_for_bin(int bin, int lpr)
{
#ifndef GNNFD_EP_BIN1
#define GNNFD_EP_BIN1 1
#endif
#ifndef GNNFD_EP_BIN2
#define GNNFD_EP_BIN2 4
#endif
#ifndef GNNFD_EP_BIN3
#define GNNFD_EP_BIN3 32
#endif
    const int want[kNumBins] = {1, GNNFD_EP_BIN1, GNNFD_EP_BIN2, GNNFD_EP_BIN3, 32};
    const int cap = 32 / lpr;
    return want[bin] < cap ? want[bin] : cap;
}

// Fills ranges for `lpr` lanes per row; returns the blocks of one column tile of one sweep.
inline int64_t plan_ranges(const gnnfd_csr_t* csr, int lpr, Range* range, int32_t* n_ranges)
{
    int nr = 0;
    int64_t blocks = 0;
    if (csr->n_segments > 0) {
        const int ep = ep_for_bin(4, lpr);
        const int rows_per_block = kBlock / (lpr * ep);
        range[nr++] = Range{(int32_t)blocks, 0, (int32_t)csr->n_segments, ilog2(ep), 1};
        blocks += (csr->n_segments + rows_per_block - 1) / rows_per_block;
    }
    for (int bin = 3; bin >= 0; --bin) {
        if (csr->bin_count[bin] == 0) continue;
        const int ep = ep_for_bin(bin, lpr);
        const int rows_per_block = kBlock / (lpr * ep);
        range[nr++] = Range{(int32_t)blocks, (int32_t)csr->bin_start[bin], (int32_t)csr->bin_count[bin], ilog2(ep), 0};
        blocks += (csr->bin_count[bin] + rows_per_block - 1) / rows_per_block;
    }
    *n_ranges = nr;
    return blocks;
}

}  // namespace gnnfd
