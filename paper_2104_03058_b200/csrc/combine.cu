// Combination ahead of aggregation (Section III of the paper runs the dense transform first, so that
// the aggregation works on the narrower transformed features): z[n, f_out] = x[n, f_in] * W, W given
// transposed as w_t[f_out, f_in].
//
// This is a dense contraction, so it runs on the tensor cores: tcgen05.mma with tf32 operands (fp32
// inputs) or bf16 operands (bf16 inputs) read from shared memory, fp32 accumulation in tensor memory.  With f_out of 8 - 256 the product is bound
// by streaming x from HBM once (f_in * 4 bytes per row against 2 * f_in * f_out flops), which the
// fp32 ALUs could not keep up with.
//
// One block per 128 rows of x and per tile of up to 256 output columns.  Roles inside a block of four
// warps: one lane of warp 0 issues the TMA loads (x tile 128 rows x 128 bytes, w_t tile N rows x 128 bytes,
// both with the 128-byte swizzle) into a ring of stages, one lane of warp 1 issues four 32-byte-deep MMAs per
// stage and commits them to the stage's "empty" barrier, warp 2 owns the tensor-memory allocation;
// after the last commit all four warps read the accumulator (warp w owns lanes 32 w .. 32 w + 31,
// i.e. one output row per thread) and store it.  Rows past n and columns past f_in are filled with
// zeros by the TMA unit, so ragged sizes need no special tiles.
//
// fp32-faithful mode (fp32 inputs only): a tf32 operand keeps 10 mantissa bits, which is 50 x coarser than the
// fp32 arithmetic a framework runs the Combination in.  In this mode every operand value v is used as the pair
// (hi, lo) with hi = v cut to tf32 (the tensor core does that cut itself when it reads v) and lo = v - hi (exact
// in fp32, then cut to tf32 by the read), and the product is accumulated as x_lo w_hi + x_hi w_lo + x_hi w_hi:
// three MMAs per K slice.  The extra warps of the block compute the lo tiles in shared memory (same swizzled
// layout, element by element) as soon as a stage has landed.  What is dropped is x_lo w_lo (below 2^-20 of the
// product) and the low bits of lo (below 2^-21).
//
// GAT scores from the epilogue: a thread holds a whole row of the output tile in registers, so the two
// attention scores per head (dot products of the head's columns with a_src / a_dst) are formed there and z
// is not read again by a separate scores pass.
//
// Every wait on a barrier is bounded: when a limit runs out the block records an error in the
// caller's status word, drains the copies it has in flight (again bounded), frees its tensor memory
// and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace gnnfd {

constexpr int kCombineThreads = 128;
constexpr int kSplitThreads = 256;          // fp32-faithful mode: warps 2..7 compute the lo tiles
constexpr int kTileM = 128;                 // rows of x per block (the MMA's M)
constexpr int kTileKBytes = 128;            // bytes per stage row: one 128-byte swizzle span (32 floats or 64 bf16)
constexpr int kMmaKBytes = 32;              // depth of one MMA: K = 8 for tf32, K = 16 for bf16
constexpr int kMaxTileN = 256;
constexpr uint64_t kWaitNs = 1000000000ull; // one second on one barrier before the block gives up
constexpr int kSmemBudget = 100 * 1024;     // per block, so that two blocks share an SM
constexpr int kSmemBudgetSplit = 108 * 1024; // fp32-faithful mode (hi and lo tiles per stage): still two blocks per SM
constexpr int kSmemBudgetMax = 200 * 1024;  // fp32-faithful mode with wide tiles: one block per SM
constexpr int kMaxStages = 6;

struct CombineArgs {
    void* z;
    int64_t ldz;
    int32_t n, f_in, f_out, tile_n, stages, tmem_cols, z_bf16;
    int32_t acc_cols, n_main;   // tensor-memory columns per accumulator; accumulators the K blocks rotate over
    int32_t xlo_col;            // first tensor-memory column of the x_lo ring (32 columns per stage), XT kernels only
    int32_t* status;        // set to 1 when a wait ran out (may be null)
    // GAT scores formed in the epilogue (all null / 0 when not wanted): a_src / a_dst [heads * dim] over the
    // output columns, s_src / s_dst [n, heads]
    const float* a_src;
    const float* a_dst;
    float* s_src;
    float* s_dst;
    int32_t heads, dim;
    uint64_t wait_ns;       // limit of one barrier wait
    int32_t skip_k_block;   // fault drill: the producer leaves this K block's loads out (-1: none)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint64_t now_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool mbar_test(uint32_t addr, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    return done != 0;
}

// true once the phase with the given parity has completed; gives up after limit_ns
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint64_t limit_ns)
{
    const uint32_t addr = smem_u32(bar);
    if (mbar_test(addr, parity)) return true;
    const uint64_t t0 = now_ns();
    while (!mbar_test(addr, parity))
        if (now_ns() - t0 > limit_ns) return false;
    return true;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int32_t x, int32_t y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        :
        : "r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

// Shared-memory operand descriptor of a K-major tile whose rows are 128 bytes, stored with the 128-byte
// swizzle: groups of 8 rows are 1024 bytes apart; descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr)
{
    uint64_t d = (uint64_t)((smem_addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;                    // leading-dimension offset: not used by swizzled K-major tiles
    d |= (uint64_t)(1024 >> 4) << 32;          // stride between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}

// Instruction descriptor: fp32 accumulator, A and B of one type (format 2 = tf32, 1 = bf16), both
// K-major, M = 128, N = tile_n.
template <bool BF16>
__device__ __forceinline__ uint32_t instr_desc(int tile_n)
{
    constexpr uint32_t fmt = BF16 ? 1u : 2u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(tile_n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

template <bool BF16>
__device__ __forceinline__ void mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    if constexpr (BF16) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
            "}"
            :
            : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t"
            "}"
            :
            : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}

// tf32 MMA whose A operand (128 rows x 8 K elements, one 32-bit column per element, row = lane) lies in tensor memory
__device__ __forceinline__ void mma_a_tmem(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t"
        "}"
        :
        : "r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 32 consecutive columns of the calling thread's lane (a warp covers 32 lanes)
__device__ __forceinline__ void tmem_store_32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        :
        : "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// arrives on the barrier once every MMA issued so far by this thread has finished
__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// Adds one output value to the running attention scores of its row; at the last column of a head the two
// scores are written and the sums start again.  `d` is the column's position inside its head.
struct ScoreState {
    float ss, sd;
    int d, head;
};

__device__ __forceinline__ void score_step(ScoreState& st, float val, int col, const CombineArgs& a, int row, const float* a_src_s,
                                           const float* a_dst_s, int col0)
{
    st.ss = fmaf(a_src_s[col - col0], val, st.ss);
    st.sd = fmaf(a_dst_s[col - col0], val, st.sd);
    if (++st.d == a.dim) {
        a.s_src[(int64_t)row * a.heads + st.head] = st.ss;
        a.s_dst[(int64_t)row * a.heads + st.head] = st.sd;
        st.ss = st.sd = 0.f;
        st.d = 0;
        ++st.head;
    }
}

// SPLIT: fp32-faithful mode (fp32 operands as tf32 hi + lo pairs, three MMAs per K slice); launched with
// kSplitThreads threads, of which warps 2.. compute the lo tiles.
// XT (with SPLIT): the lo part of the x tile is kept in tensor memory and fed to the MMA as its A operand from
// there (warps 4 - 7 own one row each: they read it out of the swizzled stage, subtract the tf32 cut and store 32
// columns), so a stage holds only x, w and w_lo in shared memory and the ring is a stage deeper.
template <bool BF16, bool SPLIT, bool XT = false>
__global__ void __launch_bounds__(SPLIT ? kSplitThreads : kCombineThreads)
combine_mma(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const CombineArgs a)
{
    static_assert(!(BF16 && SPLIT), "bf16 operands are used as they are");
    static_assert(!XT || SPLIT, "x_lo in tensor memory belongs to the fp32-faithful mode");
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], split_bar[kMaxStages], accum_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float a_src_s[kMaxTileN], a_dst_s[kMaxTileN];

    // the dynamic buffer is aligned to 1024 bytes by hand (the swizzle pattern repeats every 1024 bytes)
    unsigned char* tiles = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int kTileK = kTileKBytes / (BF16 ? 2 : 4);      // elements of K per stage
    constexpr int kSplitWarps = !SPLIT ? 0 : XT ? 4 : kSplitThreads / 32 - 2;
    const uint32_t a_bytes = kTileM * kTileKBytes;
    const uint32_t b_bytes = (uint32_t)a.tile_n * kTileKBytes;
    const uint32_t stage_bytes = a_bytes + b_bytes;            // what the TMA unit delivers per stage
    // the lo tiles follow the loaded ones (with XT only w's: x_lo lives in tensor memory)
    const uint32_t stage_pitch = !SPLIT ? stage_bytes : XT ? stage_bytes + b_bytes : 2 * stage_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = blockIdx.x * kTileM;
    const int col0 = blockIdx.y * a.tile_n;
    const int k_blocks = (a.f_in + kTileK - 1) / kTileK;
    const bool want_scores = a.s_src != nullptr;

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
            mbar_init(&split_bar[s], SPLIT ? kSplitWarps : 1);
        }
        mbar_init(&accum_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (want_scores)
        for (int c = threadIdx.x; c < a.tile_n; c += blockDim.x) {
            const bool in = col0 + c < a.f_out;
            a_src_s[c] = in ? a.a_src[col0 + c] : 0.f;
            a_dst_s[c] = in ? a.a_dst[col0 + c] : 0.f;
        }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"((uint32_t)a.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    int issued = 0;            // K blocks the producer lane has gone through (thread 0 only)
    if (warp == 0 && lane == 0) {
        // producer: fills stage kb % stages once the MMAs that read its previous contents have finished
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % a.stages;
            if (kb >= a.stages) ok = mbar_wait(&empty_bar[s], ((kb / a.stages) - 1) & 1, a.wait_ns);
            if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
            issued = kb + 1;
            if (kb == a.skip_k_block) continue;        // fault drill: nothing is issued for this block, so nothing of it is in flight
            unsigned char* stage = tiles + (size_t)s * stage_pitch;
            mbar_expect_tx(&full_bar[s], stage_bytes);
            tma_load_2d(stage, &map_x, &full_bar[s], kb * kTileK, row0);
            tma_load_2d(stage + a_bytes, &map_w, &full_bar[s], kb * kTileK, col0);
        }
        if (!ok) *(volatile int*)&abort_flag = 1;
    } else if (warp == 1 && lane == 0) {
        // MMA issuer
        const uint32_t idesc = instr_desc<BF16>(a.tile_n);
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % a.stages;
            ok = mbar_wait(SPLIT ? &split_bar[s] : &full_bar[s], (kb / a.stages) & 1, a.wait_ns);
            if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(tiles + (size_t)s * stage_pitch);
            const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
            for (int k = 0; k < kTileKBytes / kMmaKBytes; ++k) {
                // inside the 128-byte swizzle span the next K slice starts 32 bytes further on
                const uint64_t da = operand_desc(a_addr + k * kMmaKBytes);
                const uint64_t db = operand_desc(b_addr + k * kMmaKBytes);
                // K block kb adds into accumulator kb % n_main: every addition into an accumulator cuts the sum's
                // low bits, so spreading the additions keeps the chain (and its one-sided drift on same-sign data) short
                const uint32_t acc = tmem_base + (uint32_t)((kb % a.n_main) * a.acc_cols);
                const uint32_t carry = (kb >= a.n_main || k > 0) ? 1u : 0u;
                if constexpr (SPLIT) {
                    // the two small products go to an accumulator of their own (the last one), where they lose nothing
                    // against the large sum; the epilogue adds it once
                    const uint32_t acc_lo = tmem_base + (uint32_t)(a.n_main * a.acc_cols);
                    if constexpr (XT) {
                        const uint64_t db_lo = operand_desc(a_addr + stage_bytes + k * kMmaKBytes);
                        mma_a_tmem(acc_lo, tmem_base + (uint32_t)(a.xlo_col + s * 32 + k * 8), db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                        mma<BF16>(acc_lo, da, db_lo, idesc, 1u);
                    } else {
                        const uint64_t da_lo = operand_desc(a_addr + stage_bytes + k * kMmaKBytes);
                        const uint64_t db_lo = operand_desc(b_addr + stage_bytes + k * kMmaKBytes);
                        mma<BF16>(acc_lo, da_lo, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                        mma<BF16>(acc_lo, da, db_lo, idesc, 1u);
                    }
                    mma<BF16>(acc, da, db, idesc, carry);
                } else {
                    mma<BF16>(acc, da, db, idesc, carry);
                }
            }
            mma_commit(&empty_bar[s]);
        }
        if (ok) mma_commit(&accum_bar);
        else *(volatile int*)&abort_flag = 1;
    } else if (SPLIT && !XT && warp >= 2) {
        // lo tiles: element by element over the stage (the swizzle only permutes 16-byte pieces, so the lo tile
        // has the layout of the loaded one), then visible to the tensor core's reads, then one arrival per warp
        const int t = threadIdx.x - 64;
        const int n_vec = (int)(stage_bytes / 16);
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % a.stages;
            ok = mbar_wait(&full_bar[s], (kb / a.stages) & 1, a.wait_ns);
            ok = __all_sync(0xffffffffu, ok && !*(volatile int*)&abort_flag);
            if (!ok) break;
            const float4* hi = reinterpret_cast<const float4*>(tiles + (size_t)s * stage_pitch);
            float4* lo = reinterpret_cast<float4*>(tiles + (size_t)s * stage_pitch + stage_bytes);
#pragma unroll 4
            for (int i = t; i < n_vec; i += kSplitWarps * 32) {
                const float4 v = hi[i];
                float4 r;
                r.x = v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
                r.y = v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
                r.z = v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
                r.w = v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
                lo[i] = r;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&split_bar[s]);
        }
        if (!ok && lane == 0) *(volatile int*)&abort_flag = 1;
    } else if (SPLIT && XT && warp >= 4) {
        // x_lo into tensor memory: thread t of warps 4 - 7 owns row t of the tile (lane t of tensor memory).  The
        // stage stores row r's 16-byte piece c at position c ^ (r & 7) (128-byte swizzle); w_lo as above.
        const int t = threadIdx.x - 128;
        const int n_vec_w = (int)(b_bytes / 16);
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % a.stages;
            ok = mbar_wait(&full_bar[s], (kb / a.stages) & 1, a.wait_ns);
            ok = __all_sync(0xffffffffu, ok && !*(volatile int*)&abort_flag);
            if (!ok) break;
            const unsigned char* stage = tiles + (size_t)s * stage_pitch;
            uint32_t lo_bits[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 v = *reinterpret_cast<const float4*>(stage + (size_t)t * kTileKBytes + ((c ^ (t & 7)) << 4));
                lo_bits[4 * c + 0] = __float_as_uint(v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u));
                lo_bits[4 * c + 1] = __float_as_uint(v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u));
                lo_bits[4 * c + 2] = __float_as_uint(v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u));
                lo_bits[4 * c + 3] = __float_as_uint(v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u));
            }
            tmem_store_32(tmem_base + ((uint32_t)((warp - 4) * 32) << 16) + (uint32_t)(a.xlo_col + s * 32), lo_bits);
            const float4* hi = reinterpret_cast<const float4*>(stage + a_bytes);
            float4* lo = reinterpret_cast<float4*>(const_cast<unsigned char*>(stage) + stage_bytes);
            for (int i = t; i < n_vec_w; i += 128) {
                const float4 v = hi[i];
                float4 r;
                r.x = v.x - __uint_as_float(__float_as_uint(v.x) & 0xffffe000u);
                r.y = v.y - __uint_as_float(__float_as_uint(v.y) & 0xffffe000u);
                r.z = v.z - __uint_as_float(__float_as_uint(v.z) & 0xffffe000u);
                r.w = v.w - __uint_as_float(__float_as_uint(v.w) & 0xffffe000u);
                lo[i] = r;
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&split_bar[s]);
        }
        if (!ok && lane == 0) *(volatile int*)&abort_flag = 1;
    }
    __syncwarp();

    // epilogue (warps 0 - 3): thread t of warp w holds row 32 w + t of the tile
    bool ok = true;
    if (warp < 4) {
        ok = mbar_wait(&accum_bar, 0, a.wait_ns) && !*(volatile int*)&abort_flag;
        // on an abort the accumulator barrier never completes: all lanes of all warps agree through the flag
        ok = __all_sync(0xffffffffu, ok);
    }
    if (ok && warp < 4) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int row = row0 + warp * 32 + lane;
        const int col_end = min(a.f_out, col0 + a.tile_n);
        const int zsize = a.z_bf16 ? 2 : 4;
        const bool vec_ok = ((reinterpret_cast<uintptr_t>(a.z) | (uintptr_t)(a.ldz * zsize)) & 15u) == 0;
        ScoreState st{0.f, 0.f, 0, 0};
        if (want_scores) { st.d = col0 % a.dim; st.head = col0 / a.dim; }     // tiles start on head boundaries (host check)
        for (int c = 0; c < a.tile_n; c += 32) {
            uint32_t r[32];
            const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c;
            tmem_load_32(lane_base, r);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            // the other accumulators that received K blocks, then (fp32-faithful mode) the small products
            const int used = k_blocks < a.n_main ? k_blocks : a.n_main;
            for (int j = 1; j < used + (SPLIT ? 1 : 0); ++j) {
                uint32_t t[32];
                tmem_load_32(lane_base + (uint32_t)((j < used ? j : a.n_main) * a.acc_cols), t);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(t[i]));
            }
            if (row >= a.n) continue;
            if (a.z_bf16) {
                // the stored value is the fp32 sum rounded to bf16; scores are formed from what is stored
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__bfloat162float(__float2bfloat16_rn(__uint_as_float(r[j]))));
                __nv_bfloat16* zrow = static_cast<__nv_bfloat16*>(a.z) + (int64_t)row * a.ldz + col0 + c;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    const int col = col0 + c + j;
                    if (vec_ok && col + 8 <= col_end) {
                        uint4 v;
                        uint32_t* pv = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
                        for (int i = 0; i < 4; ++i) pv[i] = (r[j + 2 * i] >> 16) | (r[j + 2 * i + 1] & 0xffff0000u);
                        __stcs(reinterpret_cast<uint4*>(zrow + j), v);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (col + i < col_end) zrow[j + i] = __float2bfloat16_rn(__uint_as_float(r[j + i]));
                    }
                }
            } else {
                float* zrow = static_cast<float*>(a.z) + (int64_t)row * a.ldz + col0 + c;
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const int col = col0 + c + j;
                    if (vec_ok && col + 4 <= col_end) {
                        __stcs(reinterpret_cast<float4*>(zrow + j),
                               make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                           __uint_as_float(r[j + 3])));
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (col + i < col_end) zrow[j + i] = __uint_as_float(r[j + i]);
                    }
                }
            }
            if (want_scores) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + c + j < col_end) score_step(st, __uint_as_float(r[j]), col0 + c + j, a, row, a_src_s, a_dst_s, col0);
            }
        }
    } else if (threadIdx.x == 0) {
        if (a.status) atomicExch(a.status, 1);
        // This thread is the producer lane.  The copies of the last `stages` K blocks it issued may still be in
        // flight; they must land before the block's shared memory is given back, so it waits for each of them
        // once more (bounded).  A block left out by the fault drill has nothing in flight.
        const int first = issued > a.stages ? issued - a.stages : 0;
        for (int kb = first; kb < issued; ++kb)
            if (kb != a.skip_k_block) mbar_wait(&full_bar[kb % a.stages], (kb / a.stages) & 1, a.wait_ns);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// tensor map of a row-major matrix [rows, ld] of which `cols` columns are valid; box = box_rows x 128 bytes
static bool make_map(CUtensorMap* map, const void* base, bool bf16, int64_t rows, int64_t cols, int64_t ld, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const int esize = bf16 ? 2 : 4;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * esize};
    const cuuint32_t box[2] = {(cuuint32_t)(kTileKBytes / esize), (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims,
              strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace gnnfd

namespace gnnfd {

// One-shot settings of the fault drill (see gnnfd_debug_combine_fault): consumed by the next launch on this thread.
static thread_local uint64_t t_drill_wait_ns = 0;
static thread_local int32_t t_drill_skip = -1;

int combine_impl(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t, int64_t ldw,
                 int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int mode, const float* d_a_src,
                 const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst, int32_t* d_status,
                 cudaStream_t s)
{
    if (n <= 0 || !d_x || !d_w_t || !d_z || f_in <= 0 || f_out <= 0 || ldx < f_in || ldw < f_in || ldz < f_out)
        return GNNFD_INVALID_ARG;
    if ((xdt != GNNFD_F32 && xdt != GNNFD_BF16) || (zdt != GNNFD_F32 && zdt != GNNFD_BF16)) return GNNFD_UNSUPPORTED;
    if (mode != GNNFD_COMBINE_TF32 && mode != GNNFD_COMBINE_FP32) return GNNFD_INVALID_ARG;
    if (n > 0x7fffffffll - kTileM) return GNNFD_TOO_LARGE;
    const bool bf16 = xdt == GNNFD_BF16;
    const bool split = !bf16 && mode == GNNFD_COMBINE_FP32;     // bf16 products are exact already
    const int esize = bf16 ? 2 : 4;
    // the TMA unit wants 16-byte aligned bases and row pitches
    if (((uintptr_t)d_x | (uintptr_t)d_w_t) % 16 != 0 || (ldx * esize) % 16 != 0 || (ldw * esize) % 16 != 0)
        return GNNFD_UNSUPPORTED;
    const bool scores = d_s_src || d_s_dst || d_a_src || d_a_dst;
    if (scores && (!d_s_src || !d_s_dst || !d_a_src || !d_a_dst || heads <= 0 || dim <= 0 || (int64_t)heads * dim != f_out))
        return GNNFD_INVALID_ARG;

    CombineArgs a;
    a.z = d_z; a.ldz = ldz; a.n = (int32_t)n; a.f_in = f_in; a.f_out = f_out; a.status = d_status;
    a.z_bf16 = zdt == GNNFD_BF16;
    a.a_src = scores ? d_a_src : nullptr; a.a_dst = scores ? d_a_dst : nullptr;
    a.s_src = scores ? d_s_src : nullptr; a.s_dst = scores ? d_s_dst : nullptr;
    a.heads = heads; a.dim = dim;
    a.wait_ns = t_drill_wait_ns ? t_drill_wait_ns : kWaitNs;
    a.skip_k_block = t_drill_skip;
    t_drill_wait_ns = 0;
    t_drill_skip = -1;
    // output columns per block: all of them up to 256, rounded up to the MMA's N granularity of 16
    const int n_col_tiles = (f_out + kMaxTileN - 1) / kMaxTileN;
    const int per_tile = (f_out + n_col_tiles - 1) / n_col_tiles;
    a.tile_n = (per_tile + 15) / 16 * 16;
    // a head's scores are formed by one thread: with several column tiles every tile must hold whole heads
    if (scores && n_col_tiles > 1 && a.tile_n % dim != 0) return GNNFD_UNSUPPORTED;
    a.acc_cols = 32;
    while (a.acc_cols < a.tile_n) a.acc_cols <<= 1;
    // Shared memory per stage, blocks per SM, tensor memory.  Tensor memory has 512 columns per SM, shared by the
    // blocks resident there; a block takes its whole share: accumulators first and, in the fp32-faithful mode when
    // it fits, a ring of 32 columns per stage for the lo part of the x tile (`xt`).
    bool xt = false;
    int stage_bytes = 0;
    size_t smem = 0;
    a.xlo_col = 0;
    if (split) {
        const int stage_xt = (kTileM + 2 * a.tile_n) * kTileKBytes;          // x, w, w_lo
        for (int pass = 0; pass < 2 && !xt; ++pass) {
            const int budget = pass == 0 ? kSmemBudgetSplit : kSmemBudgetMax;
            const int tmem = pass == 0 ? 256 : 512;
            int stages = budget / stage_xt;
            if (stages > kMaxStages) stages = kMaxStages;
            const int n_acc = stages >= 2 ? (tmem - stages * 32) / a.acc_cols : 0;
            if (n_acc >= 2) {
                xt = true;
                stage_bytes = stage_xt;
                a.stages = stages;
                a.tmem_cols = tmem;
                a.n_main = n_acc - 1;
                a.xlo_col = tmem - stages * 32;
            }
        }
    }
    if (!xt) {
        stage_bytes = (kTileM + a.tile_n) * kTileKBytes * (split ? 2 : 1);
        int budget = split ? kSmemBudgetSplit : kSmemBudget;
        bool two_per_sm = true;
        if (budget / stage_bytes < 2) { budget = kSmemBudgetMax; two_per_sm = false; }      // wide tiles: one block per SM
        a.tmem_cols = two_per_sm ? 256 : 512;
        const int n_acc = a.tmem_cols / a.acc_cols;
        a.n_main = split ? n_acc - 1 : n_acc;
        if (a.n_main < 1) return GNNFD_UNSUPPORTED;
        a.stages = budget / stage_bytes;
        if (a.stages > kMaxStages) a.stages = kMaxStages;
        if (a.stages < 2) return GNNFD_UNSUPPORTED;
    }
    smem = (size_t)a.stages * stage_bytes + 1024;
    // a block that takes half of the SM's tensor memory must not meet a third one on its SM (it would sit in its
    // allocation until one of the others left); one that takes all of it must be alone: size the shared-memory
    // request accordingly
    if (a.tmem_cols == 256 && smem < 80 * 1024) smem = 80 * 1024;
    if (a.tmem_cols == 512 && smem < 120 * 1024) smem = 120 * 1024;

    CUtensorMap map_x, map_w;
    if (!make_map(&map_x, d_x, bf16, n, f_in, ldx, kTileM) || !make_map(&map_w, d_w_t, bf16, f_out, f_in, ldw, a.tile_n)) {
        set_cuda_error(cudaErrorInvalidValue);
        return GNNFD_CUDA_ERROR;
    }
    const dim3 grid((unsigned)((n + kTileM - 1) / kTileM), (unsigned)((f_out + a.tile_n - 1) / a.tile_n));
    if (bf16) {
        GNNFD_CUDA_CHECK(cudaFuncSetAttribute(combine_mma<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GNNFD_LAUNCH("combine_bf16", s, (combine_mma<true, false>), grid, kCombineThreads, smem, map_x, map_w, a);
    } else if (split && xt) {
        GNNFD_CUDA_CHECK(cudaFuncSetAttribute(combine_mma<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GNNFD_LAUNCH("combine_fp32_3xtf32", s, (combine_mma<false, true, true>), grid, kSplitThreads, smem, map_x, map_w, a);
    } else if (split) {
        GNNFD_CUDA_CHECK(cudaFuncSetAttribute(combine_mma<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GNNFD_LAUNCH("combine_fp32_3xtf32", s, (combine_mma<false, true>), grid, kSplitThreads, smem, map_x, map_w, a);
    } else {
        GNNFD_CUDA_CHECK(cudaFuncSetAttribute(combine_mma<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GNNFD_LAUNCH("combine_tf32", s, (combine_mma<false, false>), grid, kCombineThreads, smem, map_x, map_w, a);
    }
    GNNFD_CUDA_CHECK(cudaGetLastError());
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" {

int gnnfd_combine(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t, int64_t ldw,
                  int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int32_t* d_status, void* stream)
{
    return gnnfd::combine_impl(n, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, d_z, ldz, zdt, GNNFD_COMBINE_TF32, nullptr, nullptr,
                               0, 0, nullptr, nullptr, d_status, static_cast<cudaStream_t>(stream));
}

int gnnfd_combine_ex(int64_t n, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt, int32_t f_in, const void* d_w_t, int64_t ldw,
                     int32_t f_out, void* d_z, int64_t ldz, gnnfd_dtype_t zdt, int mode, const float* d_a_src,
                     const float* d_a_dst, int32_t heads, int32_t dim, float* d_s_src, float* d_s_dst, int32_t* d_status,
                     void* stream)
{
    return gnnfd::combine_impl(n, d_x, ldx, xdt, f_in, d_w_t, ldw, f_out, d_z, ldz, zdt, mode, d_a_src, d_a_dst, heads, dim,
                               d_s_src, d_s_dst, d_status, static_cast<cudaStream_t>(stream));
}

int gnnfd_debug_combine_fault(int64_t wait_ns, int32_t skip_k_block)
{
    if (wait_ns < 0 || wait_ns > 1000000000ll) return GNNFD_INVALID_ARG;
    gnnfd::t_drill_wait_ns = (uint64_t)wait_ns;
    gnnfd::t_drill_skip = skip_k_block;
    return GNNFD_OK;
}

}  // extern "C"
