// bf16 dense products on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   D[m, n] = sum_k A[m, k] * B[n, k]        A: [rows x K] row-major, B: [N x K] row-major (both K-major)
//
// Output tiles are 128 x NT (NT = the widest multiple of 32, at most 256, that divides N).  A single thread feeds TMA
// loads of 128 x 64 (A) and NT x 64 (B) bf16 boxes into a ring of 128-byte-swizzled shared-memory stages that runs on
// across tiles, a single thread issues tcgen05.mma (M = 128, N = NT, K = 16 per instruction) into one of two fp32
// accumulators in tensor memory, and eight warps read the other accumulator back with tcgen05.ld for the epilogue
// (bias / ReLU / per-row scale / mask, rounding to bf16).  Where NT is a multiple of 64 the plain epilogue stages boxes of
// 128 rows x 64 columns in shared memory and sends them off with bulk tensor stores (whole 128-byte lines; a lane's own
// 16-byte stores fill only half a sector each); otherwise, and in the fused forms, each lane stores its row's columns.
// No cluster launch, no multicast.  Every mbarrier wait is bounded; on a timeout the CTA raises E2EGREC_DEV_TIMEOUT in
// the status word, skips its remaining tiles, releases its tensor memory and returns.
#include "gemm_tc.cuh"

#include <cuda.h>

#include <algorithm>

namespace e2egrec {

namespace {

constexpr int kTileM = 128;
constexpr int kTileK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kThreads = 128;
constexpr int kTnEpilogueWarps = 8;          // tc_gemm_tn_kernel: TMA warp, MMA warp, eight epilogue warps
constexpr int kTnThreads = (2 + kTnEpilogueWarps) * 32;
constexpr int kMaxStages = 4;
constexpr int kMinSplitBlocks = 8;          // k-blocks of 64 rows per split of the weight-gradient product
constexpr uint32_t kSpinLimit = 4u * 1000u * 1000u;

// ------------------------------------------------------------------------- PTX wrappers
__device__ inline uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ inline void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

// Bounded wait for the phase with the given parity; false when the limit ran out or another
// thread of the CTA has already given up.
__device__ inline bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t done;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ inline void tma_load_2d(void *smem_dst, const CUtensorMap *map, int x, int y, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// Bulk tensor store shared -> global of one box, and the bookkeeping of such stores (issued and awaited by one thread).
__device__ inline void tma_store_2d(const CUtensorMap *map, const void *smem_src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(reinterpret_cast<uint64_t>(map)),
                 "r"(x), "r"(y), "r"(smem_u32(smem_src))
                 : "memory");
}
__device__ inline void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ inline void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ inline void named_barrier(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
// barrier over `threads` threads that also tells every one of them whether all arrived with ok set
__device__ inline bool named_barrier_all(int id, int threads, bool ok)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r)
                 : "r"((uint32_t)ok), "r"(id), "r"(threads)
                 : "memory");
    return r != 0;
}

__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle.  Eight rows
// form one 1024-byte swizzle atom, so the stride between 8-row groups is 1024 bytes; the leading
// byte offset is not used for this layout.
__device__ inline uint64_t make_smem_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset (ignored, canonical 1)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset
    d |= (uint64_t)1 << 46;                               // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}

// Shared-memory operand descriptor for an operand whose M (or N) index is the contiguous one: the tile is
// a row of 64-element (128-byte) wide column blocks, each block holding one 128-byte line per K index,
// 128-byte swizzled in groups of eight lines.  Leading byte offset = distance between column blocks,
// stride byte offset = distance between groups of eight K lines.
__device__ inline uint64_t make_smem_desc_mn(uint32_t smem_addr, uint32_t block_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((block_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: bf16 x bf16 -> fp32; a_mn_major / b_mn_major = that operand has its M / N
// index contiguous in memory, else it is K-major.
__device__ inline uint32_t make_idesc(int m, int n, bool a_mn_major = false, bool b_mn_major = false)
{
    uint32_t d = 0;
    if (a_mn_major) d |= 1u << 15;
    if (b_mn_major) d |= 1u << 16;
    d |= 1u << 4;                    // accumulator fp32
    d |= 1u << 7;                    // A bf16
    d |= 1u << 10;                   // B bf16
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(m >> 4) << 24;
    return d;
}

__device__ inline void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ inline void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ inline void tmem_load32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct TcEpilogue {
    __nv_bfloat16 *out;        // [rows x ldo]
    int64_t ldo;
    const float *bias;         // per output column, optional
    int relu;
    const float *row_scale;    // optional: columns >= scale_from are multiplied by row_scale[row]
    int scale_from;
    const __nv_bfloat16 *mask; // optional [rows x ld_mask]: outputs are zeroed where mask <= 0 (ReLU derivative)
    int64_t ld_mask;
    const int32_t *m_dev;      // rows at and beyond *m_dev are written as zeros
    __nv_bfloat16 *out2;       // optional second copy of the output: rows below rows2, leading dimension ldo2
    int64_t ldo2, rows2;
    int32_t *status;           // device status word (E2EGREC_DEV_TIMEOUT)
    TcFuse fuse;               // optional gating / product-plus-term forms of the epilogue
    // Several right-hand sides stacked along the rows: A and the output hold n_rhs blocks of rhs_rows rows each (a
    // multiple of 128); in every block the first *m_dev rows are live.  Row scale and mask are shared by the blocks and
    // indexed by the row inside its block.  n_rhs = 1: one block, rhs_rows unused.
    int n_rhs;
    int64_t rhs_rows;
    int tma_out;               // the output leaves through bulk tensor stores of 128 x 64 boxes staged in shared memory (map_out)
    int mode;                  // which steps the plain epilogue has (epi_mode), fixed on the host
};

// Steps of the plain epilogue as bits: bias, ReLU, mask, and the row scale either for whole blocks of 32 columns
// (scale_from a multiple of 32) or decided column by column.
constexpr int kEpiBias = 1, kEpiRelu = 2, kEpiMask = 4, kEpiScaleBlock = 8, kEpiScaleColumn = 16;

// One block of 32 accumulator columns of one row -> 16 packed bf16 pairs:  v = max((acc + bias) * scale, floor), zero where the
// row is dead or the mask says so.  Bias, ReLU and a scale that holds for the whole block are plain arithmetic with neutral
// operands when absent (bias 0, floor -inf, scale 1); the mask and a scale that starts inside a block are compiled in.
// keep: bit j set = column j keeps its value (mask and liveness folded together).
template <bool kMask, bool kScaleColumn>
__device__ inline void epi_block(const uint32_t (&r)[32], uint32_t (&packed)[16], const float *__restrict__ bias_c, bool bias_vec,
                                 float floor_v, float s_block, float rs, int col0, int scale_from, uint32_t keep, bool live)
{
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        float b[4] = {0.f, 0.f, 0.f, 0.f};
        if (bias_c) {
            if (bias_vec) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(bias_c) + q);
                b[0] = v.x; b[1] = v.y; b[2] = v.z; b[3] = v.w;
            } else {
#pragma unroll
                for (int h = 0; h < 4; ++h) b[h] = bias_c[4 * q + h];
            }
        }
        float v[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int j = 4 * q + h;
            v[h] = fmaxf((__uint_as_float(r[j]) + b[h]) * s_block, floor_v);
            if constexpr (kScaleColumn) { if (col0 + j >= scale_from) v[h] *= rs; }
            if constexpr (kMask) { if (!((keep >> j) & 1u)) v[h] = 0.f; }
        }
        __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
        packed[2 * q] = *reinterpret_cast<uint32_t *>(&p0);
        packed[2 * q + 1] = *reinterpret_cast<uint32_t *>(&p1);
    }
    if constexpr (!kMask) {
#pragma unroll
        for (int i = 0; i < 16; ++i) packed[i] = live ? packed[i] : 0u;
    }
}

__device__ inline float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// 32 bf16 values of one row (columns c .. c+31) as 16 packed words; zeros when there is no source
__device__ inline void load_row32(const __nv_bfloat16 *row, bool on, uint32_t (&w)[16])
{
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (on) v = *reinterpret_cast<const uint4 *>(row + q * 8);
        w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
    }
}
__device__ inline float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ inline float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ------------------------------------------------------------------------- kernel
// Persistent: the grid has at most one CTA per SM and every CTA walks over the live output tiles
// t = blockIdx.x, blockIdx.x + gridDim.x, ... (tile t = row tile t / n_tiles_n, column tile t % n_tiles_n, so
// that neighbouring CTAs read the same rows of A and find them in L2).  Warp 0 feeds the TMA ring, warp 1
// issues the MMAs into one of two accumulator buffers in tensor memory, warps 2-9 run the epilogue of the
// previous tile from the other buffer meanwhile (two warps per group of 32 accumulator lanes, each taking
// every other block of 32 columns).
__device__ inline void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// What the plain epilogue knows about its row of the current tile.
struct EpiRow {
    const TcEpilogue *ep;
    const CUtensorMap *map_out;
    __nv_bfloat16 *orow, *orow2;         // the row's slice of the output tile (and of the second copy, or null)
    const __nv_bfloat16 *mrow;           // the row's slice of the mask, or null
    uint8_t *out_stage;                  // the two staging boxes of the bulk stores
    float rs, floor_v;
    int n0, m0, rt;                      // first column / row of the tile, the row inside the tile
    bool live, bias_vec, store_lead;
};

// One block of 32 columns of one row, from accumulator registers to memory.
template <bool kMask, bool kScaleColumn>
__device__ inline void epi_finish_block(const EpiRow &e, const uint32_t (&r)[32], int c, uint32_t &n_box)
{
    const TcEpilogue &ep = *e.ep;
    uint32_t keep = e.live ? 0xFFFFFFFFu : 0u;
    if (kMask && e.live) {
        keep = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 mv = *reinterpret_cast<const uint4 *>(e.mrow + c + q * 8);
            const uint32_t w[4] = {mv.x, mv.y, mv.z, mv.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (__uint_as_float(w[u] << 16) > 0.f) keep |= 1u << (q * 8 + 2 * u);
                if (__uint_as_float(w[u] & 0xFFFF0000u) > 0.f) keep |= 1u << (q * 8 + 2 * u + 1);
            }
        }
    }
    uint32_t packed[16];
    const float s_block = ((ep.mode & kEpiScaleBlock) && e.n0 + c >= ep.scale_from) ? e.rs : 1.f;
    epi_block<kMask, kScaleColumn>(r, packed, ep.bias ? ep.bias + e.n0 + c : nullptr, e.bias_vec, e.floor_v, s_block, e.rs, e.n0 + c,
                                   ep.scale_from, keep, e.live);
    if (ep.tma_out) {
        // The eight warps fill one box of 128 rows x 64 columns (warps 2-5 its left half, 6-9 its right half) in the
        // 128-byte swizzle of the output map, and one thread sends it off as whole lines; two boxes alternate, so a box
        // is refilled only after the store issued two boxes earlier has read it.
        uint8_t *box = e.out_stage + (size_t)(n_box & 1u) * (kTileM * 128);
        ++n_box;
        if (e.store_lead) tma_store_wait_read<1>();
        named_barrier(1, kTnEpilogueWarps * 32);
        const int chunk0 = ((c >> 5) & 1) * 4;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(box + e.rt * 128 + (((chunk0 + q) ^ (e.rt & 7)) << 4)) =
                make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        named_barrier(1, kTnEpilogueWarps * 32);
        if (e.store_lead) {
            tma_store_2d(e.map_out, box, e.n0 + (c & ~63), e.m0);
            tma_store_commit();
        }
    } else {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(e.orow + c + q * 8) =
                make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
    }
    if (e.orow2) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(e.orow2 + c + q * 8) =
                make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
    }
}

// The blocks of 32 columns (c_first, c_first + 64, ...) that one warp takes from a finished accumulator; the accumulator
// buffer goes back to the MMA warp as soon as the warp's last block is in registers.
template <bool kMask, bool kScaleColumn>
__device__ inline void epi_tile_plain(const EpiRow &e, uint32_t taddr, int c_first, int nt, uint64_t *acc_empty, int lane, uint32_t &n_box)
{
    for (int c = c_first; c < nt; c += 64) {
        uint32_t r[32];
        tmem_load32(taddr + (uint32_t)c, r);
        if (c + 64 >= nt) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);
        }
        epi_finish_block<kMask, kScaleColumn>(e, r, c, n_box);
    }
}

// kFuse: the gating / product-plus-term forms of the epilogue (TcFuse); the plain instantiation carries none of their
// registers or branches.
template <bool kFuse>
__global__ void __launch_bounds__(kTnThreads)
tc_gemm_tn_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_out, int k_blocks, int stages, int nt, int n_tiles_n, uint32_t tmem_cols,
                  int b_mn, TcEpilogue ep)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();                    // (with programmatic launches) the next kernel may set itself up beside this one
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t a_bytes = kTileM * kTileK * 2, b_bytes = (uint32_t)nt * kTileK * 2;
    uint8_t *a_tiles = tiles;
    uint8_t *b_tiles = tiles + (size_t)stages * a_bytes;
    uint8_t *out_stage = b_tiles + (size_t)stages * b_bytes;      // two boxes of 128 rows x 128 bytes (ep.tma_out)

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], kTnEpilogueWarps);
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                            // tensor memory: two accumulators of tmem_cols / 2 fp32 columns x 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t buf_stride = tmem_cols >> 1;
    // barriers and tensor memory are set up; global memory is touched only once the preceding kernel has completed
    pdl_wait();
    const int32_t m_valid = *ep.m_dev;
    const int64_t live_tiles = ((int64_t)m_valid + kTileM - 1) / kTileM;    // per block of rows; tiles wholly beyond *m_dev stay as they are
    const int64_t n_work = live_tiles * n_tiles_n * ep.n_rhs;
    // tile t of the list: column tile t % n_tiles_n of live row tile (t / n_tiles_n) % live_tiles of block (t / n_tiles_n) / live_tiles
    auto tile_rows = [&](int64_t t, int64_t &m0, int64_t &m0_local) {
        const int64_t rt = t / n_tiles_n;
        const int64_t rhs = ep.n_rhs > 1 ? rt / live_tiles : 0;
        m0_local = (rt - rhs * live_tiles) * kTileM;
        m0 = rhs * ep.rhs_rows + m0_local;
    };

    if ((int64_t)blockIdx.x >= n_work) {
        // nothing for this CTA: straight to the release of its tensor memory
    } else if (warp == 0) {
        if (lane == 0) {
            // ---- producer: TMA loads into the stage ring, k-block after k-block across tiles
            uint32_t g = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_work && ok; t += gridDim.x) {
                int64_t m0_64, m0_local;
                tile_rows(t, m0_64, m0_local);
                const int m0 = (int)m0_64, n0 = (int)(t % n_tiles_n) * nt;
                for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                    const uint32_t s = g % (uint32_t)stages, ph = (g / (uint32_t)stages) & 1u;
                    ok = mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&full_bar[s], a_bytes + b_bytes);
                    tma_load_2d(a_tiles + (size_t)s * a_bytes, &map_a, kb * kTileK, m0, &full_bar[s]);
                    if (b_mn) {                 // B stored [K x N]: one 64-column block of 64 K lines per copy
                        for (int j = 0; j < nt / 64; ++j)
                            tma_load_2d(b_tiles + (size_t)s * b_bytes + j * (kTileK * 128), &map_b, n0 + j * 64, kb * kTileK,
                                        &full_bar[s]);
                    } else {
                        tma_load_2d(b_tiles + (size_t)s * b_bytes, &map_b, kb * kTileK, n0, &full_bar[s]);
                    }
                }
            }
            if (!ok) {
                // giving up: let the copies that were started land before the shared memory is released
                int never = 0;
                for (uint32_t j = g > (uint32_t)stages ? g - stages : 0; j < g; ++j)
                    mbar_wait(&full_bar[j % stages], (j / stages) & 1u, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer
            const uint32_t idesc = make_idesc(kTileM, nt, false, b_mn != 0);
            uint32_t g = 0, lt = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_work && ok; t += gridDim.x, ++lt) {
                const uint32_t buf = lt & 1u;
                ok = mbar_wait(&acc_empty[buf], ((lt >> 1) & 1u) ^ 1u, &abort_flag);   // the epilogue has drained this buffer
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * buf_stride;
                for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                    const uint32_t s = g % (uint32_t)stages, ph = (g / (uint32_t)stages) & 1u;
                    ok = mbar_wait(&full_bar[s], ph, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(a_tiles + (size_t)s * a_bytes);
                    const uint32_t b_addr = smem_u32(b_tiles + (size_t)s * b_bytes);
#pragma unroll
                    for (int k = 0; k < kTileK / kUmmaK; ++k) {
                        const uint64_t ad = make_smem_desc(a_addr + k * kUmmaK * 2);
                        const uint64_t bd = b_mn ? make_smem_desc_mn(b_addr + k * kUmmaK * 128, kTileK * 128)
                                                 : make_smem_desc(b_addr + k * kUmmaK * 2);
                        umma(d_tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[s]);     // the stage is free again once these MMAs have read it
                }
                if (ok) umma_commit(&acc_full[buf]);   // accumulator complete
            }
        }
    } else {
        // ---- epilogue: warp w reads accumulator lanes 32 (w % 4) .. + 31 = rows m0 + 32 (w % 4) + lane
        const int lg = warp & 3;                    // the lane group a warp may read is fixed by its index mod 4
        const int c_first = warp >= 6 ? 32 : 0;     // warps 2-5 take column blocks 0, 2, 4, ...; warps 6-9 the odd ones
        int c_last = c_first;                       // this warp's last column block
        while (c_last + 64 < nt) c_last += 64;
        uint32_t lt = 0, n_box = 0;                 // n_box: boxes of 64 columns handed to the bulk stores so far
        const bool store_lead = warp == 2 && lane == 0;
        for (int64_t t = blockIdx.x; t < n_work; t += gridDim.x, ++lt) {
            const uint32_t buf = lt & 1u;
            bool ready = mbar_wait(&acc_full[buf], (lt >> 1) & 1u, &abort_flag);
            // with staged stores the warps meet at barriers inside the tile: all of them take it, or none does
            if (!kFuse && ep.tma_out) ready = named_barrier_all(2, kTnEpilogueWarps * 32, ready);
            if (!ready) break;
            tc_fence_after();
            int64_t m0, m0_local;
            tile_rows(t, m0, m0_local);
            const int n0 = (int)(t % n_tiles_n) * nt;
            const int64_t row = m0 + lg * 32 + lane;
            const int64_t row_local = m0_local + lg * 32 + lane;        // the row inside its block of rows
            const bool live = row_local < m_valid;
            const float rs = (ep.row_scale && live) ? ep.row_scale[row_local] : 1.f;
            __nv_bfloat16 *orow = ep.out + row * ep.ldo + n0;
            const __nv_bfloat16 *mrow = ep.mask ? ep.mask + row_local * ep.ld_mask + n0 : nullptr;
            __nv_bfloat16 *orow2 = (ep.out2 && row < ep.rows2) ? ep.out2 + row * ep.ldo2 + n0 : nullptr;
            if (c_first >= nt) {                          // a single column block: nothing for the second set of warps
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
                continue;
            }
            if constexpr (!kFuse) {
                EpiRow e;
                e.ep = &ep;
                e.map_out = &map_out;
                e.orow = orow;
                e.orow2 = orow2;
                e.mrow = mrow;
                e.out_stage = out_stage;
                e.rs = rs;
                e.n0 = n0;
                e.m0 = (int)m0;
                e.rt = lg * 32 + lane;
                e.live = live;
                e.bias_vec = (reinterpret_cast<uintptr_t>(ep.bias) & 15) == 0;
                e.store_lead = store_lead;
                const uint32_t taddr = tmem_base + buf * buf_stride + ((uint32_t)(lg * 32) << 16);
                e.floor_v = ep.relu ? 0.f : -INFINITY;
                if (ep.mode & kEpiMask) {
                    if (ep.mode & kEpiScaleColumn) epi_tile_plain<true, true>(e, taddr, c_first, nt, &acc_empty[buf], lane, n_box);
                    else epi_tile_plain<true, false>(e, taddr, c_first, nt, &acc_empty[buf], lane, n_box);
                } else {
                    if (ep.mode & kEpiScaleColumn) epi_tile_plain<false, true>(e, taddr, c_first, nt, &acc_empty[buf], lane, n_box);
                    else epi_tile_plain<false, false>(e, taddr, c_first, nt, &acc_empty[buf], lane, n_box);
                }
            } else {
            for (int c = c_first; c < nt; c += 64) {
                uint32_t r[32];
                tmem_load32(tmem_base + buf * buf_stride + ((uint32_t)(lg * 32) << 16) + (uint32_t)c, r);
                if (c == c_last) {                        // this warp's share of the buffer is in registers: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[buf]);
                }
                uint32_t packed[16];
                uint32_t mbits = 0xFFFFFFFFu;                 // bit j: output column c + j keeps its value
                if (mrow && live) {
                    mbits = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint4 mv = *reinterpret_cast<const uint4 *>(mrow + c + q * 8);
                        const uint32_t w[4] = {mv.x, mv.y, mv.z, mv.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (__uint_as_float(w[u] << 16) > 0.f) mbits |= 1u << (q * 8 + 2 * u);
                            if (__uint_as_float(w[u] & 0xFFFF0000u) > 0.f) mbits |= 1u << (q * 8 + 2 * u + 1);
                        }
                    }
                }
                if (kFuse && ep.fuse.gate_in) {
                    // gating: the accumulator (+ bias) is the pre-activation; g = sigmoid(pre) with pre and g rounded to
                    // their storage type, the output is g * F and g itself goes to gate_out
                    uint32_t fw[16], gpk[16];
                    load_row32(ep.fuse.gate_in + row * ep.fuse.ld_gate_in + n0 + c, live, fw);
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float g[2];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            float p = __uint_as_float(r[j + h]);
                            if (ep.bias) p += ep.bias[n0 + c + j + h];
                            p = bf16_round(p);
                            const float e = expf(-fabsf(p));
                            g[h] = live ? bf16_round(p >= 0.f ? 1.0f / (1.0f + e) : e / (1.0f + e)) : 0.f;
                        }
                        __nv_bfloat162 gh = __floats2bfloat162_rn(g[0], g[1]);
                        gpk[j >> 1] = *reinterpret_cast<uint32_t *>(&gh);
                        __nv_bfloat162 oh = __floats2bfloat162_rn(g[0] * bf16_lo(fw[j >> 1]), g[1] * bf16_hi(fw[j >> 1]));
                        packed[j >> 1] = *reinterpret_cast<uint32_t *>(&oh);
                    }
                    if (ep.fuse.gate_out) {
                        __nv_bfloat16 *grow = ep.fuse.gate_out + row * ep.fuse.ld_gate_out + n0 + c;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            *reinterpret_cast<uint4 *>(grow + q * 8) = make_uint4(gpk[4 * q], gpk[4 * q + 1], gpk[4 * q + 2], gpk[4 * q + 3]);
                    }
                } else {
                uint32_t aw[16], bw[16];                      // dead (and removed) in the plain instantiation
                if constexpr (kFuse) {
                    if (ep.fuse.add_a) {                      // out = round(product) + a * b
                        load_row32(ep.fuse.add_a + row * ep.fuse.ld_add_a + n0 + c, live, aw);
                        load_row32(ep.fuse.add_b + row * ep.fuse.ld_add_b + n0 + c, live, bw);
                    }
                }
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float v0 = __uint_as_float(r[j]), v1 = __uint_as_float(r[j + 1]);
                    const int col = n0 + c + j;
                    if (ep.bias) { v0 += ep.bias[col]; v1 += ep.bias[col + 1]; }
                    if (ep.relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
                    if (ep.row_scale) {
                        if (col >= ep.scale_from) v0 *= rs;
                        if (col + 1 >= ep.scale_from) v1 *= rs;
                    }
                    if constexpr (kFuse) {
                        if (ep.fuse.add_a) {
                            v0 = bf16_round(v0) + bf16_lo(aw[j >> 1]) * bf16_lo(bw[j >> 1]);
                            v1 = bf16_round(v1) + bf16_hi(aw[j >> 1]) * bf16_hi(bw[j >> 1]);
                        }
                    }
                    if (!live || !((mbits >> j) & 1u)) v0 = 0.f;
                    if (!live || !((mbits >> (j + 1)) & 1u)) v1 = 0.f;
                    __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                    packed[j >> 1] = *reinterpret_cast<uint32_t *>(&h);
                }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    *reinterpret_cast<uint4 *>(orow + c + q * 8) =
                        make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                if (orow2) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(orow2 + c + q * 8) =
                            make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                }
            }
            }
        }
        if (store_lead) tma_store_wait_read<0>();   // the staging boxes have been read; the kernel's end publishes the stores
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicOr(reinterpret_cast<unsigned *>(ep.status), E2EGREC_DEV_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

constexpr int kMaxDevices = 64;
constexpr int kMaxDynSmem = 226 * 1024;             // of the 227 KB a block may have; the kernels' static part is below 1 KB

int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return 0; }
    return dev;
}

int sm_count()
{
    static int n[kMaxDevices] = {};                  // per device; a race between threads writes the same value twice
    const int dev = current_device();
    if (n[dev] <= 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        n[dev] = v;
    }
    return n[dev];
}

// Raises the kernel's dynamic shared-memory limit once per device (the attribute belongs to the device's copy of
// the kernel, so a second device in the same process needs its own call).
template <typename Kernel>
bool raise_smem_limit(Kernel kernel, bool (&done)[kMaxDevices])
{
    const int dev = current_device();
    if (done[dev]) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem) != cudaSuccess) return false;
    done[dev] = true;
    return true;
}

// [rows x k] bf16 row-major, box = 64 x box_rows, 128-byte swizzle
bool make_map(CUtensorMap *map, const void *base, int64_t rows, int64_t k, int64_t ld, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)k, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map_mn(CUtensorMap *map, const void *base, int64_t rows, int64_t cols);

// b_mn: B is stored [k x n] row-major (its N index contiguous) instead of [n x k]
bool launch_tn(const __nv_bfloat16 *A, int64_t rows, int k, int64_t lda, const __nv_bfloat16 *B, int n, int64_t ldb,
               const TcEpilogue &ep_in, cudaStream_t st, bool b_mn = false, int n_rhs = 1)
{
    if (rows <= 0 || rows % kTileM || k % kTileK || k < kTileK || n_rhs < 1) return false;
    TcEpilogue ep = ep_in;
    ep.n_rhs = n_rhs;
    ep.rhs_rows = rows;
    int nt = 0;                                 // widest tile <= 256 columns that divides n (a multiple of 32, or of 64 for b_mn)
    const int unit = b_mn ? 64 : 32;
    for (int c = 256; c >= unit; c -= unit)
        if (n % c == 0) { nt = c; break; }
    if (!nt) return false;
    if (reinterpret_cast<uintptr_t>(A) % 16 || reinterpret_cast<uintptr_t>(B) % 16 || (lda * 2) % 16 || (ldb * 2) % 16 ||
        reinterpret_cast<uintptr_t>(ep.out) % 16 || (ep.ldo * 2) % 16)
        return false;
    const bool fused = ep.fuse.gate_in || ep.fuse.add_a;
    const int k_blocks = k / kTileK;
    // the stage ring runs on across tiles, so a short K still keeps kMaxStages loads in flight (the next tiles' operands)
    // Two to kMaxStages stages inside a budget that leaves a quarter of the SM's shared memory to the blocks of other
    // streams' kernels: the stage ring runs on across tiles, and a third or fourth stage buys this kernel less than the
    // co-resident blocks of the sampling kernels lose when they find no room (E2EGREC_GEMM_SMEM_KB overrides the budget).
    static const bool direct_only = []() { const char *e = getenv("E2EGREC_GEMM_DIRECT_STORE"); return e && *e && e[0] != '0'; }();
    static const size_t budget = []() {
        const char *e = getenv("E2EGREC_GEMM_SMEM_KB");
        const long kb = e && *e ? atol(e) : 178;
        return (size_t)std::min<long>(std::max<long>(kb, 64), kMaxDynSmem / 1024) * 1024;
    }();
    const size_t stage_bytes = kTileM * kTileK * 2 + (size_t)nt * kTileK * 2;
    ep.tma_out = !fused && !direct_only && nt % 64 == 0;
    const size_t fixed_bytes = 1024 + (ep.tma_out ? 2 * kTileM * 128 : 0);
    const int stages = (int)std::max<size_t>(2, std::min<size_t>(kMaxStages, (budget - fixed_bytes) / stage_bytes));
    const size_t smem = (size_t)stages * stage_bytes + fixed_bytes;
    ep.mode = (ep.bias ? kEpiBias : 0) | (ep.relu ? kEpiRelu : 0) | (ep.mask ? kEpiMask : 0) |
              (ep.row_scale ? (ep.scale_from % 32 == 0 ? kEpiScaleBlock : kEpiScaleColumn) : 0);
    CUtensorMap ma, mb, mo;
    if (!make_map(&ma, A, rows * n_rhs, k, lda, kTileM)) return false;
    if (ep.tma_out ? !make_map(&mo, ep.out, rows * n_rhs, n, ep.ldo, kTileM) : false) return false;
    if (!ep.tma_out) mo = ma;
    if (b_mn ? (ldb != n || !make_map_mn(&mb, B, k, n)) : !make_map(&mb, B, n, k, ldb, nt)) return false;
    uint32_t tmem_cols = 64;                    // two accumulator buffers, each a power of two of columns >= nt
    while ((int)tmem_cols < 2 * nt) tmem_cols <<= 1;
    static bool attr_set[2][kMaxDevices] = {};
    if (!(fused ? raise_smem_limit(tc_gemm_tn_kernel<true>, attr_set[1]) : raise_smem_limit(tc_gemm_tn_kernel<false>, attr_set[0])))
        return false;
    const int n_tiles_n = n / nt;
    const int64_t tiles_cap = (rows / kTileM) * n_tiles_n * n_rhs;
    const unsigned grid = (unsigned)std::min<int64_t>(tiles_cap, sm_count());
    note_launch();
    if (fused)
        launch_pdl(tc_gemm_tn_kernel<true>, dim3(grid), dim3(kTnThreads), smem, st, ma, mb, mo, k_blocks, stages, nt, n_tiles_n, tmem_cols,
                   b_mn ? 1 : 0, ep);
    else
        launch_pdl(tc_gemm_tn_kernel<false>, dim3(grid), dim3(kTnThreads), smem, st, ma, mb, mo, k_blocks, stages, nt, n_tiles_n, tmem_cols,
                   b_mn ? 1 : 0, ep);
    return true;
}


// ------------------------------------------------------------------------- transposed product, split over rows
//   part[z][m, n] = sum over the rows r of split z of  Y[r, m] * X[r, n]      (weight gradients)
// Y [rows x M] and X [rows x N] are row-major, so both operands reach the tensor cores with their M / N
// index contiguous.  A k-block is 64 rows; the blocks up to the first multiple of 64 at or above *m_dev
// are shared evenly by gridDim.z CTAs per output tile (rows between *m_dev and that multiple must hold
// zeros in both matrices).  A CTA without blocks writes zeros.
__global__ void __launch_bounds__(kThreads)
tc_gemm_rows_kernel(const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_x, int nt,
                    uint32_t tmem_cols, int stages, const int32_t *m_dev, float *__restrict__ part, int64_t ldp,
                    int64_t split_stride, int32_t *status, int n_rhs, int64_t rhs_rows)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], accum_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kTileM, n0 = blockIdx.y * nt;
    pdl_launch_dependents();
    pdl_wait();                                 // the preceding kernel of the stream has completed
    const int64_t m_valid = *m_dev;
    // Y may hold n_rhs blocks of rhs_rows rows (the first *m_dev of each live) that all meet the same rows of X: the
    // k-blocks of the blocks of rows form one list, and the sum runs over all of them
    const int64_t blocks_per_rhs = (m_valid + kTileK - 1) / kTileK;
    const int64_t total_blocks = blocks_per_rhs * n_rhs;
    // at least kMinSplitBlocks k-blocks per split: only the first ceil(total / per) splits do work and
    // write a partial (split 0 writes zeros when there are no rows); splitk_reduce_kernel uses the same rule
    const int64_t per = max((int64_t)kMinSplitBlocks, (total_blocks + gridDim.z - 1) / gridDim.z);
    const int64_t active = max((int64_t)1, (total_blocks + per - 1) / per);
    if ((int64_t)blockIdx.z >= active) return;
    const int64_t kb0 = (int64_t)blockIdx.z * per;
    const int64_t kb1 = kb0 + per < total_blocks ? kb0 + per : total_blocks;
    const int k_blocks = kb1 > kb0 ? (int)(kb1 - kb0) : 0;
    float *out = part + (int64_t)blockIdx.z * split_stride + (int64_t)(m0 + warp * 32 + lane) * ldp + n0;
    if (k_blocks == 0) {
        for (int c = 0; c < nt; c += 4) *reinterpret_cast<float4 *>(out + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr uint32_t blk_bytes = kTileK * 128;            // one 64-column block: 64 K lines of 128 bytes
    const uint32_t a_bytes = (kTileM / 64) * blk_bytes, b_bytes = (uint32_t)(nt / 64) * blk_bytes;
    uint8_t *a_tiles = tiles;
    uint8_t *b_tiles = tiles + (size_t)stages * a_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    int issued = 0;
    if (warp == 0 && lane == 0) {
        for (int kb = 0; kb < k_blocks; ++kb) {
            const int s = kb % stages;
            const uint32_t ph = (uint32_t)(kb / stages) & 1u;
            if (!mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag)) break;
            mbar_expect_tx(&full_bar[s], a_bytes + b_bytes);
            const int64_t jb = kb0 + kb;
            const int64_t rhs = n_rhs > 1 ? jb / blocks_per_rhs : 0;
            const int row_x = (int)((jb - rhs * blocks_per_rhs) * kTileK);
            const int row_y = (int)(rhs * rhs_rows) + row_x;
            for (int j = 0; j < kTileM / 64; ++j)
                tma_load_2d(a_tiles + (size_t)s * a_bytes + j * blk_bytes, &map_y, m0 + j * 64, row_y, &full_bar[s]);
            for (int j = 0; j < nt / 64; ++j)
                tma_load_2d(b_tiles + (size_t)s * b_bytes + j * blk_bytes, &map_x, n0 + j * 64, row_x, &full_bar[s]);
            issued = kb + 1;
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = make_idesc(kTileM, nt, true, true);
        bool ok = true;
        for (int kb = 0; kb < k_blocks && ok; ++kb) {
            const int s = kb % stages;
            const uint32_t ph = (uint32_t)(kb / stages) & 1u;
            ok = mbar_wait(&full_bar[s], ph, &abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_addr = smem_u32(a_tiles + (size_t)s * a_bytes);
            const uint32_t b_addr = smem_u32(b_tiles + (size_t)s * b_bytes);
#pragma unroll
            for (int k = 0; k < kTileK / kUmmaK; ++k) {     // 16 K lines = 2048 bytes further into every block
                const uint64_t ad = make_smem_desc_mn(a_addr + k * kUmmaK * 128, blk_bytes);
                const uint64_t bd = make_smem_desc_mn(b_addr + k * kUmmaK * 128, blk_bytes);
                umma(tmem_base, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            umma_commit(&empty_bar[s]);
        }
        if (ok) umma_commit(&accum_bar);
    }
    __syncwarp();

    const bool ready = mbar_wait(&accum_bar, 0, &abort_flag);
    tc_fence_after();
    if (ready) {
        for (int c = 0; c < nt; c += 32) {
            uint32_t r[32];
            tmem_load32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, r);
#pragma unroll
            for (int q = 0; q < 8; ++q)
                *reinterpret_cast<float4 *>(out + c + q * 4) =
                    make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]),
                                __uint_as_float(r[4 * q + 3]));
        }
    } else if (threadIdx.x == 0) {
        atomicOr(reinterpret_cast<unsigned *>(status), E2EGREC_DEV_TIMEOUT);
        int never = 0;
        for (int kb = issued > stages ? issued - stages : 0; kb < issued; ++kb)
            mbar_wait(&full_bar[kb % stages], (uint32_t)(kb / stages) & 1u, &never);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// [rows x cols] bf16 row-major seen with the column index innermost: box = 64 columns x 64 rows
bool make_map_mn(CUtensorMap *map, const void *base, int64_t rows, int64_t cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTileK};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// ------------------------------------------------------------------------- aggregation fused into the A operand
// Eq. 2 and Eq. 3 of one layer in one kernel:  h' = act([h_self | mean of the sampled neighbours] W^T + b).  Gather warps
// build the 128 x 2d rows of a tile of Cat in shared memory, in the 128-byte-swizzled k-block layout the tensor cores read
// (the layout a TMA load of the stored Cat would leave there), and store the same rows once to global memory for the
// backward pass; the dense transform never reads Cat back.  W streams through a TMA ring as in tc_gemm_tn_kernel, four
// warps run the epilogue from two accumulators in tensor memory.  Rows are summed in the order of sage_aggregate_kernel
// and rounded to bf16 at the same points, so Cat and h' have the bits of the two-kernel path.
// LPR: lanes per gathered row = 2 d / 16 (d = 64, 128 or 256 values).
constexpr int kFusedGatherWarps = 20;
constexpr int kFusedEpiWarps = 4;
constexpr int kFusedThreads = (2 + kFusedEpiWarps + kFusedGatherWarps) * 32;

template <int LPR>
__global__ void __launch_bounds__(kFusedThreads)
tc_sage_fused_kernel(const __grid_constant__ CUtensorMap map_b, const __nv_bfloat16 *__restrict__ Hsrc, int64_t ld,
                     const int32_t *__restrict__ nbr, const int32_t *__restrict__ self_ids, const int32_t *__restrict__ indptr,
                     __nv_bfloat16 *__restrict__ cat, int nt, int stages, int a_bufs, uint32_t tmem_cols, TcEpilogue ep)
{
    constexpr int kKbHalf = LPR / 8;                 // k-blocks of 64 columns per half of Cat
    constexpr int kKb = 2 * kKbHalf;
    constexpr uint32_t kKbBytes = kTileM * 128;      // one k-block of the A tile: 128 rows x 128 bytes
    constexpr int d = LPR * 8;
    constexpr int G = 32 / LPR;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t b_full[kMaxStages], b_empty[kMaxStages], a_full[2], a_empty[2], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_tiles = tiles;
    const uint32_t b_bytes = (uint32_t)nt * kTileK * 2;
    uint8_t *b_tiles = tiles + (size_t)a_bufs * kKb * kKbBytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&b_full[s], 1);
            mbar_init(&b_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&a_full[b], kFusedGatherWarps);
            mbar_init(&a_empty[b], 1);
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], kFusedEpiWarps);
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t buf_stride = tmem_cols >> 1;
    const int32_t n_dst = *ep.m_dev;
    const int64_t live_tiles = ((int64_t)n_dst + kTileM - 1) / kTileM;

    if ((int64_t)blockIdx.x >= live_tiles) {
        // nothing for this CTA
    } else if (warp == 0) {
        if (lane == 0) {
            // ---- W through the stage ring, k-block after k-block across tiles
            uint32_t g = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < live_tiles && ok; t += gridDim.x) {
                for (int kb = 0; kb < kKb; ++kb, ++g) {
                    const uint32_t s = g % (uint32_t)stages, ph = (g / (uint32_t)stages) & 1u;
                    ok = mbar_wait(&b_empty[s], ph ^ 1u, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&b_full[s], b_bytes);
                    tma_load_2d(b_tiles + (size_t)s * b_bytes, &map_b, kb * kTileK, 0, &b_full[s]);
                }
            }
            if (!ok) {
                int never = 0;
                for (uint32_t j = g > (uint32_t)stages ? g - stages : 0; j < g; ++j)
                    mbar_wait(&b_full[j % stages], (j / stages) & 1u, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer
            const uint32_t idesc = make_idesc(kTileM, nt);
            uint32_t g = 0, lt = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < live_tiles && ok; t += gridDim.x, ++lt) {
                const uint32_t buf = lt & 1u;
                const uint32_t ab = a_bufs == 2 ? (lt & 1u) : 0u, use = a_bufs == 2 ? (lt >> 1) : lt;
                ok = mbar_wait(&acc_empty[buf], ((lt >> 1) & 1u) ^ 1u, &abort_flag) && mbar_wait(&a_full[ab], use & 1u, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * buf_stride;
                const uint32_t a_base = smem_u32(a_tiles + (size_t)ab * kKb * kKbBytes);
                for (int kb = 0; kb < kKb; ++kb, ++g) {
                    const uint32_t s = g % (uint32_t)stages, ph = (g / (uint32_t)stages) & 1u;
                    ok = mbar_wait(&b_full[s], ph, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = a_base + kb * kKbBytes;
                    const uint32_t b_addr = smem_u32(b_tiles + (size_t)s * b_bytes);
#pragma unroll
                    for (int k = 0; k < kTileK / kUmmaK; ++k)
                        umma(d_tmem, make_smem_desc(a_addr + k * kUmmaK * 2), make_smem_desc(b_addr + k * kUmmaK * 2), idesc,
                             (kb | k) != 0 ? 1u : 0u);
                    umma_commit(&b_empty[s]);
                }
                if (ok) {
                    umma_commit(&a_empty[ab]);      // the tile of Cat has been read: the gather warps may refill it
                    umma_commit(&acc_full[buf]);
                }
            }
        }
    } else if (warp < 2 + kFusedEpiWarps) {
        // ---- epilogue: warp w reads accumulator lanes 32 (w % 4) .. + 31, all column blocks
        const int lg = warp & 3;
        uint32_t lt = 0, n_box = 0;
        for (int64_t t = blockIdx.x; t < live_tiles; t += gridDim.x, ++lt) {
            const uint32_t buf = lt & 1u;
            if (!mbar_wait(&acc_full[buf], (lt >> 1) & 1u, &abort_flag)) break;
            tc_fence_after();
            const int64_t row = t * kTileM + lg * 32 + lane;
            EpiRow e;
            e.ep = &ep;
            e.map_out = nullptr;
            e.orow = ep.out + row * ep.ldo;
            e.orow2 = (ep.out2 && row < ep.rows2) ? ep.out2 + row * ep.ldo2 : nullptr;
            e.mrow = nullptr;
            e.out_stage = nullptr;
            e.rs = 1.f;
            e.floor_v = ep.relu ? 0.f : -INFINITY;
            e.n0 = 0;
            e.m0 = (int)(t * kTileM);
            e.rt = lg * 32 + lane;
            e.live = row < n_dst;
            e.bias_vec = (reinterpret_cast<uintptr_t>(ep.bias) & 15) == 0;
            e.store_lead = false;
            const uint32_t taddr = tmem_base + buf * buf_stride + ((uint32_t)(lg * 32) << 16);
            for (int c = 0; c < nt; c += 32) {
                uint32_t r[32];
                tmem_load32(taddr + (uint32_t)c, r);
                if (c + 32 >= nt) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[buf]);
                }
                epi_finish_block<false, false>(e, r, c, n_box);
            }
        }
    } else {
        // ---- gather: warp gw builds rows gw, gw + kFusedGatherWarps, ... of every tile
        const int gw = warp - (2 + kFusedEpiWarps);
        const int g = lane / LPR, c = lane % LPR;
        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < live_tiles; t += gridDim.x, ++lt) {
            const uint32_t ab = a_bufs == 2 ? (lt & 1u) : 0u, use = a_bufs == 2 ? (lt >> 1) : lt;
            if (!mbar_wait(&a_empty[ab], (use & 1u) ^ 1u, &abort_flag)) break;
            uint8_t *A = a_tiles + (size_t)ab * kKb * kKbBytes;
            // swizzled place of 16-byte chunk q (0 .. 2 LPR - 1) of row r of the tile
            auto a_slot = [&](int r, int q) { return A + (q >> 3) * kKbBytes + r * 128 + (((q & 7) ^ (r & 7)) << 4); };
            int32_t beg = 0, end = 0, mine = 0;
            int64_t self_row = 0;
            auto fetch = [&](int64_t ii, int32_t &b, int32_t &e, int32_t &m, int64_t &sr) {
                b = e = m = 0;
                sr = ii;
                if (ii < n_dst) {
                    b = indptr[ii];
                    e = indptr[ii + 1];
                    if (lane < e - b) m = nbr[b + lane];
                    if (self_ids) sr = (int64_t)self_ids[ii];
                }
            };
            fetch(t * kTileM + gw, beg, end, mine, self_row);
            for (int r = gw; r < kTileM; r += kFusedGatherWarps) {
                const int64_t i = t * kTileM + r;
                int32_t beg_n = 0, end_n = 0, mine_n = 0;
                int64_t self_n = 0;
                if (r + kFusedGatherWarps < kTileM) fetch(i + kFusedGatherWarps, beg_n, end_n, mine_n, self_n);
                __nv_bfloat16 *out = cat + i * 2 * d;
                if (i >= n_dst) {
                    // rows beyond the last destination: zeros (the weight gradient reads whole k-blocks of 64 rows of Cat)
                    for (int q = lane; q < 2 * LPR; q += 32) {
                        *reinterpret_cast<uint4 *>(out + q * 8) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(a_slot(r, q)) = make_uint4(0, 0, 0, 0);
                    }
                } else {
                    if (lane < LPR) {           // self half
                        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(Hsrc + self_row * ld + lane * 8));
                        *reinterpret_cast<uint4 *>(out + lane * 8) = v;
                        *reinterpret_cast<uint4 *>(a_slot(r, lane)) = v;
                    }
                    float acc[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
                    for (int32_t base = beg; base < end; base += 32) {
                        const int m = min(32, end - base);
                        if (base != beg) mine = lane < m ? nbr[base + lane] : 0;
                        for (int tt = 0; tt * G < m; tt += 4) {
                            uint4 v[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const int j = (tt + u) * G + g;
                                const int32_t id = __shfl_sync(0xffffffffu, mine, j & 31);
                                v[u] = make_uint4(0, 0, 0, 0);
                                if (j < m) v[u] = __ldg(reinterpret_cast<const uint4 *>(Hsrc + (int64_t)id * ld + c * 8));
                            }
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                float x[8];
                                Chunk<__nv_bfloat16>::unpack(v[u], x);
#pragma unroll
                                for (int k = 0; k < 8; k += 2) add2(acc[k], acc[k + 1], x[k], x[k + 1]);
                            }
                        }
                    }
#pragma unroll
                    for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                        for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], off);
                    if (g == 0) {
                        const int32_t cnt = end - beg;
                        const float inv = cnt > 0 ? 1.0f / (float)cnt : 0.0f;
                        uint32_t w[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * k] * inv, acc[2 * k + 1] * inv);
                            w[k] = *reinterpret_cast<uint32_t *>(&h);
                        }
                        const uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
                        *reinterpret_cast<uint4 *>(out + d + c * 8) = v;
                        *reinterpret_cast<uint4 *>(a_slot(r, LPR + c)) = v;
                    }
                }
                beg = beg_n;
                end = end_n;
                mine = mine_n;
                self_row = self_n;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // the tensor cores read what this warp wrote
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[ab]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicOr(reinterpret_cast<unsigned *>(ep.status), E2EGREC_DEV_TIMEOUT);
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

template <int LPR>
bool launch_fused(const CUtensorMap &mb, const __nv_bfloat16 *Hsrc, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                  const int32_t *indptr, __nv_bfloat16 *cat, int64_t rows, int n, const TcEpilogue &ep, cudaStream_t st)
{
    constexpr int kKb = 2 * (LPR / 8);
    const size_t a_bytes = (size_t)kKb * kTileM * 128, b_bytes = (size_t)n * kTileK * 2;
    // two tiles of Cat where they fit beside at least two stages of W, else one
    const int a_bufs = 2 * a_bytes + 2 * b_bytes + 1024 <= (size_t)kMaxDynSmem ? 2 : 1;
    if (a_bufs * a_bytes + 2 * b_bytes + 1024 > (size_t)kMaxDynSmem) return false;
    const int stages = (int)std::min<size_t>(kMaxStages, ((size_t)kMaxDynSmem - 1024 - a_bufs * a_bytes) / b_bytes);
    const size_t smem = a_bufs * a_bytes + (size_t)stages * b_bytes + 1024;
    static bool attr_set[kMaxDevices] = {};
    if (!raise_smem_limit(tc_sage_fused_kernel<LPR>, attr_set)) return false;
    uint32_t tmem_cols = 64;
    while ((int)tmem_cols < 2 * n) tmem_cols <<= 1;
    const unsigned grid = (unsigned)std::min<int64_t>(rows / kTileM, sm_count());
    note_launch();
    tc_sage_fused_kernel<LPR><<<grid, kFusedThreads, smem, st>>>(mb, Hsrc, ld, nbr, self_ids, indptr, cat, n, stages, a_bufs,
                                                                 tmem_cols, ep);
    return true;
}

}  // namespace

bool tc_update_forward(const __nv_bfloat16 *cat, int64_t rows, int k, const __nv_bfloat16 *W, int n, const float *bias,
                       int relu, __nv_bfloat16 *out, const int32_t *m_dev, int32_t *status, cudaStream_t st,
                       __nv_bfloat16 *out2, int64_t ldo2, int64_t rows2)
{
    if (out2 && (reinterpret_cast<uintptr_t>(out2) % 16 || (ldo2 * 2) % 16 || ldo2 < n)) return false;
    TcEpilogue ep{};
    ep.out2 = out2;
    ep.ldo2 = ldo2;
    ep.rows2 = rows2;
    ep.out = out;
    ep.ldo = n;
    ep.bias = bias;
    ep.relu = relu;
    ep.row_scale = nullptr;
    ep.scale_from = 0;
    ep.m_dev = m_dev;
    ep.status = status;
    return launch_tn(cat, rows, k, k, W, n, k, ep, st);
}

bool tc_linear(const __nv_bfloat16 *A, int64_t rows, int k, const __nv_bfloat16 *B, int n, const float *bias, int relu,
               const __nv_bfloat16 *mask, int64_t ld_mask, __nv_bfloat16 *out, int64_t ldo, const int32_t *m_dev,
               int32_t *status, cudaStream_t st, bool b_is_k_by_n, const TcFuse *fuse)
{
    TcEpilogue ep{};
    if (fuse) {
        ep.fuse = *fuse;
        const TcFuse &f = ep.fuse;
        auto bad = [](const void *p, int64_t ld) { return p && (reinterpret_cast<uintptr_t>(p) % 16 || (ld * 2) % 16); };
        if (bad(f.gate_in, f.ld_gate_in) || bad(f.gate_out, f.ld_gate_out) || bad(f.add_a, f.ld_add_a) || bad(f.add_b, f.ld_add_b))
            return false;
        if ((f.add_a == nullptr) != (f.add_b == nullptr) || (f.gate_in && f.add_a)) return false;
    }
    ep.out = out;
    ep.ldo = ldo;
    ep.bias = bias;
    ep.relu = relu;
    ep.mask = mask;
    ep.ld_mask = ld_mask;
    ep.m_dev = m_dev;
    ep.status = status;
    return b_is_k_by_n ? launch_tn(A, rows, k, k, B, n, n, ep, st, true) : launch_tn(A, rows, k, k, B, n, k, ep, st);
}

bool tc_dcat_backward(const __nv_bfloat16 *dz, int64_t rows, int d_out, const __nv_bfloat16 *W, int two_d_in,
                      const float *inv_cnt, __nv_bfloat16 *dcat, const int32_t *m_dev, int32_t *status, cudaStream_t st,
                      int n_rhs)
{
    TcEpilogue ep{};
    ep.out = dcat;
    ep.ldo = two_d_in;
    ep.bias = nullptr;
    ep.relu = 0;
    ep.row_scale = inv_cnt;
    ep.scale_from = two_d_in / 2;
    ep.m_dev = m_dev;
    ep.status = status;
    return launch_tn(dz, rows, d_out, d_out, W, two_d_in, two_d_in, ep, st, true, n_rhs);
}

}  // namespace e2egrec

namespace e2egrec {

// widest tile of 64 .. 256 columns that divides n (0: none)
static int weight_grad_nt(int n)
{
    for (int c = 256; c >= 64; c -= 64)
        if (n % c == 0) return c;
    return 0;
}

int tc_weight_grad_tiles(int m, int n)
{
    const int nt = weight_grad_nt(n);
    return nt && m >= kTileM ? (m / kTileM) * (n / nt) : 1;
}

bool tc_weight_grad(const __nv_bfloat16 *dY, int64_t rows, int m, const __nv_bfloat16 *Xin, int n, const int32_t *m_dev,
                    float *part, int splits, int32_t *status, cudaStream_t st, int n_rhs)
{
    if (rows <= 0 || rows % kTileK || m % kTileM || n % 64 || n_rhs < 1 || splits < 1) return false;
    const int nt = weight_grad_nt(n);
    if (!nt) return false;
    if (reinterpret_cast<uintptr_t>(dY) % 16 || reinterpret_cast<uintptr_t>(Xin) % 16) return false;
    CUtensorMap my, mx;
    if (!make_map_mn(&my, dY, rows * n_rhs, m) || !make_map_mn(&mx, Xin, rows, n)) return false;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < nt) tmem_cols <<= 1;
    const int stages = 4;
    const size_t smem = (size_t)stages * ((kTileM / 64) + (nt / 64)) * (kTileK * 128) + 1024;
    static bool attr_set[kMaxDevices] = {};
    if (!raise_smem_limit(tc_gemm_rows_kernel, attr_set)) return false;
    dim3 grid((unsigned)(m / kTileM), (unsigned)(n / nt), (unsigned)splits);
    note_launch();
    launch_pdl(tc_gemm_rows_kernel, grid, dim3(kThreads), smem, st, my, mx, nt, tmem_cols, stages, m_dev, part, (int64_t)n,
               (int64_t)m * n, status, n_rhs, rows);
    return true;
}

bool tc_sage_fused_forward(const __nv_bfloat16 *Hsrc, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                           const int32_t *indptr, int d_in, __nv_bfloat16 *cat, int64_t rows, const __nv_bfloat16 *W, int n,
                           const float *bias, int relu, __nv_bfloat16 *out, const int32_t *m_dev, int32_t *status,
                           cudaStream_t st, __nv_bfloat16 *out2, int64_t ldo2, int64_t rows2)
{
    if (rows <= 0 || rows % kTileM || n < 32 || n > 256 || n % 32) return false;
    if (d_in != 64 && d_in != 128 && d_in != 256) return false;
    if (reinterpret_cast<uintptr_t>(Hsrc) % 16 || (ld * 2) % 16 || reinterpret_cast<uintptr_t>(cat) % 16 ||
        reinterpret_cast<uintptr_t>(W) % 16 || reinterpret_cast<uintptr_t>(out) % 16)
        return false;
    if (out2 && (reinterpret_cast<uintptr_t>(out2) % 16 || (ldo2 * 2) % 16 || ldo2 < n)) return false;
    TcEpilogue ep{};
    ep.out = out;
    ep.ldo = n;
    ep.out2 = out2;
    ep.ldo2 = ldo2;
    ep.rows2 = rows2;
    ep.bias = bias;
    ep.relu = relu;
    ep.m_dev = m_dev;
    ep.status = status;
    ep.n_rhs = 1;
    ep.rhs_rows = rows;
    ep.mode = (bias ? kEpiBias : 0) | (relu ? kEpiRelu : 0);
    CUtensorMap mb;
    if (!make_map(&mb, W, n, 2 * d_in, 2 * d_in, n)) return false;
    switch (d_in) {
    case 64: return launch_fused<8>(mb, Hsrc, ld, nbr, self_ids, indptr, cat, rows, n, ep, st);
    case 128: return launch_fused<16>(mb, Hsrc, ld, nbr, self_ids, indptr, cat, rows, n, ep, st);
    default: return launch_fused<32>(mb, Hsrc, ld, nbr, self_ids, indptr, cat, rows, n, ep, st);
    }
}


}  // namespace e2egrec
