// Mean aggregation of a sampled block (Eq. 2) for 512-byte rows with a private TMA ring per warp (sm_100a).
//
// A warp owns destinations [i0, i1) and therefore entries [b, e) of the block's neighbour list.  Group q of its entries
// (b + 4q .. b + 4q + 3) is fetched by one cp.async.bulk.tensor tile::gather4 into slot q mod kNbrSlots of the warp's
// ring; an mbarrier per slot counts the bytes in.  The warp issues kNbrSlots groups ahead, consumes the groups in order
// (rows are added in entry order, one fp32 partial per lane and 16-byte piece, exactly as sage_aggregate_kernel adds them
// for rows of 32 pieces), closes a destination whenever the next entry lies beyond its end, and refills a slot as soon as
// it has read it.  The self rows come the same way, four destinations per gather, through a second small ring.  The
// neighbour ids, the destinations' end offsets and their self ids are read 32 at a time, one per lane, one window ahead.
// Nothing is shared between warps, so there is no protocol between them: a warp waits only for bytes it asked for itself.
// Every wait is bounded; when one runs out the warp raises E2EGREC_DEV_TIMEOUT, waits (bounded) for its copies in flight
// and leaves.
#include "gather_stream.cuh"

#include "tensor_map.cuh"

#include <algorithm>

namespace e2egrec {

namespace {

constexpr int kD = 256;                       // values per row
constexpr uint32_t kRowBytes = kD * 2, kSlotBytes = 4 * kRowBytes;

// 32 consecutive values of an int32 array, one per lane, positions at or beyond `limit` repeating the last valid one
// (limit > first); two such windows (the current and the next) are kept in registers.
__device__ inline int32_t load_window(const int32_t *__restrict__ a, int64_t first, int64_t limit, int lane)
{
    const int64_t k = first + lane;
    return a[k < limit ? k : limit - 1];
}

// kWarps warps per block, each with kNbrSlots groups of four neighbour rows and kSelfSlots groups of four self rows in flight
template <int kWarps, int kNbrSlots, int kSelfSlots>
__global__ void __launch_bounds__(kWarps * 32, 1)
sage_aggregate_stream_kernel(const __grid_constant__ CUtensorMap map, const int32_t *__restrict__ nbr,
                             const int32_t *__restrict__ self_ids, const int32_t *__restrict__ indptr,
                             int32_t *__restrict__ counts, __nv_bfloat16 *__restrict__ cat, int32_t cap_dst)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_n[kWarps][kNbrSlots], bar_s[kWarps][kSelfSlots];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint8_t *ring_n = ring + (size_t)warp * (kNbrSlots + kSelfSlots) * kSlotBytes;
    uint8_t *ring_s = ring_n + (size_t)kNbrSlots * kSlotBytes;
    if (lane == 0) {
        for (int s = 0; s < kNbrSlots; ++s) tm_mbar_init(&bar_n[warp][s], 1);
        for (int s = 0; s < kSelfSlots; ++s) tm_mbar_init(&bar_s[warp][s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const int32_t n_dst = counts[CNT_DST];
    int64_t pad_end = ((int64_t)n_dst + 127) / 128 * 128;
    if (pad_end > cap_dst) pad_end = cap_dst;
    const int64_t total_warps = (int64_t)gridDim.x * kWarps, gw = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t per = (pad_end + total_warps - 1) / total_warps;
    const int64_t i0 = min(gw * per, pad_end), i1 = min(i0 + per, pad_end);
    const int64_t j0 = min(i0, (int64_t)n_dst), j1 = min(i1, (int64_t)n_dst);      // the destinations that exist
    const int32_t b_w = indptr[j0], e_w = indptr[j1];
    const int32_t n_groups = (e_w - b_w + 3) >> 2, n_self = (int32_t)((j1 - j0 + 3) >> 2);
    const uint32_t full = 0xffffffffu;

    // windows of 32: neighbour ids (window w = entries b_w + 32 w ..), end offsets and self ids (window w = destinations j0 + 32 w ..)
    int32_t ids_cur = 0, ids_next = 0, ends_cur = 0, ends_next = 0, self_cur = 0, self_next = 0;
    int id_win = 0, dst_win = 0;
    auto load_ids = [&](int w) { return n_groups > 0 ? load_window(nbr, (int64_t)b_w + 32 * w, e_w, lane) : 0; };
    auto load_ends = [&](int w) { return j1 > j0 ? load_window(indptr + 1, j0 + 32 * w, j1, lane) : 0; };
    auto load_self = [&](int w) -> int32_t {
        if (j1 <= j0) return 0;
        if (self_ids) return load_window(self_ids, j0 + 32 * w, j1, lane);
        const int64_t k = j0 + 32 * w + lane;
        return (int32_t)(k < j1 ? k : j1 - 1);
    };
    ids_cur = load_ids(0);
    ids_next = load_ids(1);
    ends_cur = load_ends(0);
    ends_next = load_ends(1);
    self_cur = load_self(0);
    self_next = load_self(1);

    int32_t issued_n = 0, issued_s = 0;
    auto issue_nbr = [&](int32_t q) {              // all lanes; window q / 8 is the current or the next one
        const int32_t w = (q >> 3) == id_win ? ids_cur : ids_next;
        const int s = (q & 7) * 4;
        const int r0 = __shfl_sync(full, w, s), r1 = __shfl_sync(full, w, s + 1), r2 = __shfl_sync(full, w, s + 2),
                  r3 = __shfl_sync(full, w, s + 3);
        if (lane == 0) tm_gather4(ring_n + (size_t)(q % kNbrSlots) * kSlotBytes, &map, r0, r1, r2, r3, &bar_n[warp][q % kNbrSlots], kRowBytes);
        issued_n = q + 1;
    };
    auto issue_self = [&](int32_t g) {
        const int32_t w = (g >> 3) == dst_win ? self_cur : self_next;
        const int s = (g & 7) * 4;
        const int r0 = __shfl_sync(full, w, s), r1 = __shfl_sync(full, w, s + 1), r2 = __shfl_sync(full, w, s + 2),
                  r3 = __shfl_sync(full, w, s + 3);
        if (lane == 0) tm_gather4(ring_s + (size_t)(g % kSelfSlots) * kSlotBytes, &map, r0, r1, r2, r3, &bar_s[warp][g % kSelfSlots], kRowBytes);
        issued_s = g + 1;
    };
    for (int32_t q = 0; q < n_groups && q < kNbrSlots; ++q) issue_nbr(q);
    for (int32_t g = 0; g < n_self && g < kSelfSlots; ++g) issue_self(g);

    bool ok = true;
    int64_t i = j0;                                 // the destination being summed
    int32_t beg_i = b_w, end_i = j1 > j0 ? __shfl_sync(full, ends_cur, 0) : b_w;
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;

    // closes destination i: mean row and self row to cat[i], then on to destination i + 1
    auto finalize = [&]() {
        __nv_bfloat16 *out = cat + i * 2 * kD;
        const int32_t m = end_i - beg_i;
        const float inv = m > 0 ? 1.0f / (float)m : 0.0f;
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] *= inv;
        Chunk<__nv_bfloat16>::store(out + kD + lane * 8, acc);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;
        const int32_t o = (int32_t)(i - j0), g = o >> 2, slot = g % kSelfSlots;
        ok = ok && __all_sync(full, tm_mbar_wait(&bar_s[warp][slot], (uint32_t)(g / kSelfSlots) & 1u));
        if (ok) {
            *reinterpret_cast<uint4 *>(out + lane * 8) =
                *reinterpret_cast<const uint4 *>(ring_s + (size_t)slot * kSlotBytes + (o & 3) * kRowBytes + lane * 16);
            if ((o & 3) == 3 || i == j1 - 1) {      // the slot's last destination: refill it
                __syncwarp();
                if (g + kSelfSlots < n_self) issue_self(g + kSelfSlots);
            }
        }
        ++i;
        beg_i = end_i;
        end_i = 0x7fffffff;                         // beyond the last destination, or after a wait that ran out: no entry closes anything
        if (i < j1 && ok) {
            const int32_t o2 = (int32_t)(i - j0);
            if ((o2 >> 5) > dst_win) {
                ++dst_win;
                ends_cur = ends_next;
                self_cur = self_next;
                ends_next = load_ends(dst_win + 1);
                self_next = load_self(dst_win + 1);
            }
            end_i = __shfl_sync(full, ends_cur, o2 & 31);
        }
    };

    int32_t q = 0;
    for (; q < n_groups && ok; ++q) {
        if ((q >> 3) > id_win) {
            ++id_win;
            ids_cur = ids_next;
            ids_next = load_ids(id_win + 1);
        }
        const int slot = q % kNbrSlots;
        ok = __all_sync(full, tm_mbar_wait(&bar_n[warp][slot], (uint32_t)(q / kNbrSlots) & 1u));
        if (!ok) break;
        const uint8_t *rows = ring_n + (size_t)slot * kSlotBytes + lane * 16;
        const int32_t k0 = b_w + 4 * q;
        auto add_row = [&](int r) {
            while (k0 + r >= end_i) finalize();     // the entry belongs to a later destination: close the ones before it
            float x[8];
            Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4 *>(rows + r * kRowBytes), x);
#pragma unroll
            for (int kk = 0; kk < 8; kk += 2) add2(acc[kk], acc[kk + 1], x[kk], x[kk + 1]);
        };
        if (k0 + 4 <= e_w) {
#pragma unroll
            for (int r = 0; r < 4; ++r) add_row(r);
        } else {                                    // the stream's last group: rows beyond its end repeat the last id
            for (int r = 0; k0 + r < e_w; ++r) add_row(r);
        }
        __syncwarp();                               // every lane has read the slot
        if (q + kNbrSlots < n_groups) issue_nbr(q + kNbrSlots);
    }
    while (ok && i < j1) finalize();

    // rows between the last destination and the end of its 128-row tile
    for (int64_t ii = max(i0, (int64_t)n_dst); ii < i1; ++ii) {
        __nv_bfloat16 *out = cat + ii * 2 * kD;
        *reinterpret_cast<uint4 *>(out + lane * 8) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(out + kD + lane * 8) = make_uint4(0, 0, 0, 0);
    }

    if (!ok) {
        // a wait ran out: report it, and let the copies that were started land before the shared memory is released
        if (lane == 0) atomicOr(reinterpret_cast<unsigned *>(&counts[CNT_STATUS]), E2EGREC_DEV_TIMEOUT);
        for (int32_t p = max(0, issued_n - kNbrSlots); p < issued_n; ++p) tm_mbar_wait(&bar_n[warp][p % kNbrSlots], (uint32_t)(p / kNbrSlots) & 1u);
        for (int32_t p = max(0, issued_s - kSelfSlots); p < issued_s; ++p) tm_mbar_wait(&bar_s[warp][p % kSelfSlots], (uint32_t)(p / kSelfSlots) & 1u);
    }
}

template <int kWarps, int kNbrSlots, int kSelfSlots>
bool launch_stream(const CUtensorMap &map, const int32_t *nbr, const int32_t *self_ids, const int32_t *indptr, const int32_t *counts,
                   __nv_bfloat16 *cat, int64_t cap_dst, cudaStream_t st)
{
    constexpr size_t smem = (size_t)kWarps * (kNbrSlots + kSelfSlots) * kSlotBytes + 128;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(sage_aggregate_stream_kernel<kWarps, kNbrSlots, kSelfSlots>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return false;
        attr_set[dev] = true;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    // at least 32 destinations per warp; one block per SM at most
    const int64_t blocks = std::max<int64_t>(1, std::min<int64_t>(sms, (cap_dst + kWarps * 32 - 1) / (kWarps * 32)));
    note_launch();
    sage_aggregate_stream_kernel<kWarps, kNbrSlots, kSelfSlots><<<(unsigned)blocks, kWarps * 32, smem, st>>>(
        map, nbr, self_ids, indptr, const_cast<int32_t *>(counts), cat, (int32_t)cap_dst);
    return true;
}

}  // namespace

bool stream_sage_aggregate(const __nv_bfloat16 *Hsrc, int64_t src_rows, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                           const int32_t *indptr, const int32_t *counts, __nv_bfloat16 *cat, int d, int64_t cap_dst,
                           cudaStream_t st)
{
    if (d != kD) return false;
    if (src_rows <= 0 || src_rows > 0x7fffffffll || cap_dst <= 0 || cap_dst > 0x7fffffffll) return false;
    if (reinterpret_cast<uintptr_t>(cat) % 16) return false;
    CUtensorMap map;
    if (!make_row_gather_map(&map, Hsrc, src_rows, kD, ld)) return false;
    // 24 warps, each with two groups of neighbour rows and one of self rows in flight (144 KB of shared memory): measured
    // against 16 x (4 + 2), 20 / 24 / 28 x (3 + 1), 28 / 32 x (2 + 1) and 8 / 12 warps with deeper rings on the outer block of
    // the 2 * 10^9-entry workload (0.232 .. 0.483 ms; this one 0.240, and the smallest footprint among the fast ones).
    return launch_stream<24, 2, 1>(map, nbr, self_ids, indptr, counts, cat, cap_dst, st);
}

}  // namespace e2egrec
