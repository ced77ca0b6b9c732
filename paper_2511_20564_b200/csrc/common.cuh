// Shared device/host helpers of the e2egrec kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/e2egrec.h"

namespace e2egrec {

// indices into e2egrec_block::counts
enum { CNT_DST = 0, CNT_SRC = 1, CNT_EDGES = 2, CNT_STATUS = 3 };

constexpr int kMaxHops = 4;
constexpr int kMaxFanout = 128;
constexpr int kMaxDim = 1024;

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

inline size_t dtype_size(int32_t dtype) { return dtype == E2EGREC_BF16 ? 2 : 4; }

// host side: remember the text of a failed launch for e2egrec_last_error()
void set_last_error(const char *msg);
int32_t check_launch(const char *what);
// host side: one helper stream per device and caller's stream for work that may overlap the caller's stream
// inside one entry point.  fork() makes the helper stream wait for what the caller's stream has enqueued so far; join()
// makes the caller's stream wait for the helper stream.  Both are plain event record / wait pairs, so they
// are legal inside a stream capture.  get() returns nullptr if the stream cannot be created (the caller
// then stays on its own stream).  defer() leaves the helper stream's work unjoined and notes it for the device;
// join_pending() makes a stream wait for everything deferred on this helper's device, whichever stream deferred it.
struct SideStream {
    cudaStream_t stream;
    cudaStream_t owner;           // the caller's stream this helper belongs to
    int device;
    cudaEvent_t ev[32];
    unsigned next;
    cudaEvent_t pending;          // end of helper-stream work that a later entry point has to wait for
    bool has_pending;
    static SideStream *get(cudaStream_t caller);
    void defer();                 // remember the helper stream's current end as pending work of the device
    void join_pending(cudaStream_t into);   // `into` waits for all pending work of this helper's device
    cudaEvent_t event();
    void fork(cudaStream_t from);
    void join(cudaStream_t into);
};
// host side: every kernel launch is counted (e2egrec_launch_count)
void note_launch();
// host side: true when the environment variable E2EGREC_PDL is set to a non-empty value other than "0"
bool pdl_enabled();

// Launch, optionally (E2EGREC_PDL=1) with programmatic stream serialization: the kernel's blocks may then become
// resident while the kernel before it in the stream is still finishing, so that its set-up (and the launch latency)
// overlaps that kernel's tail.  Off by default: measured on B200 inside a step whose three legs run on three streams,
// the early-resident blocks (a persistent product holds ~200 KB of shared memory per SM while it waits) keep the
// other legs' kernels off the SMs and the step gets slower (0.126 -> 0.148 ms on the 20 M-entry workload).  Only for
// kernels that call pdl_wait() in every thread before they touch global memory: the wait returns once the
// preceding kernel has completed and its writes are visible, which makes the pair behave like an ordinary dependent
// launch.  Kernels launched this way call pdl_launch_dependents() first, so that their own successor is admitted early.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// host side: timing taps (e2egrec_profile_tap).  tap_begin/tap_end record the armed events around
// kernel group `which` and disarm the tap.
enum { TAP_AGG_FWD_OUTER = 1, TAP_AGG_BWD_OUTER = 2, TAP_UPDATE_FWD_OUTER = 3, TAP_DW_OUTER = 4, TAP_DCAT_OUTER = 5,
       TAP_SAMPLE = 6, TAP_SEG_L1 = 7, TAP_SEG_L3 = 9, TAP_LAST = 9 };   // 8 is unused
void tap_begin(int which, cudaStream_t st);
void tap_end(int which, cudaStream_t st);

// ---------------------------------------------------------------------------------------
// 16-byte row chunks: 8 bf16 or 4 fp32 values, accumulated in fp32.
// ---------------------------------------------------------------------------------------
template <typename T> struct Chunk;

template <> struct Chunk<float> {
    static constexpr int kElems = 4;
    __device__ static inline uint4 load_raw(const float *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
    __device__ static inline void unpack(const uint4 &r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
    __device__ static inline void load(const float *p, float (&v)[4]) {
        float4 r = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = r.x; v[1] = r.y; v[2] = r.z; v[3] = r.w;
    }
    __device__ static inline void store(float *p, const float (&v)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};

template <> struct Chunk<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static inline uint4 load_raw(const __nv_bfloat16 *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
    __device__ static inline void unpack(const uint4 &r, float (&v)[8]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static inline void load(const __nv_bfloat16 *p, float (&v)[8]) {
        uint4 r = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {           // bf16 -> fp32 is a 16-bit shift
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static inline void store(__nv_bfloat16 *p, const float (&v)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);   // round to nearest even
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// Two fp32 adds in one instruction (packed f32x2 of sm_100): the same round-to-nearest result per element as
// two scalar adds, at half the issue slots.  Through the compiler's builtin, so that it can keep the operands in
// aligned register pairs instead of packing and unpacking them around the instruction.
__device__ __forceinline__ void add2(float &a0, float &a1, float b0, float b1)
{
    const float2 r = __fadd2_rn(make_float2(a0, a1), make_float2(b0, b1));
    a0 = r.x;
    a1 = r.y;
}
template <typename T> __device__ inline float to_float(T v);
template <> __device__ inline float to_float<float>(float v) { return v; }
template <> __device__ inline float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ inline T from_float(float v);
template <> __device__ inline float from_float<float>(float v) { return v; }
template <> __device__ inline __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

}  // namespace e2egrec
