// Status strings and error bookkeeping of the C ABI.
#include <atomic>
#include <functional>
#include <mutex>
#include <unordered_map>
#include <vector>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace e2egrec {

static thread_local char g_last_error[256] = "";

void set_last_error(const char *msg)
{
    strncpy(g_last_error, msg ? msg : "", sizeof(g_last_error) - 1);
    g_last_error[sizeof(g_last_error) - 1] = 0;
}

int32_t check_launch(const char *what)
{
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return E2EGREC_OK;
    char buf[256];
    snprintf(buf, sizeof(buf), "%s: %s", what, cudaGetErrorString(e));
    set_last_error(buf);
    return E2EGREC_ERR_CUDA;
}

bool pdl_enabled()
{
    static const bool on = []() {
        const char *v = getenv("E2EGREC_PDL");
        return v && *v && strcmp(v, "0") != 0;
    }();
    return on;
}

static bool helper_streams_enabled()
{
    static const bool on = []() {
        const char *v = getenv("E2EGREC_NO_HELPER_STREAM");
        return !(v && *v && strcmp(v, "0") != 0);
    }();
    return on;
}

// Helper streams: one per (device, caller's stream), created on first use and kept until the process ends, so calls
// made on different streams (a sampling leg beside a compute leg, say) never meet on a common helper stream.
// Deferred work (a block transposition left running by e2egrec_sample_khop) is tracked per device: whichever stream
// of that device asks next (e2egrec_sage_backward, e2egrec_sample_join, the next e2egrec_sample_khop) waits for all of
// it.  The table and the pending lists are guarded by one mutex; the event ring of a helper stream is touched only by
// calls issued on its caller's stream, which the caller must not issue from two host threads at once.
static std::mutex g_side_mutex;
struct SideKey {
    int dev;
    cudaStream_t stream;
    bool operator==(const SideKey &o) const { return dev == o.dev && stream == o.stream; }
};
struct SideKeyHash {
    size_t operator()(const SideKey &k) const { return std::hash<const void *>()(k.stream) * 31u + (size_t)k.dev; }
};
static std::unordered_map<SideKey, SideStream *, SideKeyHash> g_side;
static std::vector<SideStream *> g_pending[64];          // per device: helper streams whose `pending` event is unjoined

SideStream *SideStream::get(cudaStream_t caller)
{
    if (!helper_streams_enabled()) return nullptr;     // every entry point then stays on its caller's stream
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_side_mutex);
    auto it = g_side.find(SideKey{dev, caller});
    if (it != g_side.end()) return it->second;
    SideStream *s = new SideStream();
    s->next = 0;
    s->owner = caller;
    s->device = dev;
    int prio = 0;                                // the helper runs at its caller's priority
    if (cudaStreamGetPriority(caller, &prio) != cudaSuccess) { prio = 0; cudaGetLastError(); }
    if (cudaStreamCreateWithPriority(&s->stream, cudaStreamNonBlocking, prio) != cudaSuccess) { delete s; cudaGetLastError(); return nullptr; }
    for (int i = 0; i < 32; ++i)
        if (cudaEventCreateWithFlags(&s->ev[i], cudaEventDisableTiming) != cudaSuccess) { delete s; cudaGetLastError(); return nullptr; }
    if (cudaEventCreateWithFlags(&s->pending, cudaEventDisableTiming) != cudaSuccess) { delete s; cudaGetLastError(); return nullptr; }
    s->has_pending = false;
    g_side.emplace(SideKey{dev, caller}, s);
    return s;
}

cudaEvent_t SideStream::event() { return ev[(next++) & 31u]; }

void SideStream::fork(cudaStream_t from)
{
    cudaEvent_t e = event();
    cudaEventRecord(e, from);
    cudaStreamWaitEvent(stream, e, 0);
}

void SideStream::join(cudaStream_t into)
{
    cudaEvent_t e = event();
    cudaEventRecord(e, stream);
    cudaStreamWaitEvent(into, e, 0);
}

void SideStream::defer()
{
    std::lock_guard<std::mutex> lock(g_side_mutex);
    cudaEventRecord(pending, stream);
    if (!has_pending) g_pending[device].push_back(this);
    has_pending = true;
}

void SideStream::join_pending(cudaStream_t into)
{
    std::lock_guard<std::mutex> lock(g_side_mutex);
    for (SideStream *s : g_pending[device]) {
        cudaStreamWaitEvent(into, s->pending, 0);
        s->has_pending = false;
    }
    g_pending[device].clear();
}

static std::atomic<uint64_t> g_launches{0};
void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

static thread_local int g_tap_which = 0;
static thread_local cudaEvent_t g_tap_start = nullptr, g_tap_stop = nullptr;

void tap_begin(int which, cudaStream_t st)
{
    if (which == g_tap_which && g_tap_start) cudaEventRecord(g_tap_start, st);
}

void tap_end(int which, cudaStream_t st)
{
    if (which != g_tap_which) return;
    if (g_tap_stop) cudaEventRecord(g_tap_stop, st);
    g_tap_which = 0;
}

}  // namespace e2egrec

extern "C" int32_t e2egrec_sample_join(void *stream)
{
    e2egrec::SideStream *side = e2egrec::SideStream::get(static_cast<cudaStream_t>(stream));
    if (side) side->join_pending(static_cast<cudaStream_t>(stream));
    return e2egrec::check_launch("sample_join");
}

extern "C" uint64_t e2egrec_launch_count(void) { return e2egrec::g_launches.load(std::memory_order_relaxed); }

extern "C" int32_t e2egrec_profile_tap(int32_t which, void *start_event, void *stop_event)
{
    if (which < 0 || which > e2egrec::TAP_LAST) return E2EGREC_ERR_ARG;
    if (which && (!start_event || !stop_event)) return E2EGREC_ERR_NULL;
    e2egrec::g_tap_which = which;
    e2egrec::g_tap_start = static_cast<cudaEvent_t>(start_event);
    e2egrec::g_tap_stop = static_cast<cudaEvent_t>(stop_event);
    return E2EGREC_OK;
}

extern "C" const char *e2egrec_status_string(int32_t code)
{
    switch (code) {
    case E2EGREC_OK: return "ok";
    case E2EGREC_ERR_NULL: return "a required pointer is NULL";
    case E2EGREC_ERR_ARG: return "argument out of range";
    case E2EGREC_ERR_DTYPE: return "unknown or mismatched dtype";
    case E2EGREC_ERR_ALIGN: return "pointer or row not 16-byte aligned";
    case E2EGREC_ERR_WORKSPACE: return "buffer smaller than required";
    case E2EGREC_ERR_UNSUPPORTED: return "size beyond the supported limits";
    case E2EGREC_ERR_CUDA: return "CUDA launch failed";
    default: return "unknown status";
    }
}

extern "C" const char *e2egrec_last_error(void) { return e2egrec::g_last_error; }
