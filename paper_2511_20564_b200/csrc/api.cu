// Status strings and error bookkeeping of the C ABI.
#include <atomic>
#include <stdio.h>
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
