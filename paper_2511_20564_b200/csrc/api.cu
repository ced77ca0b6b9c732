// Status strings and error bookkeeping of the C ABI.
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

}  // namespace e2egrec

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
