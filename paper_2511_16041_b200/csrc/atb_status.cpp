// Status strings, per-thread error detail and the plane-size helpers of the C ABI.
#include <cstring>

#include "atb_internal.h"

namespace atb {
namespace {
thread_local char g_message[512] = "";
}

atb_status_t fail(atb_status_t status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_message, sizeof g_message, fmt, ap);
    va_end(ap);
    return status;
}

void clear_error() { g_message[0] = '\0'; }
}  // namespace atb

extern "C" {

const char* atb_status_string(atb_status_t s) {
    switch (s) {
        case ATB_OK: return "ATB_OK";
        case ATB_ERR_NULL_POINTER: return "ATB_ERR_NULL_POINTER";
        case ATB_ERR_BAD_SHAPE: return "ATB_ERR_BAD_SHAPE";
        case ATB_ERR_BAD_TILING: return "ATB_ERR_BAD_TILING";
        case ATB_ERR_MISALIGNED: return "ATB_ERR_MISALIGNED";
        case ATB_ERR_UNSUPPORTED_DEVICE: return "ATB_ERR_UNSUPPORTED_DEVICE";
        case ATB_ERR_CUDA: return "ATB_ERR_CUDA";
        case ATB_ERR_BUFFER_TOO_SMALL: return "ATB_ERR_BUFFER_TOO_SMALL";
        case ATB_ERR_DEVICE_TIMEOUT: return "ATB_ERR_DEVICE_TIMEOUT";
    }
    return "ATB_ERR_UNKNOWN";
}

const char* atb_last_error_message(void) { return atb::g_message; }

size_t atb_bfp16_mant_bytes(int64_t M, int64_t K) {
    if (M <= 0 || K <= 0) return 0;
    return static_cast<size_t>(M) * static_cast<size_t>(K);
}

size_t atb_bfp16_exp_bytes(int64_t M, int64_t K) {
    if (M <= 0 || K <= 0) return 0;
    return static_cast<size_t>(atb::ceil_div(K, 64)) * static_cast<size_t>(atb::round_up(M, 32)) * 8u;
}

}  // extern "C"
