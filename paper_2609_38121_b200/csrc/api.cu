// Small host-only entry points of the C ABI.
#include "host_common.h"

extern "C" size_t wushkv_page_bytes(int32_t n_kv, int32_t d, int32_t bits, int32_t page_tokens) {
    if (n_kv <= 0 || d != wushkv::D || page_tokens != wushkv::PAGE_TOKENS || (bits != 2 && bits != 4)) return 0;
    return static_cast<size_t>(n_kv) * wushkv::record_bytes(bits);
}

extern "C" const char* wushkv_status_string(int status) {
    switch (status) {
        case WUSHKV_OK: return "ok";
        case WUSHKV_EINVAL: return "invalid argument";
        case WUSHKV_ENOTPD: return "damped Gram or Hessian matrix is not positive definite";
        case WUSHKV_ECUDA: return "CUDA runtime or launch error";
        case WUSHKV_ECAPACITY: return "workspace, ring buffer or page table too small";
        default: return "unknown status";
    }
}
