// Small host-only entry points of the C ABI.
#include <cstdlib>
#include <cstring>

#include "host_common.h"

namespace wushkv {

Knobs& knobs() {
    static Knobs k = [] {
        Knobs v;
        if (const char* e = std::getenv("WUSHKV_DECODE_CTAS")) v.decode_ctas = std::atoll(e);
        if (const char* e = std::getenv("WUSHKV_APPEND_PATH")) v.append_path_cuda = e[0] == 'c';
        if (const char* e = std::getenv("WUSHKV_HOST_IO")) v.host_io_copy = e[0] == 'c';
        return v;
    }();
    return k;
}

}  // namespace wushkv

extern "C" int wushkv_set_test_option(const char* name, long long value) {
    if (!name) return WUSHKV_EINVAL;
    wushkv::Knobs& k = wushkv::knobs();
    if (!std::strcmp(name, "decode_ctas")) k.decode_ctas = value;
    else if (!std::strcmp(name, "append_path_cuda")) k.append_path_cuda = value != 0;
    else if (!std::strcmp(name, "host_io_copy")) k.host_io_copy = value != 0;
    else if (!std::strcmp(name, "drop_copy_unit")) k.drop_copy_unit = value;
    else if (!std::strcmp(name, "wait_limit")) k.wait_limit = value;
    else if (!std::strcmp(name, "drop_chunk_mma")) k.drop_chunk_mma = value != 0;
    else if (!std::strcmp(name, "prefill_legacy")) k.prefill_legacy = value != 0;
    else if (!std::strcmp(name, "prefill_no_tma")) k.prefill_no_tma = value != 0;
    else if (!std::strcmp(name, "prefill_one_tile")) k.prefill_one_tile = value != 0;
    else if (!std::strcmp(name, "prefill_split")) k.prefill_split = static_cast<int>(value);
    else if (!std::strcmp(name, "append_no_tma")) k.append_no_tma = value != 0;
    else if (!std::strcmp(name, "drop_prefill")) k.drop_prefill = static_cast<int>(value);
    else return WUSHKV_EINVAL;
    return WUSHKV_OK;
}

extern "C" size_t wushkv_page_bytes(int32_t n_kv, int32_t d, int32_t bits, int32_t page_tokens) {
    if (n_kv <= 0 || d != wushkv::D || page_tokens != wushkv::PAGE_TOKENS || (bits != 2 && bits != 3 && bits != 4)) return 0;
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
