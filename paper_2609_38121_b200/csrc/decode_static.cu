// Decode attention for callers that are not allowed to allocate device memory.
//
// Who that is: code that runs where cudaMalloc is off limits or would fail - a serving loop whose
// framework reserved all device memory for its own pool at start-up, a plug-in that was handed
// fixed input / output buffers by its host application and nothing else, or a latency-critical
// section where an allocation's implicit device synchronisation is not acceptable.  Such a caller
// has nowhere to get the workspace that wushkv_decode_attn asks for, so this entry point brings
// its own: a fixed array that lives in the library's device image.
//
// The array is part of every CUDA context that loads the library (WUSHKV_STATIC_SCRATCH_BYTES of
// device memory per GPU, held until the process exits), which is why it is kept modest and why
// larger requests are refused rather than served some other way.
#include <cuda_runtime.h>

#include "../../include/wushkv.h"

static __device__ __align__(256) unsigned char g_static_scratch[WUSHKV_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch on each GPU.  In host code the name g_static_scratch is only
// a handle for the runtime, not a device address, so the address is looked up once per device
// (with that device current) and remembered here.
void* g_scratch_addr[kMaxDevices] = {};

}  // namespace

namespace wushkv {
// Never launched; it names the array from device code so that the array is always part of the
// device image, whatever the compiler decides about variables only the host refers to.
__global__ void static_scratch_anchor(unsigned char* out) {
    if (out != nullptr) out[0] = g_static_scratch[0];
}
}  // namespace wushkv

extern "C" int wushkv_decode_attn_static(const wushkv_cache* cache, int32_t batch, const int32_t* slot,
                                         const int32_t* seq_len, int32_t max_seq_len, const uint16_t* Q, float* O,
                                         void* stream) {
    const size_t need = wushkv_decode_workspace_bytes(cache, batch, max_seq_len);
    if (need == 0) return WUSHKV_EINVAL;                        // bad cache description or sizes
    if (need > WUSHKV_STATIC_SCRATCH_BYTES) return WUSHKV_ECAPACITY;   // beyond the built-in scratch: use wushkv_decode_attn
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return WUSHKV_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return WUSHKV_EINVAL;
    if (g_scratch_addr[dev] == nullptr) {                       // first call on this device: resolve the symbol
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return WUSHKV_ECUDA;
        g_scratch_addr[dev] = p;
    }
    // Nothing in the scratch has to start at zero: every partial that the combine pass reads is
    // written by the main kernel of the same call, so the previous call's leftovers are never seen.
    return wushkv_decode_attn(cache, batch, slot, seq_len, max_seq_len, Q, O, g_scratch_addr[dev],
                              WUSHKV_STATIC_SCRATCH_BYTES, stream);
}
