// Host-side argument validation shared by the entry points.
#pragma once
#include <cstdint>
#include <cstring>
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/wushkv.h"
#include "layout.cuh"

namespace wushkv {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Checks the cache description and fills the device-side view.  Returns WUSHKV_OK or WUSHKV_EINVAL / ECAPACITY.
inline int make_view(const wushkv_cache* c, CacheView& v) {
    if (!c) return WUSHKV_EINVAL;
    if (c->d != D || c->page_tokens != PAGE_TOKENS) return WUSHKV_EINVAL;
    if (c->bits != 2 && c->bits != 3 && c->bits != 4) return WUSHKV_EINVAL;
    if (c->n_kv <= 0 || c->n_q <= 0 || c->n_q % c->n_kv != 0) return WUSHKV_EINVAL;
    const int G = c->n_q / c->n_kv;
    if (G < 1 || G > 8) return WUSHKV_EINVAL;
    if (c->s_sink < 0 || c->s_keep < 1 || c->s_flush < 1 || c->boundary_lag < 0) return WUSHKV_EINVAL;
    if (c->n_slots <= 0 || c->max_pages <= 0 || c->n_pages <= 0) return WUSHKV_EINVAL;
    if (!(c->kappa_k >= 0.f && c->kappa_k <= 1.f) || !(c->kappa_v >= 0.f && c->kappa_v <= 1.f)) return WUSHKV_EINVAL;
    if (!(c->sm_scale > 0.f)) return WUSHKV_EINVAL;
    if (c->quantizer != WUSHKV_QUANTIZER_AFFINE && c->quantizer != WUSHKV_QUANTIZER_QUEST) return WUSHKV_EINVAL;
    if (!c->pages || !c->page_table || !c->ring_kv || !c->T_K || !c->T_K_invT || !c->dev_status) return WUSHKV_EINVAL;
    if (c->s_sink > 0 && !c->sink_kv) return WUSHKV_EINVAL;
    if (!aligned(c->pages, 256) || !aligned(c->ring_kv, 16) || !aligned(c->sink_kv, 16) || !aligned(c->T_K, 16) ||
        !aligned(c->T_K_invT, 16) || !aligned(c->page_table, 4) || !aligned(c->dev_status, 4))
        return WUSHKV_EINVAL;
    if (c->ring_cap < c->s_keep + c->s_flush - 1 + c->boundary_lag) return WUSHKV_ECAPACITY;
    v.n_q = c->n_q; v.n_kv = c->n_kv; v.bits = c->bits;
    v.s_sink = c->s_sink; v.s_keep = c->s_keep; v.s_flush = c->s_flush; v.lag = c->boundary_lag;
    v.n_slots = c->n_slots; v.max_pages = c->max_pages; v.ring_cap = c->ring_cap; v.G = G;
    v.n_pages = c->n_pages;
    v.pages = static_cast<unsigned char*>(c->pages);
    v.page_table = c->page_table;
    v.sink_kv = static_cast<unsigned short*>(c->sink_kv);
    v.ring_kv = static_cast<unsigned short*>(c->ring_kv);
    v.T_K = c->T_K; v.T_K_invT = c->T_K_invT;
    v.dev_status = c->dev_status;
    v.sm_scale = c->sm_scale;
    return WUSHKV_OK;
}

// Testing aids (wushkv_set_test_option).  The environment is read once, when the first call needs a
// knob; afterwards only the setter changes them.  Process-global, not synchronised.
struct Knobs {
    long long decode_ctas = 0;      // > 0: number of thread blocks of the decode main kernel (the split count)
    int append_path_cuda = 0;       // 1: chunks take the CUDA-core append path
    int host_io_copy = 0;           // 1: wushkv_decode_step_host stages its buffers with copies even when they are mapped
    long long drop_copy_unit = -1;  // >= 0: the decode main kernel never issues the copy of this unit of the flattened list
    long long wait_limit = 0;       // > 0: poll limit of the device-side barrier waits (default: about a second)
    int drop_chunk_mma = 0;         // 1: the chunk append never commits its first tile's MMAs to the barrier
    int prefill_legacy = 0;         // 1: chunk attention on the mma.sync kernel instead of the tcgen05 one
    int prefill_one_tile = 0;       // 1: chunk attention on the tcgen05 kernel with one query tile per CTA (no role split) instead of the warp-specialised one
    int prefill_split = 0;          // > 0: CTAs per tile pair of the warp-specialised chunk attention (capped by what the workspace holds); 0: chosen by the grid size
    int prefill_no_tma = 0;         // 1: the tcgen05 kernel stages the chunk's tiles with 16-byte copies instead of bulk tensor copies
    int drop_prefill = 0;           // chunk attention: 1 the first tile's score MMAs are never committed, 2 one bulk copy is never issued, 3 one bulk copy of the transform kernel is never issued
    int append_no_tma = 0;          // 1: the chunk append stages its tiles with 16-byte copies instead of bulk tensor copies
};
Knobs& knobs();

// Opts a kernel in to `bytes` of dynamic shared memory, once per (kernel, device).  Concurrent first calls
// may both set the attribute (same value: harmless).
inline bool opt_in_dynamic_smem(const void* fn, int bytes) {
    struct Entry { const void* fn; unsigned long long devs; };
    static Entry table[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool dev_ok = dev >= 0 && dev < 64;
    for (Entry& e : table) {
        if (e.fn != fn && e.fn != nullptr) continue;
        if (e.fn == fn && dev_ok && ((e.devs >> dev) & 1ull)) return true;
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
        e.fn = fn;
        if (dev_ok) e.devs |= 1ull << dev;
        return true;
    }
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// Tensor map of a 16-bit row tensor [rows][n_heads][128 channels]: boxes of box_rows x 64 channels (128 bytes), written to
// shared memory as 128-byte-swizzled rows.  Coordinates of a copy: (channel 0 or 64, head, first row).  False when the
// driver entry point is missing or refuses (callers then stage with 16-byte copies).
inline bool make_row_tensor_map(CUtensorMap& map, bool bf16, const void* base, int n_heads, long long rows, int box_rows, int box_heads = 1) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) fn = nullptr;
        return reinterpret_cast<EncodeFn>(fn);
    }();
    std::memset(&map, 0, sizeof(map));
    if (!encode || rows <= 0 || n_heads <= 0) return false;
    const cuuint64_t gdim[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(n_heads), static_cast<cuuint64_t>(rows)};
    const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(n_heads) * D * 2};
    const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_heads), static_cast<cuuint32_t>(box_rows)}, estr[3] = {1, 1, 1};
    return encode(&map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int sm_count() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return 148;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
        cached = n;
    }
    return cached;
}

}  // namespace wushkv
