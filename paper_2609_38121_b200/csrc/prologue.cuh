// Normalisation and rotary embedding ahead of the transform (Algorithm 2 lines 1-2), applied to a
// projected key or query vector at the point where a kernel has just loaded it, so that the
// projected form is read once and the normalised, rotated form never goes through memory.
//
// Arithmetic: fp32 throughout, ONE rounding to bf16 at the end (the activation format the transform
// then consumes exactly).  Headwise RMS normalisation x / sqrt(mean(x^2) + eps) times a per-channel
// weight; rotation of the channel pair (j, j + 64) by position * theta^(-2j/128), with the cosines
// and sines read from a table built once in double precision (wushkv_build_rope_table).
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

#include "../../include/wushkv.h"
#include "layout.cuh"

namespace wushkv {

struct Prologue {
    const float2* rope;      // [n_pos][64] (cos, sin); nullptr: the inputs are already normalised and rotated
    int n_pos;
    int normalise;           // 1: RMS normalisation ahead of the rotation
    const float* weight;     // [heads][128] per-channel weights of the normalisation, or nullptr (ones)
    float eps;
};

__device__ __forceinline__ float prologue_bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// A position beyond the table is flagged and clamped (the vector is then rotated by the wrong angle).
__device__ __forceinline__ int prologue_position(const Prologue& pro, int pos, int* dev_status, bool reporter) {
    if (pos >= pro.n_pos || pos < 0) {
        if (reporter) atomicOr(dev_status, WUSHKV_DEV_ROPE_RANGE);
        pos = min(max(pos, 0), pro.n_pos - 1);
    }
    return pos;
}

// Warp-wide form: lane L holds channels 4L..4L+3 of one head vector in x[0..3].  This form takes what it needs from
// memory as arguments (w: the lane's four weights, read only if pro.weight is set; cs0, cs1: (cos, sin) of the lane's
// four channel pairs), so that a caller with several vectors can have their loads in flight together.
__device__ __forceinline__ void norm_rope_warp_loaded(float (&x)[4], int lane, const Prologue& pro, const float4& w,
                                                      const float4& cs0, const float4& cs1) {
    if (pro.normalise) {
        float ss = fmaf(x[0], x[0], fmaf(x[1], x[1], fmaf(x[2], x[2], x[3] * x[3])));
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const float r = ss > 0.f ? 1.f / sqrtf(ss * (1.f / D) + pro.eps) : 0.f;
        if (pro.weight) {
            x[0] *= r * w.x; x[1] *= r * w.y; x[2] *= r * w.z; x[3] *= r * w.w;
        } else {
            x[0] *= r; x[1] *= r; x[2] *= r; x[3] *= r;
        }
    }
    const float c[4] = {cs0.x, cs0.z, cs1.x, cs1.z}, s[4] = {cs0.y, cs0.w, cs1.y, cs1.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float other = __shfl_xor_sync(0xffffffffu, x[e], 16);
        // lanes 0-15 hold the pair's first member a (a c - b s), lanes 16-31 its second member b (a s + b c)
        const float y = lane < 16 ? fmaf(x[e], c[e], -other * s[e]) : fmaf(other, s[e], x[e] * c[e]);
        x[e] = prologue_bf16_round(y);
    }
}
// the lane's weights of `head` and its (cos, sin) table entries at `pos`
__device__ __forceinline__ float4 prologue_weights(const Prologue& pro, int lane, int head) {
    return (pro.normalise && pro.weight) ? __ldg(reinterpret_cast<const float4*>(pro.weight + static_cast<long long>(head) * D) + lane)
                                         : make_float4(1.f, 1.f, 1.f, 1.f);
}
__device__ __forceinline__ const float4* prologue_table(const Prologue& pro, int lane, int pos) {
    return reinterpret_cast<const float4*>(pro.rope + static_cast<long long>(pos) * (D / 2) + 4 * (lane & 15));      // pairs 4(L&15) .. 4(L&15)+3
}
__device__ __forceinline__ void norm_rope_warp(float (&x)[4], int lane, const Prologue& pro, int head, int pos) {
    const float4 w = prologue_weights(pro, lane, head);
    const float4* tab = prologue_table(pro, lane, pos);
    const float4 cs0 = __ldg(tab), cs1 = __ldg(tab + 1);
    norm_rope_warp_loaded(x, lane, pro, w, cs0, cs1);
}

// Host-side check of a caller's prologue; `weight` is the key or the query weights.
inline bool make_prologue(const wushkv_prologue* in, const float* weight, Prologue& out) {
    if (!in || !in->rope_table || in->rope_positions <= 0 || !(in->norm_eps >= 0.f)) return false;
    if (in->normalise != 0 && in->normalise != 1) return false;
    if ((reinterpret_cast<uintptr_t>(in->rope_table) & 15) || (reinterpret_cast<uintptr_t>(weight) & 15)) return false;
    out.rope = reinterpret_cast<const float2*>(in->rope_table);
    out.n_pos = in->rope_positions;
    out.normalise = in->normalise;
    out.weight = weight;
    out.eps = in->norm_eps;
    return true;
}

}  // namespace wushkv
