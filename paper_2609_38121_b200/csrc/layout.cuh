// Physical layout of one packed (page, KV head) record and small shared device helpers.
//
// A record holds PAGE_TOKENS = 64 tokens as 4 blocks of 16 tokens:
//     [K codes: 4 blocks][V codes: 4 blocks][meta: 4 blocks x 128 B]
// with a code block of 512 B (2-bit) or 1024 B (4-bit); 3-bit records are described further down.  Inside a code block
// byte 16*L .. 16*L+15 (of each 512-byte half) belongs to lane L = 4*g + t of the decode warp,
// so that one 16-byte shared-memory load per lane yields exactly the words that lane turns into
// mma A-fragments with a mask (and at most one shift) per register.
//
//  K block (integer mma.m16n8k32: A = codes[16 tokens x 32 channels] as unsigned bytes, one k-step s per
//  32 channels):
//    token row rr -> g = rr & 7, rs = rr >> 3;  channel ch -> s = ch >> 5, hh = (ch >> 4) & 1,
//    b = 2 ((ch >> 3) & 1) + (ch & 1), t = (ch >> 1) & 3.  Word j = rs + 2 hh of lane (g,t) is A register j.
//    2-bit: byte b of that word, at byte 16L + 4j + b of the block; code at bits 2s of the byte (one mask per
//           k-step leaves the code, or four times the code, in every byte).
//    4-bit: 512-byte half p = s >> 1; byte at 512p + 16L + 4j + b; code in nibble s & 1.
//  V block (mma.m16n8k16: A = codes^T[16 channels x 16 tokens] as fp16 per channel block i, channels 16i..16i+15):
//    token rr -> ps = rr >> 3, t = (rr & 7) >> 1, hi = rr & 1;  channel ch -> i = ch >> 4,
//    r16 = ch & 15, rsel = r16 >> 3, g = r16 & 7.
//    2-bit: half-word hi of word (ps, rsel) at byte 16L + 4(2ps + rsel) + 2hi; code at bits 2i.
//    4-bit: 512-byte half ps; word (rsel, j = i>>2) at byte 512ps + 16L + 4(2rsel + j) + 2hi; code at bits 4(i&3).
//    Masked out of a 16-bit lane and read as an fp16 bit pattern, a code field that lies inside bits 0..10 is the
//    exact value code * 2^(shift-24) (fp16 subnormals and the first binade are linear in the bit pattern), so
//    no int->float conversion is executed; the powers of two are folded into the output epilogue.
//  3-bit records store a code c as a 2-bit plane (c & 3, laid out exactly like the 2-bit blocks above) and a 1-bit
//  plane (c >> 2) of 256 bytes per block, 8 bytes = two words per lane:
//    K: word rs of lane (g,t), byte b, bit 2s + hh: (word >> (2s + hh)) & 0x01010101 is A register rs + 2hh of k-step s.
//    V: word ps of lane (g,t), half-word hi; the bit of (rsel, channel block i) sits where one shift of the word puts
//       it two bits above the 2-bit plane's field of block i (so that, read as fp16, it is 4 c1 on that field's
//       scale and both planes accumulate into the same output fragment): v1_bit(rsel, i) below.
//    record: [K 2-bit plane 4 x 512][K 1-bit plane 4 x 256][V 2-bit plane][V 1-bit plane][meta] = 6656 bytes.
//  meta block bi: token rr -> 8 bytes {K step, K x_min, V step, V x_min} (fp16) at 128bi + 16(rr&7) + 8(rr>>3).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace wushkv {

constexpr int D = 128;
constexpr int PAGE_TOKENS = 64;
constexpr int BLOCK_TOKENS = 16;
constexpr int BLOCKS_PER_PAGE = PAGE_TOKENS / BLOCK_TOKENS;

// code_block_bytes: bytes of the (low-plane) code block the decode warp reads with one 16-byte load per lane and
// 512-byte half: 512 at 2 and 3 bits, 1024 at 4 bits; a 3-bit record adds the 256-byte 1-bit-plane blocks.
__host__ __device__ constexpr int code_block_bytes(int bits) { return bits == 4 ? 1024 : 512; }
__host__ __device__ constexpr int hi_block_bytes(int bits) { return bits == 3 ? 256 : 0; }
__host__ __device__ constexpr int side_bytes(int bits) { return BLOCKS_PER_PAGE * (code_block_bytes(bits) + hi_block_bytes(bits)); }
__host__ __device__ constexpr int k_codes_offset(int) { return 0; }
__host__ __device__ constexpr int k_hi_offset(int bits) { return BLOCKS_PER_PAGE * code_block_bytes(bits); }
__host__ __device__ constexpr int v_codes_offset(int bits) { return side_bytes(bits); }
__host__ __device__ constexpr int v_hi_offset(int bits) { return side_bytes(bits) + BLOCKS_PER_PAGE * code_block_bytes(bits); }
__host__ __device__ constexpr int meta_offset(int bits) { return 2 * side_bytes(bits); }
__host__ __device__ constexpr int record_bytes(int bits) { return meta_offset(bits) + PAGE_TOKENS * 8; }

// Bit (inside its 16-bit half-word) of the V 1-bit-plane field of (row half rsel, channel block i), and the shift
// that brings it to its target position 2 + field shift of block i (targets 2,4,6,8,10,2,4,6): a negative shift
// is a left shift.  rsel 0: blocks 0-4 in place, blocks 5-7 from bits 11,13,15 (>> 9); rsel 1: blocks 0-4 from
// bits 1,3,5,7,9 (<< 1), blocks 5,6 from bits 12,14 (>> 10), block 7 from bit 0 (<< 6).
__host__ __device__ constexpr int v1_target(int i) { return i < 5 ? 2 * i + 2 : 2 * (i - 5) + 2; }
__host__ __device__ constexpr int v1_shift(int rsel, int i) { return rsel == 0 ? (i < 5 ? 0 : 9) : (i < 5 ? -1 : (i < 7 ? 10 : -6)); }
__host__ __device__ constexpr int v1_bit(int rsel, int i) { return v1_target(i) + v1_shift(rsel, i); }

// Byte offset (within the record) of the byte holding K code (token r, channel ch) and the bit position
// of the code inside that byte.
__host__ __device__ inline void k_code_location(int bits, int r, int ch, int& byte_off, int& bit) {
    const int bi = r >> 4, rr = r & 15, g = rr & 7, rs = rr >> 3;
    const int s = ch >> 5, hh = (ch >> 4) & 1, b = 2 * ((ch >> 3) & 1) + (ch & 1), t = (ch >> 1) & 3;
    const int L = 4 * g + t, j = rs + 2 * hh;
    if (bits == 2 || bits == 3) {
        byte_off = bi * 512 + 16 * L + 4 * j + b;
        bit = 2 * s;
    } else {
        byte_off = bi * 1024 + 512 * (s >> 1) + 16 * L + 4 * j + b;
        bit = 4 * (s & 1);
    }
}

// The same for V code (token r, channel ch): offset of its 16-bit half-word and the bit position inside it.
__host__ __device__ inline void v_code_location(int bits, int r, int ch, int& byte_off, int& bit) {
    const int bi = r >> 4, rr = r & 15, ps = rr >> 3, t = (rr & 7) >> 1, hi = rr & 1;
    const int i = ch >> 4, r16 = ch & 15, rsel = r16 >> 3, g = r16 & 7;
    const int L = 4 * g + t;
    if (bits == 2 || bits == 3) {
        byte_off = v_codes_offset(bits) + bi * 512 + 16 * L + 4 * (2 * ps + rsel) + 2 * hi;
        bit = 2 * i;
    } else {
        byte_off = v_codes_offset(4) + bi * 1024 + 512 * ps + 16 * L + 4 * (2 * rsel + (i >> 2)) + 2 * hi;
        bit = 4 * (i & 3);
    }
}

// 3-bit records: location of the high bit (c >> 2) of K / V code (token r, channel ch); byte offset of the byte (K)
// or half-word (V) and the bit inside it.  (The functions above give the low two bits.)
__host__ __device__ inline void k_hi_location(int r, int ch, int& byte_off, int& bit) {
    const int bi = r >> 4, rr = r & 15, g = rr & 7, rs = rr >> 3;
    const int s = ch >> 5, hh = (ch >> 4) & 1, b = 2 * ((ch >> 3) & 1) + (ch & 1), t = (ch >> 1) & 3;
    byte_off = k_hi_offset(3) + bi * 256 + 8 * (4 * g + t) + 4 * rs + b;
    bit = 2 * s + hh;
}
__host__ __device__ inline void v_hi_location(int r, int ch, int& byte_off, int& bit) {
    const int bi = r >> 4, rr = r & 15, ps = rr >> 3, t = (rr & 7) >> 1, hi = rr & 1;
    const int i = ch >> 4, r16 = ch & 15, rsel = r16 >> 3, g = r16 & 7;
    byte_off = v_hi_offset(3) + bi * 256 + 8 * (4 * g + t) + 4 * ps + 2 * hi;
    bit = v1_bit(rsel, i);
}

__host__ __device__ inline int meta_location(int bits, int r) {
    const int bi = r >> 4, rr = r & 15;
    return meta_offset(bits) + 128 * bi + 16 * (rr & 7) + 8 * (rr >> 3);
}

// Number of positions read from the packed codes when S positions are cached (closed form of the
// boundary recurrence of Algorithm 2 lines 7-8); they are [s_sink, s_sink + n).
__host__ __device__ inline int n_quantized(int S, int s_sink, int s_keep, int s_flush) {
    const int room = S - s_keep - s_sink;
    if (room < s_flush) return 0;
    return (room / s_flush) * s_flush;
}

// Device-side mirror of the parts of the cache description that kernels need.
struct CacheView {
    int n_q, n_kv, bits, s_sink, s_keep, s_flush, lag;
    int n_slots, max_pages, ring_cap, G;
    long long n_pages;
    unsigned char* pages;
    const int* page_table;
    unsigned short* sink_kv;
    unsigned short* ring_kv;
    const float* T_K;
    const float* T_K_invT;
    int* dev_status;
    float sm_scale;
};

__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) {
    return __uint_as_float(static_cast<unsigned>(b) << 16);
}
__device__ __forceinline__ unsigned short float_to_bf16_bits(float x) {   // round to nearest even
    unsigned u = __float_as_uint(x);
    if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<unsigned short>((u >> 16) | 0x40);
    u += 0x7fffu + ((u >> 16) & 1u);
    return static_cast<unsigned short>(u >> 16);
}

// Sum v[i] over the 32 lanes of a warp for i = 0..31 at once: on return lane L holds the total of
// v[L] in v[0].  31 shuffles instead of 32 x 5 (a butterfly that halves the live values each step).
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[32], int lane) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float send = upper ? v[i] : v[i + off];
            const float keep = upper ? v[i + off] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    return v[0];
}

}  // namespace wushkv
