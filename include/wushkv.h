/*
 * wushkv.h - C ABI of the WUSH-KV serving hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, for ONE attention module on ONE GPU,
 *   (1) calibration-time construction of the per-KV-head key transforms T_K
 *       (WUSH closed form, Section 3 Eq. 1, specialised to keys by Eq. 4 / Algorithm 1),
 *   (2) quantize-on-append: k' = T_K k for each new post-RoPE key, values taken as they
 *       are (already in the weight-folded basis, Section 4.2), the per-token
 *       percentile-clipped affine quantizer of Section 5.3 Eq. 6 at 2, 3 or 4 bits, and packing of
 *       codes + (scale, zero) into a paged cache (Algorithm 2 lines 3-4, 9-12),
 *   (3) decode attention over that packed cache for one new query per sequence
 *       (Algorithm 2 lines 3 and 5; Eq. 2; Eq. 3), reading the first S_sink and the most
 *       recent positions from a bf16 copy (Section 4.4).
 *
 * General rules
 *   - Every function returns an int status (WUSHKV_OK = 0).  No exceptions.  Global state is
 *     limited to a cached device-attribute query, the optional event pair of
 *     wushkv_set_profile_events and the built-in scratch of wushkv_decode_attn_static.
 *   - "host" / "device" beside a pointer says where the memory must live.  All memory is
 *     owned by the caller before, during and after every call; the library allocates nothing
 *     and keeps no pointer between calls.
 *   - wushkv_append / wushkv_decode_attn / wushkv_unpack_debug only ENQUEUE work on the CUDA
 *     stream passed in (a cudaStream_t cast to void*, NULL = default stream) and do not
 *     synchronise.  Arguments are validated on the host before anything is launched; a bad
 *     argument returns WUSHKV_EINVAL and launches nothing.
 *   - Problems that only the device can see (a position beyond the page table, a page id
 *     outside the pool, a copy that never arrived) never trap: the offending access is
 *     skipped and a bit is OR-ed into *dev_status, which the caller reads when it likes.
 *   - Head dimension d must be 128 and page_tokens must be 64.  bits is 2, 3 or 4 (3-bit codes are stored as a 2-bit plane plus a 1-bit plane: 48 bytes per vector).  The query
 *     group size n_q / n_kv must be an integer between 1 and 8.
 *
 * Conventions
 *   - Vectors are rows [token][channel].  T is the paper's T stored row-major [out][in]:
 *     k'[i] = sum_j T[i][j] k[j]  (k' = T k), and q'[i] = sum_j T_invT[i][j] q[j]
 *     (q' = T^{-T} q) with T_invT = (T^{-1})^T.
 *   - Positions are 0-based.  With S positions cached, the positions read from the packed
 *     codes are [s_sink, s_sink + n) with n = floor((S - lag - s_keep - s_sink) / s_flush) * s_flush
 *     when that is >= s_flush and 0 otherwise (closed form of Algorithm 2 lines 7-8);
 *     every other position is read from its bf16 copy (sink buffer or ring buffer).
 *   - bf16 / fp16 values cross the ABI as their 16-bit patterns (uint16_t).
 */
#ifndef WUSHKV_H
#define WUSHKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes (return values) -------------------------------------------------------- */
#define WUSHKV_OK        0
#define WUSHKV_EINVAL    1  /* null pointer, unsupported shape, misaligned buffer, bad size   */
#define WUSHKV_ENOTPD    2  /* damped Gram or Hessian not positive definite (Definition 1)    */
#define WUSHKV_ECUDA     3  /* a CUDA runtime call or kernel launch failed                    */
#define WUSHKV_ECAPACITY 4  /* workspace / ring buffer / page table too small for the request */

/* ---- quantizers (wushkv_cache.quantizer) ---------------------------------------------------- */
#define WUSHKV_QUANTIZER_AFFINE 0
#define WUSHKV_QUANTIZER_QUEST  1

/* ---- bits OR-ed into *dev_status by kernels ---------------------------------------------- */
#define WUSHKV_DEV_PAGE_TABLE_FULL 1  /* a position needs page index >= max_pages: token skipped */
#define WUSHKV_DEV_BAD_PAGE_ID     2  /* page table entry outside [0, n_pages): access skipped   */
#define WUSHKV_DEV_BAD_SLOT        4  /* slot[b] outside [0, n_slots): sequence skipped          */
#define WUSHKV_DEV_COPY_TIMEOUT    8  /* a staged page copy did not arrive within the wait limit */
#define WUSHKV_DEV_BAD_COUNT      16  /* max_new == 1 was promised but a sequence brought more than one token: sequence skipped */
#define WUSHKV_DEV_VALUE_RANGE    32  /* a stored value step Delta_v >= 1024: beyond the fp16 range of the decode value contraction */
#define WUSHKV_DEV_ROPE_RANGE     64  /* a position beyond the rotary table of a *_projected call: rotated by the table's last angle */
/* After PAGE_TABLE_FULL, BAD_PAGE_ID, BAD_SLOT or BAD_COUNT in wushkv_append the length of the affected
 * sequence is left as it was (tokens of the call that did fit are orphaned: nothing reads them). */

/*
 * One layer's cache description.  Plain data; the caller fills it for every call.
 *
 * Packed pages (device): n_pages records of wushkv_page_bytes() bytes each, 256-byte aligned.
 *   A page holds page_tokens consecutive positions of one sequence for all n_kv heads; the
 *   per-(page, head) record keeps, contiguously, the K codes, the V codes and the four fp16
 *   numbers (K step, K x_min, V step, V x_min) of each token (Eq. 6: Delta and the offset
 *   x_min = -Delta z).  The bit layout inside a record is private to the library (it is
 *   permuted to match the decode kernel's register fragments); read it back through
 *   wushkv_unpack_debug.
 * page_table (device): int32 [n_slots][max_pages]; entry [s][i] is the page that holds
 *   positions [i*page_tokens, (i+1)*page_tokens) of slot s.
 * sink_kv (device): bf16 [n_slots][n_kv][2][s_sink][d]; [..][0][p] is k' (= bf16(T_K k)) and
 *   [..][1][p] is v of position p < s_sink.  May be NULL when s_sink == 0.
 * ring_kv (device): bf16 [n_slots][n_kv][2][ring_cap][d]; position p lives in row p % ring_cap.
 *   ring_cap >= s_keep + s_flush - 1 + boundary_lag.
 * T_K, T_K_invT (device): fp32 [n_kv][d][d] as produced by wushkv_build_transforms.
 * dev_status (device): one int32 that kernels OR error bits into; the caller zeroes it.
 */
typedef struct wushkv_cache {
    int32_t n_q, n_kv, d, bits;
    int32_t page_tokens, s_sink, s_keep, s_flush;
    int32_t boundary_lag;  /* 0: read boundary from the current length (serving behaviour,
                              Section 5.3); k: boundary of k positions ago (Algorithm 2 taken
                              literally has k = positions appended in this step) */
    int32_t n_slots, max_pages, ring_cap;
    float kappa_k, kappa_v; /* clipping quantiles of Eq. 6 for keys and values, in [0, 1] */
    float sm_scale;         /* 1 / tau of Eq. 2 */
    int32_t quantizer;      /* WUSHKV_QUANTIZER_AFFINE (0): percentile-clipped affine, Section 5.3 Eq. 6;
                               WUSHKV_QUANTIZER_QUEST (1): QuEST, Section 4.3 Eq. 5 (step from the group's RMS, bin-centre
                               reconstruction, Q(0) = 0; kappa_k / kappa_v unused).  Both are stored as (step, offset, codes)
                               with x_hat = offset + step * code, so decode reads either. */
    int64_t n_pages;
    void* pages;
    const int32_t* page_table;
    void* sink_kv;
    void* ring_kv;
    const float* T_K;
    const float* T_K_invT;
    int32_t* dev_status;
} wushkv_cache;

/* Bytes of one page (all n_kv heads): n_kv * page_tokens * (2 * d * bits / 8 + 8).
 * Returns 0 for an unsupported (bits, page_tokens, d). */
size_t wushkv_page_bytes(int32_t n_kv, int32_t d, int32_t bits, int32_t page_tokens);

/* Human-readable name of a status code (static storage). */
const char* wushkv_status_string(int status);

/*
 * Gram / Hessian accumulation for the key transform: Eq. 4 and Algorithm 1 lines 4-5.
 *   K (host): bf16 [n_tok][n_kv][d]  post-Norm post-RoPE keys of one calibration sequence.
 *   Q (host): bf16 [n_tok][n_q][d]   post-Norm post-RoPE queries; head j belongs to KV head j / (n_q/n_kv).
 *   M, H (host, in/out): float64 [n_kv][d][d];  M[h] += sum_t k k^T,  H[h] += 2 sum_g sum_t q q^T.
 * Call once per calibration sequence (Algorithm 1 sums over sequences); the caller zeroes M, H first.
 */
int wushkv_accumulate_gram(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tok,
                           const uint16_t* K, const uint16_t* Q, double* M, double* H);

/*
 * WUSH transforms from accumulated statistics: Section 3 Eq. 1 / Definition 1 applied per head
 * (Algorithm 1 line 7).  Host pointers, host float64 arithmetic (Cholesky, cyclic Jacobi
 * eigensolver, Sylvester Hadamard); runs once at calibration time.
 *   M, H (host): float64 [n_heads][d][d] symmetric; gamma >= 0 the damping ratio.
 *   T (host, out): fp32 [n_heads][d][d], T = c Had Lam^(-1/4) U^T L^T with eigenvalues
 *       ascending and each eigenvector signed so that its largest-magnitude entry is positive;
 *       every entry is rounded to the nearest bf16-representable value.
 *   T_invT (host, out): fp32 [n_heads][d][d], transpose of the inverse of the ROUNDED T, so that
 *       the insertion identity of Eq. 3 holds for the stored pair.
 * d must be a power of two (<= 1024).  Returns WUSHKV_ENOTPD if a damped matrix is not
 * positive definite (outputs of that head are then unspecified).
 */
int wushkv_build_transforms(int32_t n_heads, int32_t d, const double* M, const double* H, double gamma,
                            float* T, float* T_invT);

/*
 * The same two calibration steps on the GPU (Algorithm 1 lines 4-5 and 7; Eq. 4; Eq. 1), for calibration sets
 * of millions of tokens.  Results equal the host calls' up to summation order.
 *   wushkv_accumulate_gram_device: K, Q (device) bf16 as above, 16-byte aligned; M, H (device, in/out) float64
 *     [n_kv][d][d], zeroed by the caller before the first sequence.  d must be 128.  Products of the bf16
 *     inputs are exact, sums are fp32 within groups of 128 tokens and float64 beyond (relative error below 1e-6).
 *   wushkv_build_transforms_device: M, H (device) float64 [n_heads][d][d]; T, T_invT (device, out) fp32
 *     [n_heads][d][d] with the same canonical form and bf16 rounding as the host call; status (device, out):
 *     one int32 the caller zeroes, set to WUSHKV_ENOTPD if a damped matrix is not positive definite;
 *     workspace (device): >= wushkv_build_transforms_workspace_bytes() bytes, 16-byte aligned.
 * Both enqueue on `stream` and do not synchronise.
 */
int wushkv_accumulate_gram_device(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tok, const uint16_t* K, const uint16_t* Q,
                                  double* M, double* H, void* stream);
size_t wushkv_build_transforms_workspace_bytes(int32_t n_heads, int32_t d);
int wushkv_build_transforms_device(int32_t n_heads, int32_t d, const double* M, const double* H, double gamma,
                                   float* T, float* T_invT, int32_t* status, void* workspace, size_t workspace_bytes,
                                   void* stream);


/*
 * Quantize-on-append: Algorithm 2 lines 3-4 (key side) and 9-12, with Eq. 6 as the quantizer.
 * For sequence b (0 <= b < batch) the new tokens are rows cu_new[b] .. cu_new[b+1]-1 of K_new /
 * V_new and take positions seq_len[b], seq_len[b]+1, ...  Every new token is transformed
 * (keys only), quantized from the fp32 transform output, packed into its page, and its bf16
 * copy is written to the sink buffer (position < s_sink) and to the ring buffer (if it is among
 * the last ring_cap positions after this call).  Finally seq_len[b] += number of new tokens.
 *   slot (device): int32 [batch], cache slot of each sequence; slots must be distinct (not checked: two sequences
 *                  given the same slot write the same rows and no status bit is set).
 *   seq_len (device, in/out): int32 [batch].
 *   cu_new (device): int32 [batch+1] prefix sums, cu_new[0] = 0, cu_new[batch] = total_new.
 *   total_new, max_new (host): total and per-sequence maximum of new tokens.
 *   K_new (device): bf16 [total_new][n_kv][d] post-Norm post-RoPE keys, 16-byte aligned.
 *   V_new (device): bf16 [total_new][n_kv][d] values in the folded basis, 16-byte aligned.
 * Chunks (max_new >= 128) take the tensor-core transform path (tcgen05, fp32 accumulation in
 * tensor memory), max_new == 1 a single-launch decode-time path, anything else a CUDA-core path.
 * All produce the same codes up to fp32 summation order (wushkv_set_test_option("append_path_cuda", 1)
 * forces the CUDA-core path for chunks).
 */
int wushkv_append(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                  const int32_t* cu_new, int32_t total_new, int32_t max_new,
                  const uint16_t* K_new, const uint16_t* V_new, void* stream);

/* Bytes of scratch wushkv_decode_attn needs for (batch, max_seq_len); 0 on invalid arguments. */
size_t wushkv_decode_workspace_bytes(const wushkv_cache* cache, int32_t batch, int32_t max_seq_len);

/*
 * Decode attention: Algorithm 2 line 3 (query side: q' = T_K^{-T} q) and line 5 (Eq. 2 for one
 * query column that sees all seq_len[b] cached positions, softmax temperature 1/sm_scale),
 * evaluated directly on the packed cache: quantized positions are dequantized in registers
 * (x_hat = x_min + Delta * code), window positions are read from the bf16 buffers.  The
 * context is split across thread blocks (partial softmax state per split) and merged by a
 * final combine pass.  Call after wushkv_append of the step's token.
 *   slot (device): int32 [batch];  seq_len (device): int32 [batch], each >= 1.
 *   max_seq_len (host): upper bound of seq_len[b] (sizes the launch; no device read-back).
 *   Q (device): bf16 [batch][n_q][d] post-Norm post-RoPE, NOT compensated; 16-byte aligned.
 *   O (device, out): fp32 [batch][n_q][d] = V P in the folded value basis (the output
 *       projection, Algorithm 2 line 6, is outside the library).
 *   workspace (device): >= wushkv_decode_workspace_bytes(...) bytes, 256-byte aligned; contents
 *       are scratch (no initialisation needed, nothing survives the call).
 * The kernels of one call are chained by programmatic dependent launch; the first of them waits
 * for the kernel before it in the stream before it reads anything, so any producer of Q, seq_len or
 * the cache may precede the call directly.
 * Range: probabilities times the stored value step are fed to the tensor core in fp16 with up to
 * 2^6 of headroom, so a stored Delta_v of 1024 or more (a value range beyond ~3000 at 2 bits)
 * saturates and loses accuracy; keys have no such limit.
 * The scores of the quantized positions are computed from a 16-bit fixed-point copy of q' (exact
 * integer dot products with the codes), i.e. they are the scores of a query that differs from q' by
 * at most 2^-16 of its largest entry per channel.
 * NaN or infinite inputs (Q, or stored steps / offsets derived from such keys and values) give
 * unspecified finite-or-NaN outputs for the affected sequences; nothing traps.
 */
int wushkv_decode_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                       int32_t max_seq_len, const uint16_t* Q, float* O,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Chunk (prefill) attention: Algorithm 2 line 3 (q' = T_K^{-T} q, k' = T_K k) and line 5 for a chunk of new
 * positions, evaluated AFTER wushkv_append has stored the chunk (line 4).  Chunk position i of sequence b attends
 * to cached positions 0 .. seq_len[b] - n_new[b] + i (causal inside the chunk).  The chunk's own keys and values
 * are read in full precision (k' rounded to bf16, as the cache's window copies hold it; Sections 4.4 and 5.3: a new
 * chunk is appended in full precision and its attention output is computed from those copies), older
 * positions by the window rule at length seq_len[b] - boundary_lag: sink and recent window from the bf16 buffers,
 * the quantized middle from the packed pages.  boundary_lag = n_new reproduces Algorithm 2 literally (boundary
 * moved after attention); ring_cap must then cover s_keep + s_flush - 1 + boundary_lag positions.
 *   slot, cu_new, total_new, max_new, K_new, V_new: exactly what the preceding wushkv_append received.
 *   seq_len (device): int32 [batch], the lengths AFTER that append.
 *   Q_new (device): bf16 [total_new][n_q][d] post-Norm post-RoPE queries of the chunk, NOT compensated.
 *   O (device, out): fp32 [total_new][n_q][d] in the folded value basis.
 *   workspace (device): >= wushkv_prefill_workspace_bytes() bytes, 256-byte aligned, scratch.
 * Both contractions run on the tcgen05 tensor cores (fp16 operands, fp32 accumulators in tensor memory); q' enters as
 * an fp16 value plus its fp16 rounding remainder.  The query heads of a KV head share one 128-row tile.  A call whose
 * chunk is too short to fill the GPU with tiles splits every tile's keys over several CTAs and merges their partial
 * results (the workspace holds them); the result does not depend on timing, only on the call's shapes.
 */
size_t wushkv_prefill_workspace_bytes(const wushkv_cache* cache, int32_t batch, int32_t total_new);
int wushkv_prefill_attn(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                        const int32_t* cu_new, int32_t total_new, int32_t max_new,
                        const uint16_t* K_new, const uint16_t* V_new, const uint16_t* Q_new, float* O,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Attention-aware Hessians for the WUSH-A variant (Appendix C, "Aggregation for WUSH-A"): for ONE calibration
 * sequence and every key/value head, the key Hessian and the value Hessian of the module-output error, summed over
 * the perturbed cache position, added to the caller's float64 accumulators (call once per sequence; pass the sums
 * to wushkv_build_transforms[_device] in place of Eq. 4's Hessians).  They depend on the causal attention
 * probabilities p = softmax(q . k / tau), the head outputs and the output projection only (forward quantities).
 *   K, Q, V (device): bf16 [n_tokens][n_kv][d], [n_tokens][n_q][d], [n_tokens][n_kv][d]; K and Q after Norm and RoPE,
 *                     V as projected (not folded).
 *   W_O (device):     fp32 [n_q][d][d_model], the output-projection block of every query head.
 *   tau:              the logit temperature (sqrt(d) in the paper).
 *   H_K, H_V (device, in/out): float64 [n_kv][d][d], accumulated.
 *   workspace (device): >= wushkv_attention_hessians_workspace_bytes() bytes, 256-byte aligned, scratch.
 * d must be 128 and the group size n_q / n_kv at most 8 (WUSHKV_EINVAL otherwise).  Cost O(n_tokens^2) per head.
 * Arithmetic: fp32 with float64 accumulation of the sums over tokens.
 */
size_t wushkv_attention_hessians_workspace_bytes(int32_t n_kv, int32_t n_q, int32_t d, int64_t n_tokens);
int wushkv_accumulate_attention_hessians_device(int32_t n_kv, int32_t n_q, int32_t d, int32_t d_model, int64_t n_tokens,
                                                const uint16_t* K, const uint16_t* Q, const uint16_t* V, const float* W_O,
                                                double tau, double* H_K, double* H_V,
                                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Projected inputs: Algorithm 2 lines 1-2 (Norm, RoPE) fused into the kernels that apply line 3, so that
 * keys and queries are read once, in the form the projections W_K x, W_Q x left them, and their normalised,
 * rotated form never goes through memory (Section 4.1: keys are cached after normalisation and rotation).
 *   Norm: headwise RMS normalisation x / sqrt(mean(x^2) + norm_eps), times a per-channel weight.
 *   RoPE: channel pair (j, j + d/2) is rotated by the angle position * theta^(-2j/d); the position of a new
 *         key is its index in the sequence, the position of the decode query is seq_len[b] - 1.
 *   Arithmetic: fp32, one rounding to bf16 after the rotation; from there on the call is bit-identical to its
 *         plain counterpart given those bf16 values.
 *   wushkv_prologue (host struct; its pointers are DEVICE pointers, caller-owned, read-only):
 *     rope_table       fp32 [rope_positions][d/2][2] = (cos, sin), written by wushkv_build_rope_table
 *     rope_positions   positions the table covers; a token beyond it sets WUSHKV_DEV_ROPE_RANGE and is
 *                      rotated by the table's last angle (drop the sequence)
 *     normalise        0: no Norm step (RoPE only); 1: RMS normalisation
 *     k_norm_weight    fp32 [n_kv][d] or NULL (ones);  q_norm_weight  fp32 [n_q][d] or NULL (ones)
 *     norm_eps         >= 0
 * wushkv_build_rope_table: cosines and sines in double precision, rounded to fp32 (device kernel; d must be 128).
 * wushkv_append_projected / wushkv_decode_attn_projected / wushkv_prefill_attn_projected: arguments, results and errors
 * of wushkv_append / wushkv_decode_attn / wushkv_prefill_attn, with K_proj / Q_proj in place of K_new / Q and WUSHKV_EINVAL for a NULL or malformed
 * prologue.  Values are never normalised or rotated (V_new is passed as before).
 */
typedef struct wushkv_prologue {
    const float* rope_table;
    int32_t rope_positions;
    int32_t normalise;
    const float* k_norm_weight;
    const float* q_norm_weight;
    float norm_eps;
} wushkv_prologue;
int wushkv_build_rope_table(double theta, int32_t n_positions, int32_t d, float* table, void* stream);
int wushkv_append_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                            const int32_t* cu_new, int32_t total_new, int32_t max_new,
                            const uint16_t* K_proj, const uint16_t* V_new, const wushkv_prologue* prologue, void* stream);
int wushkv_decode_attn_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                 int32_t max_seq_len, const uint16_t* Q_proj, const wushkv_prologue* prologue, float* O,
                                 void* workspace, size_t workspace_bytes, void* stream);
/* wushkv_prefill_attn on projected keys and queries of the chunk (K_proj: what wushkv_append_projected received; the
 * position of chunk token i of sequence b is seq_len[b] - n_new[b] + i); otherwise as wushkv_prefill_attn. */
int wushkv_prefill_attn_projected(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                                  const int32_t* cu_new, int32_t total_new, int32_t max_new,
                                  const uint16_t* K_proj, const uint16_t* V_new, const uint16_t* Q_proj,
                                  const wushkv_prologue* prologue, float* O,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Read back the logical content of the packed cache (test / debugging aid): for positions
 * pos0 .. pos0+n-1 of (slot, kv_head), which = 0 for keys, 1 for values:
 *   codes (device, out): uint8 [n][d], one code per byte in channel order;
 *   scale (device, out): fp32 [n] the stored step Delta;  zero (device, out): fp32 [n] the stored x_min.
 * Positions are read wherever they are in the page table regardless of the windows.
 */
int wushkv_unpack_debug(const wushkv_cache* cache, int32_t slot, int32_t kv_head, int32_t which,
                        int32_t pos0, int32_t n, uint8_t* codes, float* scale, float* zero, void* stream);

/*
 * One whole decode step from DEVICE buffers: Algorithm 2 lines 3-5 and 7-12 for one new token per
 * sequence, i.e. wushkv_append of one token per sequence followed by wushkv_decode_attn over the
 * extended cache, with the same results as those two calls.  Because the library knows here what
 * runs ahead of the query preparation (its own append kernel, which begins only after all earlier
 * work in the stream has finished), it transforms the queries while the new token is being
 * quantized instead of after it.
 *   K_new, V_new (device): bf16 [batch][n_kv][d].   Q (device): bf16 [batch][n_q][d], 16-byte aligned.
 *   O (device, out): fp32 [batch][n_q][d].   cu_new (device): int32 [batch+1] = 0, 1, ..., batch.
 *   slot, seq_len (in/out), max_seq_len (bound on the lengths AFTER the append), workspace: as for
 *   wushkv_append / wushkv_decode_attn.  The decode half is validated before anything is appended.
 */
int wushkv_decode_step(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                       const int32_t* cu_new, int32_t max_seq_len,
                       const uint16_t* K_new, const uint16_t* V_new, const uint16_t* Q, float* O,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * One whole decode step from HOST buffers: Algorithm 2 lines 3-5 and 7-12 for one new token per
 * sequence.  Enqueues, in order, on `stream`: host->device copies of K_new, V_new and Q into
 * `staging`, wushkv_decode_step on the staged copies, and the device->host copy of O.  Does not synchronise; O_host is valid once the stream has been synchronised.
 *   K_new_host, V_new_host (host, pinned for the copies to be asynchronous): bf16 [batch][n_kv][d].
 *   Q_host (host): bf16 [batch][n_q][d].   O_host (host, out): fp32 [batch][n_q][d].
 *   cu_new (device): int32 [batch+1] = 0, 1, ..., batch.
 *   staging (device): >= wushkv_step_staging_bytes() bytes, 256-byte aligned, scratch.
 *   When all four host buffers are pinned and mapped into the device's address space (cudaHostAlloc or
 *   cudaHostRegister under unified addressing) and 16-byte aligned, no copy is enqueued: the kernels read
 *   K_new, V_new and Q and write O in place over the bus.  Otherwise (or with WUSHKV_HOST_IO=copy in the
 *   environment) the copies go through `staging`.  Results are identical either way.
 *   slot, seq_len (in/out), max_seq_len (bound on the lengths AFTER the append), workspace: as for
 *   wushkv_append / wushkv_decode_attn.
 */
size_t wushkv_step_staging_bytes(const wushkv_cache* cache, int32_t batch);
int wushkv_decode_step_host(const wushkv_cache* cache, int32_t batch, const int32_t* slot, int32_t* seq_len,
                            const int32_t* cu_new, int32_t max_seq_len,
                            const uint16_t* K_new_host, const uint16_t* V_new_host, const uint16_t* Q_host,
                            float* O_host, void* staging, size_t staging_bytes,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * wushkv_decode_attn without a caller-provided workspace (the paper has no counterpart: this is
 * an interface convenience).  It is meant for callers that cannot allocate device memory - for
 * example because their framework took all of it for its own pool at start-up, because they are a
 * plug-in that only ever receives input and output buffers, or because an allocation's implicit
 * synchronisation has no place in their latency-critical loop.  The scratch is a fixed array of
 * WUSHKV_STATIC_SCRATCH_BYTES inside the library's device image; each GPU that loads the library
 * holds that much memory until the process exits.
 *   - Arguments and results are exactly those of wushkv_decode_attn, minus workspace.
 *   - A request whose wushkv_decode_workspace_bytes() exceeds WUSHKV_STATIC_SCRATCH_BYTES is
 *     refused with WUSHKV_ECAPACITY and nothing is launched; use wushkv_decode_attn then.
 *     The workspace grows with batch * n_kv (8 KiB of query fragments each) and with the number
 *     of warps of the main kernel (G * 528 bytes of partial result each; the "decode_ctas"
 *     testing aid changes that number).  On a 148-SM GPU: 16 sequences x 8 KV heads x 32 query
 *     heads need 6.0 MiB, 1 x 8 x 64 needs 7.2 MiB, 8 x 4 x 28 needs 6.6 MiB - they fit;
 *     64 sequences x 8 KV heads x 32 query heads need 8.6 MiB and are refused.
 *   - The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device current); make that first call before starting any stream capture.
 *   - All calls on a GPU share the one array, and it keeps whatever the last call left in it.
 *     Nothing in it needs to be zero at entry (each call writes every value it later reads), but
 *     two calls that overlap on the GPU - different streams, or different threads - race on it.
 *     Serialise them (same stream, or an event between them).
 */
#define WUSHKV_STATIC_SCRATCH_BYTES (8u << 20)
int wushkv_decode_attn_static(const wushkv_cache* cache, int32_t batch, const int32_t* slot, const int32_t* seq_len,
                              int32_t max_seq_len, const uint16_t* Q, float* O, void* stream);

/*
 * Measurement aid (not part of the method): when both arguments are non-NULL cudaEvent_t handles,
 * every following wushkv_decode_attn records `start` immediately before and `stop` immediately after
 * its main kernel (the one that streams the packed cache) on the call's stream, so that a benchmark
 * can time that kernel alone.  Pass NULLs to switch it off.  Process-wide, not thread-safe.
 */
int wushkv_set_profile_events(void* start, void* stop);

/*
 * Testing aids (not part of the method).  Process-wide and unsynchronised: set them from one thread while
 * no call of the library is running.  The first three take their initial value from the environment
 * (WUSHKV_DECODE_CTAS=<n>, WUSHKV_APPEND_PATH=cuda, WUSHKV_HOST_IO=copy), read once per process.
 *   "decode_ctas"       n > 0: number of thread blocks of the decode main kernel (the split count); 0: automatic.
 *   "append_path_cuda"  1: prefill chunks take the CUDA-core append path instead of the tensor-core one.
 *   "host_io_copy"      1: wushkv_decode_step_host always stages its host buffers with copies.
 *   "drop_copy_unit"    u >= 0: the decode main kernel does not issue the copy of work unit u of its flattened
 *                       list, so that the wait for it runs into its limit (WUSHKV_DEV_COPY_TIMEOUT is set
 *                       in *dev_status and the kernel returns); -1: off.
 *   "wait_limit"        n > 0: poll limit of the device-side barrier waits (default: about a second); 0: default.
 *   "drop_chunk_mma"    1: the chunk append does not commit the MMAs of its first tile to their barrier (same
 *                       failure path in that kernel).
 *   "prefill_legacy"    1: wushkv_prefill_attn runs its mma.sync kernels (attention and transforms) instead of the tcgen05 ones.
 *   "prefill_one_tile"  1: the chunk attention runs on the tcgen05 kernel with one query tile per CTA and no role split
 *                       instead of the warp-specialised one.
 *   "prefill_split"     n > 0: the warp-specialised chunk attention runs n CTAs per tile pair, each over a share of the key
 *                       tiles, and merges their partial results (capped by what the workspace was sized for); 0: chosen from
 *                       the number of tile pairs (several CTAs per pair only when the pairs alone would not fill the GPU).
 *   "prefill_no_tma"    1: the tcgen05 kernel stages the chunk's own tiles with 16-byte copies, not bulk tensor copies.
 *   "append_no_tma"     1: the same for the key / value tiles of the tensor-core chunk append.
 *   "drop_prefill"      1: the tcgen05 chunk attention never commits the score MMAs of a CTA's first tile; 2: it announces
 *                       but never issues one bulk copy of a CTA's first chunk tile; 3: the tcgen05 transform kernel does the
 *                       same with a copy of its first token tile (the bounded wait runs out in each case).
 * Returns WUSHKV_EINVAL for an unknown name.
 */
int wushkv_set_test_option(const char* name, long long value);

#ifdef __cplusplus
}
#endif
#endif /* WUSHKV_H */
