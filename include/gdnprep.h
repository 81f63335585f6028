/*
 * gdnprep - chunk preparation for chunk-wise Gated DeltaNet on NVIDIA B200 (sm_100a).
 *
 * For every chunk of C consecutive tokens of every (batch, head) this library
 * builds the strictly lower-triangular matrix
 *
 *     A_ij = beta_i * exp(g_i - g_j) * <K_i, K_j>      (i > j, 0 otherwise),
 *
 * the "scaled inner product of the keys" of the paper's Sec. 2.1 with the Gated
 * DeltaNet write strength beta and gate decay, and computes
 *
 *     T = (I + A)^-1,      W = T diag(beta) K,      U = T diag(beta) V.
 *
 * The paper writes the system as (I - A)^-1 (Eq. 1); its A is -A here.
 *
 * T is obtained with the paper's multiplication-only scheme (Sec. 3, Alg. 1):
 * a Neumann series truncated at order N and masked to the band 0 <= i-j <= N
 * (Eq. 7, 10, 11), followed by the parallel residual correction
 * T = T0 * sum_{s=0..S} E^s with E = I - (I + A) T0 (Eq. 13). For C = 128 the
 * two 64 x 64 diagonal blocks are inverted this way and the lower-left block
 * follows from the block formula of App. E (Eq. 28).
 *
 * Common conventions
 *   - Every pointer is a DEVICE pointer owned by the caller. The library
 *     allocates no device memory for the caller's data, never synchronises
 *     (except gdn_device_status) and enqueues its work on `stream`.
 *   - Layouts are contiguous:  K [B, H_k, T, d_k],  V [B, H_v, T, d_v],
 *     beta, g [B, H_v, T] (fp32),  W [B, H_v, T, d_k],  U [B, H_v, T, d_v],
 *     Tinv [B, H_v, T/C, C, C] (the full matrix, unit diagonal included, zeros
 *     above it). K, V, W, U, Tinv have the element type selected by `dtype`.
 *   - g is the CUMULATIVE log-gate. Only differences inside a chunk are used,
 *     so a chunk-local or a global prefix sum give the same result. Gates are at most 1: g must not increase inside
 *     a chunk (raw log-gates <= 0). The decay factor exp(g_i - g_j), i > j, is evaluated with its exponent clamped at
 *     +64 octaves, so an increasing g gives finite but unspecified results; any rate of decrease is fine (the factor
 *     underflows to 0 for a gate that closes).
 *   - Degenerate inputs are well defined: a zero key or beta = 0 is a token that writes nothing (T keeps its unit row
 *     there); with GDN_FLAG_K_L2NORM a zero key stays zero; B = 0 or T = 0 launches nothing.
 *   - Value head h reads key head h / (H_v / H_k); H_v must be a multiple of H_k.
 *   - order = N >= 1 and residual_steps = S >= 0; -1 selects the paper's value
 *     for the chunk size (gdn_default_order, gdn_default_residual_steps).
 *     S >= ceil(C / (N + 1)) - 1 keeps every non-zero term (E^s = 0 beyond), i.e. the
 *     exact inverse: S = 15 at C = 64, N = 3.
 *   - Return value: GDN_OK or a negative gdn_status. On any error nothing is
 *     launched. No exception crosses this boundary.
 *   - Pointers must be 16-byte aligned; T must be a multiple of C.
 *   - The device must be compute capability 10.x (B200); anything else gives
 *     GDN_ERR_ARCH. There is no CPU fallback.
 */
#ifndef GDNPREP_H_
#define GDNPREP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GDN_OK = 0,
    GDN_ERR_INVALID_ARG = -1, /* a size or parameter is out of range (e.g. T % C != 0, order < 1) */
    GDN_ERR_UNSUPPORTED = -2, /* valid in principle, not implemented by the kernels (e.g. d_k = 96) */
    GDN_ERR_NULL = -3,        /* a required pointer is NULL */
    GDN_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned */
    GDN_ERR_LAUNCH = -5,      /* the CUDA runtime refused the launch or a set-up call */
    GDN_ERR_TIMEOUT = -6,     /* a bounded wait inside a kernel ran out (reported by gdn_device_status) */
    GDN_ERR_ARCH = -7,        /* the current device is not sm_100 */
    GDN_ERR_SCRATCH = -8      /* gdn_chunk_state_output_segmented_noalloc: the problem needs more scratch memory than the
                                 library's built-in array holds */
} gdn_status;

enum { GDN_DTYPE_FP32 = 0, GDN_DTYPE_BF16 = 1 };

/* flags of gdn_chunk_prepare_ex */
enum {
    GDN_FLAG_G_RAW = 1,     /* g holds the raw per-token log-gates; the kernel forms the chunk-local inclusive prefix sum */
    GDN_FLAG_K_L2NORM = 2,  /* the kernel L2-normalises the rows of K first (the normalisation Sec. 2.1 places before the path) */
    GDN_FLAG_OUT_FP32 = 4,  /* W, U, Tinv are written as fp32 although K, V are bf16 (parity debugging) */
    GDN_FLAG_W_GATED = 16,  /* W = T diag(beta * exp(g)) K: the gated form the state update of the layer consumes
                               (g as given, or the chunk-local prefix sum with GDN_FLAG_G_RAW); U is unchanged */
    GDN_FLAG_LAYOUT_BTHD = 8 /* token-major tensors as model code keeps them: K [B,T,H_k,d_k], V [B,T,H_v,d_v],
                                beta, g [B,T,H_v], W [B,T,H_v,d_k], U [B,T,H_v,d_v]; Tinv stays [B,H_v,T/C,C,C].
                                bf16 only (GDN_ERR_UNSUPPORTED with GDN_DTYPE_FP32) */
};

/* variants of the forward-substitution comparison kernel */
enum { GDN_FWDSUBST_ROWS = 0, GDN_FWDSUBST_BLOCKED = 1, GDN_FWDSUBST_BLOCKED_TC = 2 };

/* A CUDA stream handle (cudaStream_t) passed as an opaque pointer. */
typedef void* gdn_stream_t;

/*
 * The hot path (Sec. 3, Alg. 1, Eq. 7-13; App. E for C = 128): A-build, masked
 * truncated Neumann series, residual power sum, W and U.
 *   dtype GDN_DTYPE_BF16: bf16 K, V, W, U, Tinv, fp32 accumulation. The tensor-core kernel takes C in {16, 32, 64, 128},
 *                         d_k = d_v = 128, 1 <= order <= 7 (every configuration of the benchmark); any other shape
 *                         within the fp32 limits below runs on the plain FMA kernel with bf16 tensors.
 *   dtype GDN_DTYPE_FP32: fp32 everywhere, plain FMA kernel; 2 <= C <= 64 or C = 128 (two 64-blocks), d_k, d_v <= 256
 *                         in multiples of 8.
 * Tinv_out may be NULL (the store is skipped). H = H_k = H_v.
 */
int gdn_chunk_prepare(const void* K, const void* V, const float* beta, const float* g,
                      int B, int H, int T, int C, int d_k, int d_v,
                      int order, int residual_steps, int dtype,
                      void* W_out, void* U_out, void* Tinv_out, gdn_stream_t stream);

/*
 * Same operation with grouped heads: H_k key heads shared by H_v value heads
 * (beta, g, W, U, Tinv are per value head; only K is shared).
 */
int gdn_chunk_prepare_gqa(const void* K, const void* V, const float* beta, const float* g,
                          int B, int H_k, int H_v, int T, int C, int d_k, int d_v,
                          int order, int residual_steps, int dtype,
                          void* W_out, void* U_out, void* Tinv_out, gdn_stream_t stream);

/*
 * gdn_chunk_prepare_gqa with the optional prologue of the path fused in (Sec. 2.1: the l2-normalisation of the keys
 * sits right before the path; the gate prefix sum is Gated DeltaNet's): see the GDN_FLAG_* values. With
 * GDN_FLAG_OUT_FP32 the three output buffers hold fp32 elements (same shapes).
 */
int gdn_chunk_prepare_ex(const void* K, const void* V, const float* beta, const float* g,
                         int B, int H_k, int H_v, int T, int C, int d_k, int d_v,
                         int order, int residual_steps, int dtype,
                         void* W_out, void* U_out, void* Tinv_out, unsigned flags, gdn_stream_t stream);

/*
 * The comparison the paper's speed-up is measured against: the same A-build, W
 * and U, with T computed exactly by forward substitution (Eq. 2-3;
 * variant GDN_FWDSUBST_ROWS) or by 16 x 16 diagonal blocks merged with the
 * block recursion of App. E (Eq. 25-27; variant GDN_FWDSUBST_BLOCKED), or by the two 32 x 32 diagonal blocks of a
 * 64-chunk with the lower-left block from the block formula (Eq. 28) evaluated on the tensor cores (variant
 * GDN_FWDSUBST_BLOCKED_TC: bf16, C = 64 only). Same dtypes, sizes and layouts as
 * gdn_chunk_prepare_gqa. For C = 128 on the bf16 path both variants invert the two 64 x 64 diagonal blocks by
 * their substitution and obtain the lower-left block from the block formula of App. E (Eq. 28), as the Neumann
 * path does.
 */
int gdn_chunk_prepare_fwdsubst(const void* K, const void* V, const float* beta, const float* g,
                               int B, int H_k, int H_v, int T, int C, int d_k, int d_v,
                               int dtype, int variant,
                               void* W_out, void* U_out, void* Tinv_out, gdn_stream_t stream);

/*
 * INT8 variant (Sec. 3.5 "good enough under low-bit quantization"; quantiser of App. G, Eq. 32): every tensor of
 * the chain is int8 mantissas in [-127, 127] with one power-of-two exponent per chunk, int32 accumulation on the
 * tensor cores, requantisation after every product and sum with the structural mask applied first. The outputs
 * are a pure function of the integer inputs (bit-exact against an exact-integer evaluation).
 *   Kq [B,H_k,T,d_k], Vq [B,H_v,T,d_v] int8; k_exp [B,H_k,T/C], v_exp [B,H_v,T/C]: value = q * 2^exp;
 *   beta_q [B,H_v,T] = round(beta * 2^15) in [0, 32767]; decay_q [B,H_v,T] = round(-g * log2(e) * 2^8),
 *   non-decreasing inside every chunk (not checked).
 *   Wq_out [B,H_v,T,d_k], Uq_out [B,H_v,T,d_v] int8 with w_exp_out, u_exp_out [B,H_v,T/C];
 *   Toff_q_out [B,H_v,T/C,C,C] int8 (may be NULL) with t_exp_out [B,H_v,T/C]: T = I + Toff_q * 2^t_exp.
 *   dbg_acc_out (may be NULL; meant for small cases): every int32 tensor-core accumulator of the chain,
 *   [B,H_v,T/C, C, 8*C + d_k + d_v] int32. Row i of a chunk holds: columns [0, C) the Gram row Kq Kq^T;
 *   columns [(s-1)*C, s*C) for s = 2..8 the row of the power product R_{s-1} Eq (left untouched for powers
 *   that the parameters skip: the caller zeroes the buffer); then d_k columns of Tbq Kq and d_v of Tbq Vq.
 * C = 128 (Sec. 4.3 and App. H: chunks of 128 tokens as 64 x 64 blocks; block formula of App. E, Eq. 28): the three
 *   blocks of A (A11, A21, A22) are quantised separately from 2 k_exp - 15, the chain above runs on the two diagonal
 *   blocks, and with the stored blocks holding -A the lower-left block is T21q = Q8(align(X, Toff22q X)),
 *   X = Q8(align(A21q, A21q Toff11q)); W and U are requantised per 64 rows, the lower rows from the aligned sum of
 *   T21b Kq_top, T22b Kq_bot and beta_q_i Kq_i (b = the block times beta_q_j, requantised). Shapes then:
 *   k_exp [B,H_k,T/128], v_exp [B,H_v,T/128]; w_exp_out, u_exp_out [B,H_v,T/128,2] (rows 0..63, rows 64..127);
 *   Toff_q_out [B,H_v,T/128,128,128] (required: the second of the call's two launches reads the diagonal blocks back
 *   from it; the upper-right block is written as zeros) with t_exp_out [B,H_v,T/128,3] = exponents of the blocks
 *   (11, 21, 22); dbg_acc_out must be NULL (GDN_ERR_UNSUPPORTED otherwise).
 * Supported: C = 64 or 128, d_k = d_v = 128, 1 <= order <= 3 (the paper's low-bit limit), residual_steps <= 8.
 */
int gdn_chunk_prepare_int8(const int8_t* Kq, const int8_t* Vq, const int32_t* k_exp, const int32_t* v_exp,
                           const uint16_t* beta_q, const int32_t* decay_q,
                           int B, int H_k, int H_v, int T, int C, int d_k, int d_v, int order, int residual_steps,
                           int8_t* Wq_out, int8_t* Uq_out, int32_t* w_exp_out, int32_t* u_exp_out,
                           int8_t* Toff_q_out, int32_t* t_exp_out, int32_t* dbg_acc_out, gdn_stream_t stream);

/*
 * INT16 variant: the paper's primary integer precision for the inverse (Sec. 4.2, Table 1: INT16 within 0.4 dB of
 * FP16; App. G table, row "Matrix Inversion"; quantiser of App. G, Eq. 32). The same chain as
 * gdn_chunk_prepare_int8 with 16-bit mantissas in [-32767, 32767], one power-of-two exponent per chunk, aligned sums
 * that keep 16 bits below their largest term, requantisation after every product and sum with the structural mask
 * applied first. B200 has no 16-bit integer tensor path: every matrix product runs on the 8-bit integer tensor cores
 * over the high and low bytes of the mantissas (four byte-plane products, recombined exactly in 64 bits).
 * The outputs are a pure function of the integer inputs (bit-exact against an exact-integer evaluation).
 *   Kq [B,H_k,T,d_k], Vq [B,H_v,T,d_v] int16 with k_exp [B,H_k,T/C], v_exp [B,H_v,T/C]: value = q * 2^exp;
 *   beta_q, decay_q as for gdn_chunk_prepare_int8.
 *   Wq_out [B,H_v,T,d_k], Uq_out [B,H_v,T,d_v] int16 with w_exp_out, u_exp_out [B,H_v,T/C];
 *   Toff_q_out [B,H_v,T/C,C,C] int16 (may be NULL) with t_exp_out [B,H_v,T/C]: T = I + Toff_q * 2^t_exp.
 *   dbg_acc_out (may be NULL; meant for small cases): the exact matrix products of the chain as int64,
 *   [B,H_v,T/C, C, 8*C + d_k + d_v], laid out as for gdn_chunk_prepare_int8.
 * Supported: C = 64, d_k = d_v = 128, 1 <= order <= 3, residual_steps <= 8.
 */
int gdn_chunk_prepare_int16(const int16_t* Kq, const int16_t* Vq, const int32_t* k_exp, const int32_t* v_exp,
                            const uint16_t* beta_q, const int32_t* decay_q,
                            int B, int H_k, int H_v, int T, int C, int d_k, int d_v, int order, int residual_steps,
                            int16_t* Wq_out, int16_t* Uq_out, int32_t* w_exp_out, int32_t* u_exp_out,
                            int16_t* Toff_q_out, int32_t* t_exp_out, int64_t* dbg_acc_out, gdn_stream_t stream);

/*
 * gdn_chunk_prepare_ex for packed variable-length sequences (one batch of sequences laid end to end along the token
 * axis, as model code passes them with cumulative sequence lengths). Every sequence is cut into chunks of C tokens from
 * its own first token; its last chunk may be shorter. A short chunk is the chunk of C tokens whose missing tokens
 * write nothing (beta = 0, no further decay): the scheme of Sec. 3 runs on it unchanged and only the rows of real
 * tokens are stored.
 *   K [H_k,T_total,d_k], V [H_v,T_total,d_v], beta, g [H_v,T_total], W_out [H_v,T_total,d_k], U_out [H_v,T_total,d_v]
 *   (bf16; or token-major [T_total,H,d] and [T_total,H_v] with GDN_FLAG_LAYOUT_BTHD); g restarts in every chunk (or raw
 *   log-gates with GDN_FLAG_G_RAW).
 *   chunk_start, chunk_len: DEVICE arrays of n_chunks int32: first token and length (1..C) of every chunk, in any
 *   order; chunks must not overlap.
 *   Tinv_out (optional) [H_v, P, C, C] bf16 with P = n_chunks rounded up to a multiple of 128 / C: block c belongs to
 *   chunk c of the table; rows of missing tokens are rows of the identity, blocks c >= n_chunks are identities.
 * flags: GDN_FLAG_G_RAW, GDN_FLAG_K_L2NORM, GDN_FLAG_W_GATED, GDN_FLAG_LAYOUT_BTHD. bf16 only, C in {16, 32, 64, 128},
 * d_k = d_v = 128. Rows of W_out / U_out that no chunk covers are left untouched.
 */
int gdn_chunk_prepare_varlen(const void* K, const void* V, const float* beta, const float* g,
                             const int32_t* chunk_start, const int32_t* chunk_len, int n_chunks, int T_total,
                             int H_k, int H_v, int C, int d_k, int d_v, int order, int residual_steps,
                             void* W_out, void* U_out, void* Tinv_out, unsigned flags, gdn_stream_t stream);

/*
 * The rest of the chunk-wise layer (Sec. 2.1: the quantities W and U exist for this), given W and U of every chunk:
 * state passing between chunks and the output. Per (batch, value head), chunk after chunk, with S the state
 * [d_v x d_k] carried from chunk to chunk:
 *     U_new = U - W S^T
 *     o_i   = scale * ( exp(g_i) S q_i + sum_{j <= i} exp(g_i - g_j) <k_j, q_i> U_new_j )
 *     S    <- exp(g_C) S + sum_j exp(g_C - g_j) U_new_j k_j^T          (g_C: g of the chunk's last token)
 * which equals the token-by-token gated delta rule S_t = a_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,
 * o_t = scale * S_t q_t when W = T diag(beta exp(g)) K (gdn_chunk_prepare_ex with GDN_FLAG_W_GATED) and
 * U = T diag(beta) V.
 *   Q, K [B,H_k,T,d_k], W_gated [B,H_v,T,d_k], U [B,H_v,T,d_v] bf16; g [B,H_v,T] fp32, the cumulative log-gate
 *   that RESTARTS in every chunk (chunk-local inclusive prefix sum), or with flags = GDN_FLAG_G_RAW the raw per-token
 *   log-gates (the prefix sum is then formed here, as gdn_chunk_prepare_ex does); with GDN_FLAG_LAYOUT_BTHD the
 *   tensors are token-major: Q, K [B,T,H_k,d_k], W_gated, U, O_out [B,T,H_v,d], g [B,T,H_v] (the state keeps its
 *   layout); with GDN_FLAG_K_L2NORM the rows of K AND of Q are L2-normalised here (1 / ||k_j|| and 1 / ||q_i|| from the
 *   tiles in shared memory, applied to the products, so a model passes its raw projections to both calls: W_gated then
 *   comes from gdn_chunk_prepare_ex with the same flag); no other flag is accepted; S_in [B,H_v,d_v,d_k] fp32 or NULL
 *   (zero state);
 *   O_out [B,H_v,T,d_v] bf16; S_out [B,H_v,d_v,d_k] fp32 or NULL.
 * Supported: C = 64, d_k = d_v = 128, T a multiple of C. fp32 state, bf16 tensor-core operands.
 * B = 0 is a no-op; with T = 0 nothing is launched and S_out receives S_in (zeros without one).
 */
int gdn_chunk_state_output(const void* Q, const void* K, const void* W_gated, const void* U, const float* g,
                           int B, int H_k, int H_v, int T, int C, int d_k, int d_v, float scale,
                           const float* S_in, void* O_out, float* S_out, unsigned flags, gdn_stream_t stream);

/*
 * gdn_chunk_state_output for packed variable-length sequences (the tensors gdn_chunk_prepare_varlen works on): sequence s
 * holds the tokens [cu_seqlens[s], cu_seqlens[s + 1]) and has its own state. One CTA per (sequence, value head) walks
 * the sequence's chunks from its first token; in a short last chunk the tokens past the end write nothing and the rows
 * of the output past the end are not stored.
 *   Q, K [H_k,T_total,d_k], W_gated [H_v,T_total,d_k], U [H_v,T_total,d_v] bf16; g [H_v,T_total] (restarting in every
 *   chunk of every sequence, or raw with GDN_FLAG_G_RAW); cu_seqlens: DEVICE array of n_seq + 1 int32, non-decreasing,
 *   cu_seqlens[n_seq] <= T_total; S_in, S_out [n_seq,H_v,d_v,d_k] fp32 (either may be NULL); O_out [H_v,T_total,d_v].
 *   With GDN_FLAG_LAYOUT_BTHD: Q, K [T_total,H_k,d_k], W_gated, U, O_out [T_total,H_v,d], g [T_total,H_v].
 * Supported: C = 64, d_k = d_v = 128.
 */
int gdn_chunk_state_output_varlen(const void* Q, const void* K, const void* W_gated, const void* U, const float* g,
                                  const int32_t* cu_seqlens, int n_seq, int T_total, int H_k, int H_v, int C,
                                  int d_k, int d_v, float scale, const float* S_in, void* O_out, float* S_out,
                                  unsigned flags, gdn_stream_t stream);

/*
 * gdn_chunk_state_output for FEW LONG sequences (one per value head, B = 1): the chunks of a sequence are a serial
 * chain, so with fewer sequences than SMs most of the GPU idles. Here every sequence is cut into `segments` runs of
 * whole chunks. The state at the end of a segment is an affine map of the state at its start, S_end = S_start M + N
 * (M: d_k x d_k, N: d_v x d_k): a first pass forms N (the segment from a zero state) and M (the segment from the
 * identity with U = 0) of every segment in parallel, without queries or output; a short recurrence gives every
 * segment's initial state; a second pass runs all segments in parallel with their output. Three passes' worth of
 * state work instead of one, on `segments` times as many SMs.
 *   Tensors as gdn_chunk_state_output with B = 1 (head-major [H,T,d], or [T,H,d] with GDN_FLAG_LAYOUT_BTHD).
 *   segments: 1 = the plain call; gdn_chunk_state_segments(H_v) proposes the count that fills the SMs in one wave.
 *   workspace: DEVICE memory of gdn_chunk_state_segmented_workspace(H_v, segments) bytes, 16-byte aligned, owned by
 *   the caller and free to reuse when the stream has passed the call.
 * The result differs from the plain call by fp32 rounding of the state recurrence only.
 */
int gdn_chunk_state_segments(int H_v);
size_t gdn_chunk_state_segmented_workspace(int H_v, int segments);
int gdn_chunk_state_output_segmented(const void* Q, const void* K, const void* W_gated, const void* U, const float* g,
                                     int H_k, int H_v, int T, int C, int d_k, int d_v, float scale,
                                     const float* S_in, void* O_out, float* S_out, int segments,
                                     void* workspace, size_t workspace_bytes, unsigned flags, gdn_stream_t stream);

/*
 * gdn_chunk_state_output_segmented without a workspace argument (the paper has no counterpart: this is a
 * convenience of the library). It is meant for callers that must not, or cannot, allocate device memory around
 * the call: code running inside an inference engine that handed out all of the GPU's memory at start-up, a plug-in
 * with no allocator of its own, a real-time loop in which cudaMalloc's implicit synchronisation is not acceptable.
 * The scratch memory the segmented form needs (the segments' state maps and initial states) is a fixed array of
 * device memory built into the library, 8 MB + 4 KB, which every GPU that loads the library holds until the
 * process exits. The call allocates and frees nothing, neither directly nor through another library.
 *   Arguments, layouts, flags and results: exactly those of gdn_chunk_state_output_segmented (the same kernels run).
 *   Limit: H_v * (6 * segments - 6) <= 128 (the number of 128 x 128 fp32 state blocks the array holds; e.g. 8 value
 *   heads in 3 segments, 4 in 6, 16 in 2), where segments is first clamped to the number of chunks. A larger problem
 *   returns GDN_ERR_SCRATCH and launches nothing: use the variant with a workspace there. segments = 1 needs no
 *   scratch and is always accepted.
 *   First call on a device: the library looks up the device address of its array (with that device current, once
 *   per device). Make that first call outside any stream capture.
 *   Sharing: all calls on a device use the same array, and the array keeps what the last call left in it. Every
 *   call writes all the scratch it later reads, so nothing has to be cleared between calls, but two calls that
 *   overlap on the GPU (different streams, or different host threads) race on it: keep calls of this entry point
 *   on one stream, or order them with events.
 */
int gdn_chunk_state_output_segmented_noalloc(const void* Q, const void* K, const void* W_gated, const void* U,
                                             const float* g, int H_k, int H_v, int T, int C, int d_k, int d_v,
                                             float scale, const float* S_in, void* O_out, float* S_out, int segments,
                                             unsigned flags, gdn_stream_t stream);

/* Checksum of the 256-entry gate-decay table round(2^15 * 2^(-f/256)) the INT8 kernel uses
 * (sum_f: s = (31 s + table[f] + f) mod 1000000007), so that a CPU evaluation can confirm it holds the same table. */
unsigned int gdn_int8_lut_checksum(void);

/*
 * Waits for `stream`, then returns and clears the status word the kernels of
 * this library write on the current device: GDN_OK, or GDN_ERR_TIMEOUT when a
 * bounded wait inside a kernel gave up (its outputs are then undefined).
 * This is the only call that synchronises.
 */
int gdn_device_status(gdn_stream_t stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper): launches one small kernel that waits, with the
 * same wait routine and budget (about a second) as the compute kernels, on an mbarrier that nothing ever
 * completes. The wait gives up, the kernel records GDN_ERR_TIMEOUT and returns normally: the next
 * gdn_device_status(stream) reports GDN_ERR_TIMEOUT once, and the context stays usable. Returns GDN_OK when
 * the kernel was enqueued.
 */
int gdn_selftest_bounded_wait(gdn_stream_t stream);

/* Paper's parameters per chunk size: N = 3 (C - 1 for chunks of 2 or 3 tokens); S = 8 for C = 64 (Sec. 4.1) and for the
 * 64-blocks of C = 128 (App. H), S = 4 for C = 32 (Sec. 4.3); C = 16 is not in the
 * paper: S = 3, which makes the result exact. Other C: S = ceil(C/4) - 1. */
int gdn_default_order(int C);
int gdn_default_residual_steps(int C);

/* Human-readable name of a gdn_status value (static storage). */
const char* gdn_status_string(int status);

/* Number of kernels this library has launched in this process (for benchmarks that
 * must report how many of the library's own kernels ran inside a timed region). */
long long gdn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GDNPREP_H_ */
