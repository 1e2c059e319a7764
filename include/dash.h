/*
 * dash.h -- C ABI of the B200 (sm_100a) halted-prefill library.
 *
 * The library implements, for one Transformer block during prefill, the hot
 * path of DASH (Delta Attention Selective Halting): the token-wise
 * delta-attention score, the halting rule, the order-preserving compaction of
 * the still-active tokens (with the frozen states of halted tokens written back
 * to the full-length output), and causal grouped-query attention over the
 * compacted active set.
 *
 * Conventions that hold for every entry point
 *  - Every function returns an int status (DASH_OK = 0 or a DASH_ERR_* code).
 *    Nothing throws, aborts or traps; invalid arguments are rejected before
 *    any kernel is launched.
 *  - Unless a parameter says "host", tensor pointers are DEVICE pointers owned
 *    by the caller; they must stay valid until the work enqueued on `stream`
 *    has finished.  The library allocates no device memory: scratch comes from
 *    the caller's `ws` (size from dash_workspace_bytes), 256-byte aligned.
 *  - `stream` is a cudaStream_t passed as void*.  All work is enqueued
 *    asynchronously; no call synchronises except dash_check_status.
 *  - Data-dependent sizes (number of active tokens, new sequence boundaries)
 *    are written to device memory; the caller sizes outputs for the upper
 *    bound it passes (`n`, the number of rows allocated).  Where a
 *    `cu_seqlens` array is given, the true row count is cu_seqlens[S] (read on
 *    the device) and rows at or beyond it are neither read nor written.
 *  - Row-major tensors; `ld*` are row strides in ELEMENTS, `*_ld_bytes` in
 *    bytes.  Data pointers and row strides must be multiples of 16 bytes.
 *  - Kernels that wait (tile look-back, TMA/MMA barriers) give up after a
 *    bounded number of polls and set DASH_ERR_TIMEOUT in a device status word
 *    that dash_check_status returns.
 */
#ifndef DASH_H_
#define DASH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DASH_OK               0
#define DASH_ERR_INVALID_ARG  1
#define DASH_ERR_UNSUPPORTED  2
#define DASH_ERR_WORKSPACE    3
#define DASH_ERR_CUDA         4
#define DASH_ERR_TIMEOUT      5
#define DASH_ERR_TOO_LARGE    6

typedef enum { DASH_F32 = 0, DASH_BF16 = 1 } dash_dtype;
/* REL: ||U_t|| / ||H_t|| (the "relative" delta-attention of Fig. 1);
 * ABS: ||U_t||           (Eq. 2). */
typedef enum { DASH_NORM_REL = 0, DASH_NORM_ABS = 1 } dash_norm_mode;
/* The _HALT_HIGH variants are the paper's direction ablation ("High Delta_attn"): the same rules on the
 * negated scores -- a token halts iff r > tau, or the smallest scores stay. */
typedef enum { DASH_SEL_THRESHOLD = 0, DASH_SEL_KEEP_COUNT = 1,
               DASH_SEL_THRESHOLD_HALT_HIGH = 2, DASH_SEL_KEEP_COUNT_HALT_HIGH = 3 } dash_sel_mode;
/* Score of dash_block_step: the attention branch's update (Eq. 2, the method) or the change over the whole
 * block, ||H' - H|| (the paper's ablation of the delta signal). */
typedef enum { DASH_SIGNAL_ATTN = 0, DASH_SIGNAL_BLOCK = 1 } dash_signal;

#define DASH_MAX_ROW_STREAMS 8

const char* dash_status_string(int status);

/* Synchronises `stream`, returns the device status word (DASH_OK or
 * DASH_ERR_TIMEOUT) and clears it. */
int dash_check_status(void* stream);

/* ---- host helpers (pure, no device work) --------------------------------
 * Kept length.  mode 0: Eq. 3, K = floor((1 - rho) * n).
 * mode 1: Appendix A: the first keep_first and last keep_last tokens always
 * stay and floor(round(rho * (n - keep_first - keep_last))) of the others are
 * dropped (round = to nearest, ties to even).  Returns -1 on invalid input. */
int64_t dash_keep_count(int64_t n, double rho, int keep_first, int keep_last, int mode);

/* The same kept lengths on the device, one per sequence, from the sequence lengths as they
 * stand in cu_seqlens (device int32 [S+1]): keep_counts_out[s] (device int32 [S]) =
 * dash_keep_count(cu[s+1] - cu[s], ...), the same fp64 arithmetic.  For dash_select's
 * keep-count rule in layers whose entering lengths exist only on the device (behind a
 * selecting layer), so that no length has to come back to the host.  Asynchronous on
 * `stream`.  DASH_ERR_INVALID_ARG for null pointers, S < 1, rho outside [0, 1), negative
 * keep_first / keep_last or a mode other than 0 / 1. */
int dash_keep_counts_device(const int32_t* cu_seqlens, int S, double rho, int keep_first, int keep_last,
                            int mode, int32_t* keep_counts_out, void* stream);
/* Appendix A FLOPs proxy of one block: A(n) = 4 n d^2 + 2 n^2 d + 2 n d m. */
double dash_flops_per_layer(double n, double d, double m);
/* Appendix A: C_full / C_ours with C_full = L A(n), C_ours = l_s A(n) + (L - l_s) A(n_hat). */
double dash_flops_speedup(double n, double n_hat, int L, int l_s, double d, double m);

/* ---- step 1: delta-attention score (Eq. 1-2; Fig. 1 "relative") ----------
 * Optional halting rule fused into the same pass (step 2, THRESHOLD mode):
 * a token halts iff r_t < tau and it is not among the first keep_first / last
 * keep_last tokens of its sequence (Appendix A). */
typedef struct {
    float          tau;
    int            keep_first, keep_last;
    const int32_t* cu_seqlens;   /* device [S+1] */
    int            S;
    uint8_t*       mask_out;     /* device [n], 1 = stays active */
} dash_threshold;

/* r_out[t] = ||U_t||_2 / max(||H_t||_2, eps)  (REL)  or  ||U_t||_2  (ABS), fp32
 * accumulation.  U, H: [n, d] of type dt, d % 8 == 0.  If Hres_out != NULL the
 * residual update H~_t = H_t + U_t (Preliminaries) is written in the same pass
 * (Hres_out may be H or U itself, same rows and stride).  If res_index != NULL
 * (device int32 [n]), row t of the residual is written to row res_index[t] of
 * Hres_out instead of row t; Hres_out must then overlap neither input
 * (DASH_ERR_INVALID_ARG).
 * fused: NULL, or the threshold rule above.  n_dev: NULL, or a device int32
 * holding the true row count (<= n). */
int dash_delta_norm(const void* U, const void* H, int64_t n, int d, int64_t ldU, int64_t ldH,
                    dash_dtype dt, dash_norm_mode mode, float eps, float* r_out,
                    void* Hres_out, int64_t ldHres, const int32_t* res_index,
                    const dash_threshold* fused, const int32_t* n_dev, void* stream);

/* ---- step 2: halting rule (Eq. 3; Appendix A protected prefix/suffix) -----
 * THRESHOLD: mask[t] = protected(t) || !(r[t] < tau)   (NaN stays active).
 * KEEP_COUNT: per sequence s, keep_counts[s] (device int32 [S]) tokens stay in
 *   total: the protected ones plus the largest scores of the others; ties at
 *   the cut are broken toward the lower index; NaN ranks as +inf.
 * THRESHOLD_HALT_HIGH / KEEP_COUNT_HALT_HIGH: the same on -r (random halting needs no mode:
 *   pass random scores).
 * r: device fp32 [n]; cu_seqlens: device int32 [S+1] over the current packed
 * order; mask_out: device u8 [n] (1 = stays active).  Needs no workspace (the
 * radix select of the keep-count rule works in shared memory, one CTA per sequence). */
int dash_select(const float* r, int64_t n, const int32_t* cu_seqlens, int S,
                dash_sel_mode mode, float tau, const int32_t* keep_counts,
                int keep_first, int keep_last, uint8_t* mask_out, void* stream);

/* ---- step 3: compaction / scatter (Sec. 3.4; Alg. 1 "gathering tokens") ---
 * One row tensor moved by the scan: dst[k] = src[idx[k]], rows of row_bytes
 * (multiple of 4; 16-byte vector path when pointers, strides and row_bytes
 * allow it). */
typedef struct {
    const void* src;
    void*       dst;
    int64_t     row_bytes, src_ld_bytes, dst_ld_bytes;
} dash_rows;

/* Exclusive prefix sum of mask (single pass, decoupled look-back) and stable
 * gather of the active rows.  Outputs (device): idx_out[k] = source row of
 * output row k (int32 [n]); cu_out int32 [S+1] = new packed boundaries;
 * n_out_dev int32 = number of active rows (= cu_out[S]).  pos / tok (int32 per
 * row: rotary position, row in the full-length buffer) are gathered when both
 * the _in and _out pointer are non-NULL.  Any of idx_out, rows, pos, tok may be
 * absent.  ws: dash_workspace_bytes(DASH_WS_COMPACT, n, S, ...). */
int dash_compact(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                 const dash_rows* rows /*host array*/, int n_rows,
                 const int32_t* pos_in, int32_t* pos_out,
                 const int32_t* tok_in, int32_t* tok_out,
                 int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev,
                 void* ws, size_t ws_bytes, void* stream);

/* Same operation and arguments as dash_compact, for callers that cannot hand over a
 * workspace because they are not allowed to allocate device memory at all: a serving
 * loop whose device memory was handed out in full at start-up, or a plug-in whose host
 * forbids allocation calls on its worker threads (they synchronise the device).  (The
 * paper has no counterpart: it describes the method, not a memory policy.)
 * The look-back scratch lives in a fixed array inside the library instead, which every
 * GPU that loads the library holds until the process exits (256 KiB + 512 B).
 *  - Limit: n <= DASH_COMPACT_STATIC_MAX_ROWS; larger inputs are rejected with
 *    DASH_ERR_TOO_LARGE before anything is enqueued.
 *  - Allocates nothing (no cudaMalloc / cudaFree, no allocating library routine); the
 *    part of the array a call uses is cleared on `stream` before its kernel runs.
 *  - The first call on a device looks up the device address of the array (with that
 *    device current); make that first call before any stream capture begins.
 *  - All calls on one device share the array and it keeps the last call's contents:
 *    two calls whose kernels may overlap on the GPU (different streams) race.  Calls on
 *    one stream are safe. */
#define DASH_COMPACT_STATIC_MAX_ROWS (1 << 20)
int dash_compact_static(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                        const dash_rows* rows /*host array*/, int n_rows,
                        const int32_t* pos_in, int32_t* pos_out,
                        const int32_t* tok_in, int32_t* tok_out,
                        int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev, void* stream);

/* dst_full[tok_index[i]] = src[i] for every i < n with sel[i] == which
 * (which: 0 halted rows, 1 active rows, 2 every row; sel may be NULL for 2).
 * tok_index NULL means the identity.  n_dev: NULL or device true row count. */
int dash_scatter(const void* src, int64_t n, int64_t row_bytes, int64_t src_ld_bytes,
                 const int32_t* tok_index, const uint8_t* sel, int which, const int32_t* n_dev,
                 void* dst_full, int64_t dst_ld_bytes, void* stream);

/* ---- step 4: causal GQA attention over the packed active set -------------
 * For sequence s, query head h, packed row i in [cu[s], cu[s+1]):
 *   O[i,h,:] = sum_{cu[s] <= j <= i} softmax_j(scale * q_i . k_j) v_j,
 * key/value head h / (Hq / Hkv).  Only tokens present in the packed buffers
 * own keys/values (halted tokens contribute none; Sec. 3.4).
 * Q [n,Hq,D], O [n,Hq,D], K,V [n,Hkv,D] of type dt with row strides ldq, ldo,
 * ldk, ldv (elements).  bf16 tensor-core math with fp32 accumulation and fp32
 * softmax; DASH_F32 tensors are converted to bf16 on the way in (needs ws).
 * lse: NULL or fp32 [Hq, n] = log-sum-exp of the scaled scores.
 * D in {64, 128}; Hq % Hkv == 0; causal must be 1.  n: rows allocated;
 * max_seqlen: upper bound of the longest sequence (grid sizing). */
int dash_varlen_attention(const void* Q, const void* K, const void* V, void* O, float* lse,
                          int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                          const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen,
                          int Hq, int Hkv, int D, float scale, int causal, dash_dtype dt,
                          void* ws, size_t ws_bytes, void* stream);

/* The same attention with Q left where it is (Sec. 3.4: the active tokens are "gathered";
 * here the gathering happens inside the tile loads).  Q [n_full,Hq,D] is a full-length
 * tensor; packed row i of the active set is its row idx[i] (device int32 [n], e.g.
 * dash_compact's idx_out: ascending within a sequence).  kv_packed = 1: K, V [n,Hkv,D] are
 * packed (compacted by the caller: 2 * 2 Hkv * D * es bytes per active token instead of
 * 2 * (Hq + 2 Hkv) * D * es) -- the fast arrangement, a query tile is fetched once.
 * kv_packed = 0: K, V [n_full,Hkv,D] are full-length too and every key block is fetched by
 * index: no copy at all, but each query tile gathers its keys again, four rows per load --
 * measured 2.5x slower than packed K, V (with packed K, V the call is within 1-3 % of
 * dash_varlen_attention on packed Q).  cu_seqlens, S, n, max_seqlen describe the packed
 * set as above; O [n,Hq,D] and lse [Hq,n] are written packed.  DASH_BF16 only
 * (DASH_ERR_UNSUPPORTED for fp32); every idx[i] must lie in [0, n_full) -- not checked on
 * the device. */
int dash_varlen_attention_indexed(const void* Q, const void* K, const void* V, void* O, float* lse,
                                  int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                                  const int32_t* idx, int64_t n_full, int kv_packed,
                                  const int32_t* cu_seqlens, int S, int64_t n, int64_t max_seqlen,
                                  int Hq, int Hkv, int D, float scale, int causal, dash_dtype dt,
                                  void* ws, size_t ws_bytes, void* stream);

/* ---- decoding stage: one new token per sequence over the packed KV cache ---
 * (Preliminaries: decoding reuses the cached keys and values; Appendix C, "DASH settings":
 * halting prompt tokens shortens the KV cache -- the cache of a deeper layer holds only the
 * tokens that stayed active, i.e. the K and V rows a block step emits.)
 * For sequence s and query head h:  out[s,h,:] = sum_j softmax_j(scale * q[s,h] . Kc[j,kv]) Vc[j,kv,:]
 * over the cached rows cu[s] <= j < cu[s+1], kv = h / (Hq / Hkv); no mask.  An empty cache gives 0
 * (lse = -inf).  q [S,Hq,D], out [S,Hq,D], Kc, Vc [n,Hkv,D], all DASH_BF16 (DASH_F32 is
 * unsupported: the cache is read as stored), row strides ldq, ldo, ldk, ldv in elements.
 * lse: NULL or fp32 [S,Hq].  Hq / Hkv <= 8; D in {64, 128}.  ws: dash_workspace_bytes(DASH_WS_DECODE). */
int dash_decode_attention(const void* q, const void* Kc, const void* Vc, void* out, float* lse,
                          int64_t ldq, int64_t ldk, int64_t ldv, int64_t ldo,
                          const int32_t* cu_seqlens, int S, int64_t n, int Hq, int Hkv, int D, float scale,
                          dash_dtype dt, void* ws, size_t ws_bytes, void* stream);

/* ---- the whole block step (Alg. 1, loop body without the FFN) ------------ */
typedef struct {
    int          d, Hq, Hkv, D;
    dash_dtype   dt;               /* type of H, weights, x_full, H_next */
    const void*  Wqkv;             /* [d, (Hq + 2 Hkv) D]: columns = Wq | Wk | Wv */
    const void*  Wo;               /* [Hq D, d] */
    const void*  rms_weight;       /* [d] */
    float        rms_eps;
    double       rope_base;
    dash_norm_mode norm_mode;
    float        norm_eps;
    dash_sel_mode  sel_mode;
    float        tau;              /* THRESHOLD */
    const int32_t* keep_counts;    /* KEEP_COUNT: device int32 [S] */
    int          keep_first, keep_last;
    int          scatter_which;    /* rows of H~ written to x_full: 0 halted, 2 all */
    void*        k_cache;          /* NULL, or [n, Hkv, D]: this block's keys (rotary applied) of the entering tokens, */
    void*        v_cache;          /* and values: the rows a decoding step attends over at this depth (both or neither) */
    int          rms_folded;       /* 1: the norm's weight is already in Wqkv (dash_fold_norm_weight; rms_weight may then be NULL):
                                    * the norm costs no pass of its own -- one pass over H yields the row factors 1 / rms, which
                                    * the projection applies to its accumulators.  Only where the projections run with their
                                    * fused epilogues (see below); DASH_ERR_UNSUPPORTED otherwise. */
    /* What a prefill can hand from block to block instead of recomputing it (all optional; they need rms_folded = 1,
     * DASH_ERR_UNSUPPORTED otherwise):                                                                                   */
    const void*  rope_table;       /* NULL, or the (cos, sin) pairs of dash_rope_table for positions 0 .. rope_table_len - 1 (same
                                    * rope_base and D): the rotary angles of a row are looked up by its position instead of
                                    * being formed in every block (positions beyond the table use its last entry) */
    int64_t      rope_table_len;
    const float* inv_rms_in;       /* NULL, or fp32 [n]: 1 / sqrt(mean(H_in[t]^2) + rms_eps) of every entering row, e.g. the
                                    * inv_rms_next of the block step that produced H_in: no pass over H_in is needed then */
    float*       inv_rms_next;     /* NULL, or fp32 [n]: receives that row factor for every row of H_next (from the sums the step
                                    * has at hand), for the next block's inv_rms_in */
} dash_layer_cfg;
/* The projections (Wqkv, Wo; Wgu, Wd of dash_block_step) run in this library's tcgen05 GEMMs (256 x 256 tiles on CTA pairs).
 * bf16 tensors whose projections have whole 256-column tiles ((Hq + 2 Hkv) D, (Hq + Hkv) D and d multiples of 256, d and Hq D
 * multiples of 64; the FFN width a multiple of 128) get the work that follows a projection on its accumulators: the rotary
 * embedding in the QKV projection; H~ and the score's row sums in the output projection; SwiGLU in the gate | up projection --
 * one rounding less per value, no U and no gate | up intermediate.  Other shapes (rows must still start on 16-byte boundaries:
 * d, Hq D, m multiples of 8) and fp32 tensors run the same GEMM kernel plain, with the norm, the rotary embedding, the residual
 * and the score as passes of their own; fp32 operands are rounded to bf16 copies in the workspace first (fp32 accumulation,
 * fp32 results), as the attention kernel does with Q, K, V. */

/* LN of Eq. 1 is read as RMSNorm, y = x / rms(x) * w.  Its weight w can be folded, once and ahead of time, into the
 * projection that follows the norm: W_out[i, j] = w[i] * W[i, j] for W, W_out [d, N] row-major of type dt (row strides ldw,
 * ldo in elements, multiples of 16 bytes) and w [d] of type dt; the product is formed in fp32 and rounded once.  A block
 * configured with rms_folded = 1 (rms2_folded = 1 for the norm in front of the FFN) expects such a matrix as Wqkv (Wgu): the
 * norm then costs no pass of its own.  W_out may be W itself.  Asynchronous on `stream`.  DASH_ERR_INVALID_ARG for null or
 * misaligned pointers, d < 1, N < 1, N not a multiple of 8 (bf16) / 4 (fp32), strides smaller than N. */
int dash_fold_norm_weight(const void* W, const void* rms_weight, int d, int64_t N, int64_t ldw, dash_dtype dt,
                          void* W_out, int64_t ldo, void* stream);

/* Rotary angles once per prefill (the rotary embedding inside Attn of Eq. 1; rotate-half pairs (i, i + D/2), angle
 * pos * rope_base^(-2i/D)): table[pos * (D/2) + i] = (cos, sin) as two fp32, for pos = 0 .. n_pos - 1; the angle is formed and
 * reduced in fp64, its sine and cosine evaluated in fp32.  table: device, n_pos * (D/2) * 8 bytes, 8-byte aligned.  A block
 * step whose cfg.rope_table points here looks the angles up by position instead of forming them again in every block.
 * Asynchronous on `stream`.  DASH_ERR_INVALID_ARG for a null table, n_pos < 1, rope_base <= 0 or D not in {64, 128}. */
int dash_rope_table(double rope_base, int D, int64_t n_pos, void* table, void* stream);

/* Byte offsets of the intermediates inside the workspace of dash_layer_step
 * (for inspection by tests and tools).  Ht (H~ = H + U) is only written when the
 * halting rule is KEEP_COUNT or scatter_which is 0; with the threshold rule and
 * scatter_which = 2 the score, the residual, the scatter and the compaction run as
 * one pass that writes H~ straight to x_full and H_next. */
typedef struct {
    size_t Hn, QKV, O, U, Ht, scratch, total;
} dash_layer_ws_layout;
int dash_layer_workspace(const dash_layer_cfg* cfg, int64_t n, int S, dash_layer_ws_layout* out);

/* H_in [n, d]: packed hidden states of the tokens entering the block, with
 * tok_index_in (row in the full-length buffer), pos_in (rotary position) and
 * cu_in [S+1] (device).  Runs RMSNorm -> QKV projection -> rotary embedding ->
 * causal attention -> output projection U -> r, H~ = H + U -> halting rule ->
 * scatter of H~ into x_full [T, d] -> compaction of the tokens that stay
 * active into H_next / tok_index_next / pos_next / cu_next / n_next_dev.
 * r_out fp32 [n], mask_out u8 [n].  No host synchronisation.  x_full must not
 * overlap H_in (unless tok_index_in is the identity and the rows coincide). */
int dash_layer_step(const dash_layer_cfg* cfg, const void* H_in, const int32_t* tok_index_in,
                    const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n, int64_t max_seqlen,
                    void* x_full, void* H_next, int32_t* tok_index_next, int32_t* pos_next,
                    int32_t* cu_next, int32_t* n_next_dev, float* r_out, uint8_t* mask_out,
                    void* ws, size_t ws_bytes, void* stream);

/* ---- the whole block of Alg. 1, feed-forward included ----------------------
 * H' = H~ + FFN(LN(H~)) with H~ = H + U as above; the score and the selection still
 * come from U.  FFN is the gated feed-forward of the Qwen2.5 backbones:
 * FFN(x) = (silu(x Wg) * (x Wu)) Wd.  H' of every entering token is written to x_full
 * (attn.scatter_which must be 2: H' is also the last updated value of the tokens that
 * halt here, Sec. 3.4), H' of the tokens that stay to H_next. */
typedef struct {
    dash_layer_cfg attn;
    int          m;                /* feed-forward width, multiple of 8 */
    const void*  Wgu;              /* [d, 2 m]: columns = Wg | Wu */
    const void*  Wd;               /* [m, d] */
    const void*  rms2_weight;      /* [d]: weight of the norm in front of the FFN (attn.rms_eps is used) */
    dash_signal  signal;           /* what the score measures */
    int          rms2_folded;      /* as attn.rms_folded, for the norm in front of the FFN and Wgu (needs DASH_SIGNAL_ATTN and attn.rms_folded) */
} dash_block_cfg;
typedef struct {
    dash_layer_ws_layout attn;
    size_t GU, ACT, F, total;      /* gate | up [n, 2m], activation [n, m], FFN output [n, d] */
} dash_block_ws_layout;
int dash_block_workspace(const dash_block_cfg* cfg, int64_t n, int S, dash_block_ws_layout* out);
/* Arguments as dash_layer_step. */
int dash_block_step(const dash_block_cfg* cfg, const void* H_in, const int32_t* tok_index_in,
                    const int32_t* pos_in, const int32_t* cu_in, int S, int64_t n, int64_t max_seqlen,
                    void* x_full, void* H_next, int32_t* tok_index_next, int32_t* pos_next,
                    int32_t* cu_next, int32_t* n_next_dev, float* r_out, uint8_t* mask_out,
                    void* ws, size_t ws_bytes, void* stream);

/* ---- workspace sizes ------------------------------------------------------ */
typedef enum { DASH_WS_COMPACT = 1, DASH_WS_ATTENTION = 2, DASH_WS_DECODE = 3 } dash_ws_op;
/* n: rows allocated; S: sequences; Hq, Hkv, D, dt only matter for attention. */
size_t dash_workspace_bytes(dash_ws_op op, int64_t n, int S, int Hq, int Hkv, int D, dash_dtype dt);

#ifdef __cplusplus
}
#endif
#endif /* DASH_H_ */
