/*
 * lrsa.h - C ABI of the B200 (sm_100a) Lag-Relative Sparse Attention library.
 *
 * The library computes the data-parallel hot path of LRSA post-training:
 *   1. lrsa_score_select : LagKV token scores (Section 3.2, Eq. 4-8) and the top-K kept
 *                          positions of every lag window (text after Eq. 8),
 *   2. lrsa_attn_fwd     : masked softmax attention (Section 3.1, Eq. 3) under the static
 *                          chunked mask of Section 3.2 (Attn-Fill 1 / Attn-Fill 2),
 *   3. lrsa_attn_bwd     : its gradient with the mask held constant.
 *
 * Conventions common to every call
 * --------------------------------
 * Tensors  : row-major, contiguous, bf16 unless stated.  Q, O, dO, dQ are [batch, n_q_heads,
 *            seq_len, head_dim]; K, V, dK, dV are [batch, n_kv_heads, seq_len, head_dim].
 *            Query head h uses KV head h / (n_q_heads / n_kv_heads).
 * Pointers : every tensor/workspace pointer is a DEVICE pointer owned by the caller, aligned to
 *            16 bytes (workspace: 256 bytes).  `params` is a HOST pointer.  The library
 *            allocates no device memory and keeps no state between calls.
 * Geometry : positions [0, S) are sinks.  Window w covers [S + w*L, S + (w+1)*L).
 *            W = floor((N-S)/L) full windows, tail T = N - S - W*L (< L) tokens.
 *            W_sel = max(W-1, 0) windows have a full following window and are scored.
 * Packed   : with n_seqs > 0 each sequence [cu_seqlens[s], cu_seqlens[s+1]) is an independent problem
 *            (Section 3.2 applied to it alone): its sinks and windows are counted from its first token
 *            (a sequence shorter than S is all sinks) and no query sees another sequence.  Scored
 *            windows are numbered sequence after sequence, W_sel is their total, and kept positions
 *            are positions on the packed token axis.  The sequences are processed one after the
 *            other on the stream.
 * Stream   : `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *            enqueue work and return without synchronising.  Two calls that use the same
 *            workspace must be ordered (same stream, or otherwise serialised).
 * Errors   : the int return value is an lrsa_status.  All argument checks happen on the host
 *            before anything is enqueued; on a non-zero status nothing was launched, except
 *            LRSA_ERR_CUDA which reports a launch failure of the CUDA runtime.
 *            Device-side waits are bounded; if one expires the kernel records it in the
 *            workspace and lrsa_workspace_status returns LRSA_ERR_TIMEOUT (outputs are
 *            then undefined).
 */
#ifndef LRSA_H_
#define LRSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lrsa_status {
  LRSA_OK = 0,
  LRSA_ERR_INVALID_ARG = 1,         /* null pointer, non-positive size, K > L, Hq % Hkv != 0, misaligned */
  LRSA_ERR_UNSUPPORTED = 2,         /* head_dim not in {64,128}, chunk not a multiple of lag, seq_len < n_sink, ... */
  LRSA_ERR_WORKSPACE_TOO_SMALL = 3,
  LRSA_ERR_CUDA = 4,                /* CUDA runtime error while enqueueing */
  LRSA_ERR_TIMEOUT = 5              /* a bounded device-side wait expired */
} lrsa_status;

typedef struct lrsa_params {
  int32_t batch;         /* B >= 1 */
  int32_t n_q_heads;     /* Hq, multiple of n_kv_heads (GQA) */
  int32_t n_kv_heads;    /* Hkv */
  int32_t seq_len;       /* N >= n_sink */
  int32_t head_dim;      /* d in {64, 128} */
  int32_t chunk;         /* query chunk size: a positive multiple of lag.  The mask of Section 3.2 does not
                            depend on how many lag windows are filled at a time ("the number of filling chunks
                            can be optimized"), so every multiple gives the results of chunk == lag */
  int32_t lag;           /* L, lag window size */
  int32_t top_k;         /* K = r*L kept tokens per window, 1 <= K <= L */
  int32_t n_sink;        /* S >= 0 */
  int32_t n_dense_prev;  /* 1: the window just before the query chunk is seen uncompressed (the
                            paper's "sliding window"); 0: it is compressed too when scored */
  int32_t std_ddof;      /* divisor of the per-token Std is head_dim - std_ddof; 0 or 1 */
  float softmax_scale;   /* 0 -> 1/sqrt(head_dim) as in Eq. 3 */
  int32_t n_seqs;        /* 0: every batch element is one sequence of seq_len tokens.  > 0: packed batch, the
                            token axis of every batch element holds n_seqs sequences back to back */
  const int32_t* cu_seqlens; /* HOST pointer, n_seqs + 1 boundaries: cu_seqlens[0] = 0, increasing,
                            cu_seqlens[n_seqs] = seq_len.  Read during the call only.  NULL when n_seqs = 0 */
  void* o_residual;      /* optional DEVICE pointer, bf16 [B, Hq, N, d], 16-byte aligned, or NULL.  The paper has no
                            counterpart: it is the part of the attention output that the bf16 O cannot hold.
                            lrsa_attn_fwd writes bf16(O_fp32 - O) there; lrsa_attn_bwd, given the buffer the
                            forward of the same inputs filled, takes the D = rowsum(dO * O) that dK is formed
                            with over O + o_residual.  That removes the rounding of O from dK (it matters where
                            a query puts nearly all its weight on one key); dQ does not depend on it (its D is
                            the exact sum_j P dP) and dV has no D.  The other calls ignore the field. */
} lrsa_params_t;

/* Number of scored windows W_sel (see Geometry).  idx has W_sel * top_k entries per KV head. */
int lrsa_num_sel_windows(const lrsa_params_t* params, int32_t* w_sel);

/* Workspace sizes in bytes for the three calls (any output pointer may be NULL). */
int lrsa_workspace_bytes(const lrsa_params_t* params, size_t* score_select, size_t* attn_fwd,
                         size_t* attn_bwd);

/*
 * LagKV scoring and selection (Section 3.2, Eq. 4-8 and the selection rule after Eq. 8).
 * For every batch element, KV head and scored window p: per-channel min and max over the tokens
 * of window p+1 (Eq. 4, 5) normalise window p (Eq. 6); the per-token standard deviation over
 * head_dim, soft-maxed over the L tokens of the window (Eq. 7), is computed for K and for V and
 * the two are added (Eq. 8); the top_k highest-scoring positions are kept.  A channel whose
 * reference range is zero contributes normalised value 0.  Arithmetic is fp32.
 *
 *   K, V   in  : bf16 [B, Hkv, N, d]
 *   idx    out : int32 [B, Hkv, W_sel, top_k], absolute positions in [0, N), ascending inside
 *                a window; equal scores keep the lower position.
 *   score  out : optional (NULL to skip), fp32 [B, Hkv, W_sel, L], the Eq. 8 score.
 */
int lrsa_score_select(const lrsa_params_t* params, const void* K, const void* V, int32_t* idx,
                      float* score, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Same computation and outputs as lrsa_score_select, for callers that can neither supply a
 * workspace nor let the library allocate one (the paper has no counterpart; this is a packaging
 * variant).  Typical case: a plugin running inside a process whose caching allocator already owns
 * all device memory, or a loop that must not enter cudaMalloc/cudaFree because of their device-wide
 * synchronisation.  The scratch is a fixed array of LRSA_STATIC_SCRATCH_BYTES inside the library's
 * device image: every GPU that loads the library holds that much memory until the process exits.
 *
 *   - Allocates nothing: no cudaMalloc/cudaFree, no allocating library routine.  The caller still
 *     passes K, V (in) and idx, score (out; score may be NULL) exactly as for lrsa_score_select.
 *   - Problems whose scratch need (the score_select figure of lrsa_workspace_bytes: 256 bytes for lag
 *     windows of up to 4096 tokens, counters, statistics and per-token spreads beyond) exceeds
 *     LRSA_STATIC_SCRATCH_BYTES are refused with LRSA_ERR_WORKSPACE_TOO_SMALL and nothing is
 *     enqueued; use lrsa_score_select with a workspace for those.
 *   - The device that owns `cuda_stream` must be the current device.  The first call on each device
 *     looks up the array's device address (once per device); make that first call outside of any
 *     stream capture.
 *   - All calls on a device share the one array.  It keeps the previous call's contents; the
 *     call clears, on the stream, the parts that must start at zero.  Two calls whose kernels could
 *     overlap on the GPU (different streams without ordering) race on it and give undefined
 *     results: serialise them.
 */
#define LRSA_STATIC_SCRATCH_BYTES (4u << 20)
int lrsa_score_select_static(const lrsa_params_t* params, const void* K, const void* V, int32_t* idx,
                             float* score, void* cuda_stream);

/*
 * What lrsa_workspace_status is for the calls that take a workspace: reads the status word that the last
 * lrsa_score_select_static call on the current device left in the library's fixed array (the caller has
 * no pointer to it).  Synchronises `cuda_stream`, allocates nothing.  Returns LRSA_OK, LRSA_ERR_TIMEOUT
 * (a bounded device-side wait expired: idx and score are undefined), or LRSA_ERR_CUDA.
 */
int lrsa_score_select_static_status(void* cuda_stream);

/*
 * LRSA attention forward (Section 3.1, Eq. 3 with the chunked mask of Section 3.2).
 * Query position t < S attends positions [0, t].  Query t >= S in chunk c = (t-S)/L attends the
 * sinks, the kept positions idx[b, hkv, w, :] of the first n_c = min(max(c - n_dense_prev, 0),
 * W_sel) windows, and every position of [S + n_c*L, t].  bf16 tensor-core products, fp32
 * accumulation and softmax.
 *
 *   Q       in  : bf16 [B, Hq, N, d];  K, V in : bf16 [B, Hkv, N, d]
 *   idx     in  : int32 [B, Hkv, W_sel, top_k]; any set of distinct in-window positions listed
 *                 ascending per window (normally the output of lrsa_score_select)
 *   O       out : bf16 [B, Hq, N, d]
 *   LSE     out : fp32 [B, Hq, N], natural-log sum of exponentials of the scaled scores
 */
int lrsa_attn_fwd(const lrsa_params_t* params, const void* Q, const void* K, const void* V,
                  const int32_t* idx, void* O, float* LSE, void* workspace, size_t workspace_bytes,
                  void* cuda_stream);

/*
 * LRSA attention backward: gradient of Eq. 3 with respect to Q, K, V for upstream gradient dO,
 * the mask (idx) held constant.  P = exp(scale*QK^T - LSE) is recomputed; D = rowsum(dO * O);
 * dV = P^T dO; dS = P * (dO V^T - D); dQ = scale * dS K; dK = scale * dS^T Q, summed over the
 * query heads of each KV group; contributions through kept positions land on their original
 * token positions.  dQ, dK, dV are fully overwritten.
 *
 *   O, LSE in : outputs of lrsa_attn_fwd for the same inputs
 *   dO     in : bf16 [B, Hq, N, d]
 *   dQ    out : bf16 [B, Hq, N, d];  dK, dV out : bf16 [B, Hkv, N, d]
 */
int lrsa_attn_bwd(const lrsa_params_t* params, const void* Q, const void* K, const void* V,
                  const void* O, const void* dO, const float* LSE, const int32_t* idx, void* dQ,
                  void* dK, void* dV, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Inference side (Section 3.2: the KV-cache update of Attn-Fill 1 / Attn-Fill 2; its last paragraph: the mask
 * does not depend on the query, so the KV cache can be condensed physically).  The cache is one caller-owned
 * device buffer of lrsa_cache_bytes bytes per layer (256-byte aligned, contents managed by these calls).  Per
 * (batch, KV head) it holds the sink rows, top_k kept rows of every compressed window, and a ring of 2*lag rows
 * with the uncompressed recent tokens: S + W*K + 2L rows instead of seq_len.  seq_len is the capacity in tokens.
 * Only n_dense_prev = 1 and unpacked batches are supported (LRSA_ERR_UNSUPPORTED otherwise).
 *
 * lrsa_cache_append adds the tokens n_prev .. n_prev + n_new - 1 (n_prev = tokens already in the cache; the caller
 * keeps that count; the first call has n_prev = 0).  When the first token of query chunk c arrives, window c-2 is
 * scored with window c-1 as its reference (Eq. 4-8, the arithmetic of lrsa_score_select), its top_k rows are
 * appended to the kept rows and it leaves the ring; until then the queries of chunk c-1 see it whole, as the
 * mask of Section 3.2 prescribes.  Any n_new is accepted.
 *   k_new, v_new in : bf16 [B, Hkv, n_new, d]
 *
 * lrsa_attn_decode: Eq. 3 for ONE query token per (batch, query head), the token at position n_tokens - 1 of a
 * cache that holds n_tokens tokens; it sees exactly what row n_tokens - 1 of lrsa_attn_fwd sees.  bf16 tensor-core products,
 * fp32 accumulation and softmax, as in lrsa_attn_fwd.
 *   q in : bf16 [B, Hq, d];  o out : bf16 [B, Hq, d];  lse out (optional) : fp32 [B, Hq]
 *
 * lrsa_cache_kept returns a device pointer into the cache: int32 [B, Hkv, w_cap, top_k], the kept positions of the
 * windows compressed so far (rows of later windows are undefined).
 * `workspace` (lrsa_cache_bytes' second figure) is scratch for both calls; its status word is read with
 * lrsa_workspace_status.
 */
int lrsa_cache_bytes(const lrsa_params_t* params, size_t* cache_bytes, size_t* workspace_bytes);
int lrsa_cache_append(const lrsa_params_t* params, void* cache, size_t cache_bytes, const void* k_new,
                      const void* v_new, int32_t n_prev, int32_t n_new, void* workspace, size_t workspace_bytes,
                      void* cuda_stream);
int lrsa_cache_kept(const lrsa_params_t* params, const void* cache, const int32_t** idx, int32_t* w_cap);
int lrsa_attn_decode(const lrsa_params_t* params, const void* cache, size_t cache_bytes, const void* q,
                     int32_t n_tokens, void* o, float* lse, void* workspace, size_t workspace_bytes,
                     void* cuda_stream);

/*
 * Reads the status word that the last call using `workspace` left there.  Synchronises
 * `cuda_stream`.  Returns LRSA_OK, LRSA_ERR_TIMEOUT, or LRSA_ERR_CUDA if the copy failed.
 */
int lrsa_workspace_status(const void* workspace, void* cuda_stream);

/* Static, human-readable name of a status value. */
const char* lrsa_status_string(int status);

/* Number of kernels (and memset nodes) the last call on this host thread enqueued. */
int lrsa_last_launch_count(void);

/*
 * Validation switch (process-wide): 0 selects the tensor-core attention kernels (default),
 * 1 the slow CUDA-core kernels kept for cross-checking on the GPU.  Both compute the same
 * function from the same arguments and workspace.
 */
int lrsa_debug_set_impl(int impl);

/*
 * Test hook (process-wide) for the bounded device-side wait of the scoring kernel that handles lag windows
 * beyond 4096 tokens: the number of polls a work unit grants the statistics of the following window.  A
 * negative value makes that wait give up at once, so that the LRSA_ERR_TIMEOUT path can be exercised without
 * wedging a kernel (the call then leaves idx undefined and the status word set); 0 restores the default.
 */
int lrsa_debug_set_wait_limit(int polls);

#ifdef __cplusplus
}
#endif
#endif /* LRSA_H_ */
