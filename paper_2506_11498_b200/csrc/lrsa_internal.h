// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <nvtx3/nvToolsExt.h>

#include "../../include/lrsa.h"

namespace lrsa {

// Problem geometry derived from lrsa_params_t (Section 3.2: sink of size S, windows of lag L).
struct Geom {
  int B, Hq, Hkv, G, N, d, L, K, S, ndp, ddof;
  float scale;
  int W;     // full windows
  int T;     // tail tokens
  int C;     // query chunks = W + [T > 0]
  int Wsel;  // scored windows = max(W - 1, 0)
  int Rc;    // rows of the compact (sinks + kept) K/V buffer per KV head = S + Wsel*K
  // Packed batches: this Geom describes ONE sequence of N tokens that starts at token `tok0` of rows
  // that hold Nrow tokens per (batch, head); its scored windows are windows [woff, woff + Wsel) of the
  // Wtot windows of the whole row.  Single sequence: Nrow = N, tok0 = 0, Wtot = Wsel, woff = 0.
  // The launchers shift every tensor pointer by tok0 tokens and use Nrow as the row stride, so the
  // kernels see an ordinary sequence; kept positions (idx) stay positions in the whole row.
  int Nrow, tok0, Wtot, woff;
  // Scoring only: value added to the positions written to idx (tok0 unless the rows are a ring buffer)
  // and distance in tokens from window w to window w+1 (L unless the rows are a ring buffer).
  int emit_off, win_stride;
  int has_o_res;   // the caller gave a buffer for the rounding remainder of O (lrsa_params_t::o_residual)
};

// Sequence s of a packed batch (cu = boundaries, n_seqs + 1 entries) as a Geom of its own.
void seq_geom(const Geom& whole, const int32_t* cu, int n_seqs, int s, int woff, Geom* out);
// Number of sequences and boundaries of `p` (a single sequence when it has no cu_seqlens).
int geom_n_seqs(const lrsa_params_t* p);

// Validates `p` and fills `g`. Returns an lrsa_status.
int make_geom(const lrsa_params_t* p, Geom* g);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace header (first 256 bytes of every workspace).
struct WsHeader {
  int status;   // lrsa_status written by kernels (0 or LRSA_ERR_TIMEOUT)
  int ticket;   // dynamic work counter of the scoring kernel
  int pad[62];
};
static_assert(sizeof(WsHeader) == 256, "header is 256 bytes");

// Number of leading windows that query chunk c sees only through their kept tokens.
__host__ __device__ inline int n_hist_windows(int c, int ndp, int Wsel) {
  int n = c - ndp;
  if (n < 0) n = 0;
  return n < Wsel ? n : Wsel;
}

// First chunk that sees window w compressed (C if none): smallest c with n_hist_windows(c) > w.
__host__ __device__ inline int first_compressed_chunk(int w, int ndp, int Wsel, int C) {
  if (w >= Wsel) return C;
  int c = w + 1 + ndp;
  return c < C ? c : C;
}

// NVTX range around an entry point (visible in a timeline profiler; free when no tool is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

struct LaunchCounter {
  int n = 0;
};
LaunchCounter& launch_counter();

// lrsa_api.cu : clears the status header of `ws`, then scores and selects sequence after sequence.
int run_score_select(const lrsa_params_t* p, const Geom& whole, const __nv_bfloat16* K, const __nv_bfloat16* V,
                     int32_t* idx, float* score, void* ws, cudaStream_t st);

// score_select.cu (one sequence; the status header of `ws` is cleared by the caller)
size_t score_select_ws_bytes(const Geom& g);
int launch_score_select(const Geom& g, const __nv_bfloat16* K, const __nv_bfloat16* V, int32_t* idx,
                        float* score, void* ws, cudaStream_t st, bool clear_status = false);
// True when the kernel that scores `g` can clear the status word itself (clear_status above).
bool score_select_clears_status(const Geom& g);
void set_unit_wait_limit(int polls);

// attn_ref.cu : CUDA-core reference kernels (one warp per row), used for validation.
size_t attn_ref_fwd_ws_bytes(const Geom& g);
size_t attn_ref_bwd_ws_bytes(const Geom& g);
int launch_attn_ref_fwd(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const int32_t* idx, __nv_bfloat16* O, float* LSE,
                        void* ws, cudaStream_t st);
int launch_attn_ref_bwd(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const __nv_bfloat16* O, const __nv_bfloat16* dO,
                        const float* LSE, const int32_t* idx, __nv_bfloat16* dQ, __nv_bfloat16* dK,
                        __nv_bfloat16* dV, void* ws, cudaStream_t st);

// attn_fwd_sm100.cu : tcgen05 / TMEM forward (workspace: header + compact K/V).
size_t attn_fwd_ws_bytes(const Geom& g);
int launch_attn_fwd_sm100(const lrsa_params_t* params, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                          const __nv_bfloat16* V, const int32_t* idx, __nv_bfloat16* O, float* LSE,
                          void* ws, cudaStream_t st);

int launch_attn_ref_bwd_dkv(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                            const __nv_bfloat16* V, const __nv_bfloat16* dO, const float* LSE,
                            const int32_t* idx, const float* Dsum, __nv_bfloat16* dK, __nv_bfloat16* dV,
                            cudaStream_t st);

// attn_bwd_*_sm100.cu : tcgen05 / TMEM backward.
size_t attn_bwd_ws_bytes(const Geom& g);
int launch_attn_bwd_sm100(const lrsa_params_t* params, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                          const __nv_bfloat16* V, const __nv_bfloat16* O, const __nv_bfloat16* dO,
                          const float* LSE, const int32_t* idx, __nv_bfloat16* dQ, __nv_bfloat16* dK,
                          __nv_bfloat16* dV, void* ws, cudaStream_t st);
// Backward helpers.  stats[row] = (-LSE * log2(e), rowsum(dO * O)) per query row; kbar[b*Hkv+h][c] is the
// mean key (accumulated into a zeroed array).  The dK/dV kernel runs first and adds sum_j P dP, the
// accurate D of every query row, into the zeroed Dacc; the dQ kernel reads it.
int launch_bwd_prep(const Geom& g, const __nv_bfloat16* O, const __nv_bfloat16* Olo, const __nv_bfloat16* dO,
                    const float* LSE, const __nv_bfloat16* K, float2* stats, float* kbar, cudaStream_t st);
int launch_bwd_dq_sm100(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, const float2* stats,
                        const float* Dacc, const float* kbar, __nv_bfloat16* dQ, int* status, cudaStream_t st);

size_t dkv_ws_bytes(const Geom& g, size_t* prefix_bytes);
int dkv_zero(const Geom& whole, void* ws_dkv, cudaStream_t st);
int launch_bwd_dkv_sm100(const Geom& whole, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO,
                         const __nv_bfloat16* K, const __nv_bfloat16* V, const float2* stats, float* Dacc,
                         const int32_t* idx, void* ws_dkv, int* status, cudaStream_t st);
int dkv_convert(const Geom& whole, void* ws_dkv, __nv_bfloat16* dK, __nv_bfloat16* dV, cudaStream_t st);

#define LRSA_CUDA_CHECK(expr)                                 \
  do {                                                        \
    cudaError_t _e = (expr);                                  \
    if (_e != cudaSuccess) return (int)LRSA_ERR_CUDA;         \
  } while (0)

}  // namespace lrsa
