// C ABI entry points: argument validation on the host, workspace layout, kernel dispatch.
#include <math.h>

#include "lrsa_internal.h"

namespace lrsa {

LaunchCounter& launch_counter() {
  static thread_local LaunchCounter c;
  return c;
}

static int g_impl = 0;  // 0: tensor-core kernels, 1: CUDA-core validation kernels

int make_geom(const lrsa_params_t* p, Geom* g) {
  if (!p || !g) return LRSA_ERR_INVALID_ARG;
  if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->seq_len < 1 || p->head_dim < 1 ||
      p->lag < 1 || p->chunk < 1 || p->top_k < 1 || p->n_sink < 0)
    return LRSA_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return LRSA_ERR_INVALID_ARG;
  if (p->top_k > p->lag) return LRSA_ERR_INVALID_ARG;
  if (p->std_ddof != 0 && p->std_ddof != 1) return LRSA_ERR_INVALID_ARG;
  if (p->n_dense_prev != 0 && p->n_dense_prev != 1) return LRSA_ERR_INVALID_ARG;
  if (!(p->softmax_scale >= 0.f) || isinf(p->softmax_scale)) return LRSA_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return LRSA_ERR_UNSUPPORTED;
  // A query chunk of m lag windows sees exactly what m chunks of one window see (the mask of Section
  // 3.2 does not depend on how many chunks are filled at a time), so any multiple of the lag is accepted.
  if (p->chunk % p->lag != 0) return LRSA_ERR_UNSUPPORTED;
  if (p->seq_len < p->n_sink) return LRSA_ERR_UNSUPPORTED;
  if (p->lag > 32767) return LRSA_ERR_UNSUPPORTED;  // packed 16-bit counters in the selection scan
  if ((long long)p->batch * p->n_q_heads * p->seq_len > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  g->B = p->batch; g->Hq = p->n_q_heads; g->Hkv = p->n_kv_heads; g->G = g->Hq / g->Hkv;
  g->N = p->seq_len; g->d = p->head_dim; g->L = p->lag; g->K = p->top_k; g->S = p->n_sink;
  g->ndp = p->n_dense_prev; g->ddof = p->std_ddof;
  g->scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  g->W = (g->N - g->S) / g->L;
  g->T = g->N - g->S - g->W * g->L;
  g->C = g->W + (g->T > 0 ? 1 : 0);
  g->Wsel = g->W > 1 ? g->W - 1 : 0;
  g->Rc = g->S + g->Wsel * g->K;
  g->Nrow = g->N; g->tok0 = 0; g->Wtot = g->Wsel; g->woff = 0; g->emit_off = 0; g->win_stride = g->L;
  if (reinterpret_cast<uintptr_t>(p->o_residual) & 15u) return LRSA_ERR_INVALID_ARG;
  g->has_o_res = p->o_residual != nullptr;
  if (p->n_seqs < 0) return LRSA_ERR_INVALID_ARG;
  if (p->n_seqs > 0) {
    if (!p->cu_seqlens || p->cu_seqlens[0] != 0 || p->cu_seqlens[p->n_seqs] != p->seq_len) return LRSA_ERR_INVALID_ARG;
    int wtot = 0;
    for (int s = 0; s < p->n_seqs; ++s) {
      const int n = p->cu_seqlens[s + 1] - p->cu_seqlens[s];
      if (n < 1) return LRSA_ERR_INVALID_ARG;
      const int w = n > g->S ? (n - g->S) / g->L : 0;
      wtot += w > 1 ? w - 1 : 0;
    }
    g->Wtot = wtot;
  }
  return LRSA_OK;
}

int geom_n_seqs(const lrsa_params_t* p) { return p->n_seqs > 0 ? p->n_seqs : 1; }

void seq_geom(const Geom& whole, const int32_t* cu, int n_seqs, int s, int woff, Geom* out) {
  *out = whole;
  if (n_seqs <= 0 || !cu) return;   // the whole row is the one sequence
  Geom& g = *out;
  g.tok0 = cu[s];
  g.emit_off = cu[s];
  g.N = cu[s + 1] - cu[s];
  g.S = whole.S < g.N ? whole.S : g.N;   // a sequence shorter than the sink count is all sinks
  g.W = (g.N - g.S) / g.L;
  g.T = g.N - g.S - g.W * g.L;
  g.C = g.W + (g.T > 0 ? 1 : 0);
  g.Wsel = g.W > 1 ? g.W - 1 : 0;
  g.Rc = g.S + g.Wsel * g.K;
  g.woff = woff;
}

int run_score_select(const lrsa_params_t* p, const Geom& whole, const __nv_bfloat16* K, const __nv_bfloat16* V,
                     int32_t* idx, float* score, void* ws, cudaStream_t st) {
  const int n_seqs = geom_n_seqs(p);
  // one sequence scored by the kernel that clears the status word itself: a single launch
  const bool in_kernel = n_seqs == 1 && score_select_clears_status(whole);
  if (!in_kernel) {
    LRSA_CUDA_CHECK(cudaMemsetAsync(ws, 0, sizeof(WsHeader), st));
    launch_counter().n++;
  }
  int woff = 0;
  for (int s = 0; s < n_seqs; ++s) {
    Geom g;
    seq_geom(whole, p->cu_seqlens, p->n_seqs, s, woff, &g);
    const int rc = launch_score_select(g, K, V, idx, score, ws, st, in_kernel);
    if (rc != LRSA_OK) return rc;
    woff += g.Wsel;
  }
  return LRSA_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static size_t fwd_ws_bytes(const Geom& g) {
  const size_t a = attn_ref_fwd_ws_bytes(g), b = attn_fwd_ws_bytes(g);
  return a > b ? a : b;
}
static size_t bwd_ws_bytes(const Geom& g) {
  const size_t a = attn_ref_bwd_ws_bytes(g), b = attn_bwd_ws_bytes(g);
  return a > b ? a : b;
}

}  // namespace lrsa

using namespace lrsa;

extern "C" {

int lrsa_num_sel_windows(const lrsa_params_t* params, int32_t* w_sel) {
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!w_sel) return LRSA_ERR_INVALID_ARG;
  *w_sel = g.Wtot;
  return LRSA_OK;
}

int lrsa_workspace_bytes(const lrsa_params_t* params, size_t* score_select, size_t* attn_fwd,
                         size_t* attn_bwd) {
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (score_select) *score_select = score_select_ws_bytes(g);
  if (attn_fwd) *attn_fwd = fwd_ws_bytes(g);
  if (attn_bwd) *attn_bwd = bwd_ws_bytes(g);
  return LRSA_OK;
}

int lrsa_score_select(const lrsa_params_t* params, const void* K, const void* V, int32_t* idx,
                      float* score, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  NvtxRange nvtx_range("lrsa_score_select");
  launch_counter().n = 0;
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!K || !V || !workspace) return LRSA_ERR_INVALID_ARG;
  if (g.Wtot > 0 && !idx) return LRSA_ERR_INVALID_ARG;
  if (!aligned(K, 16) || !aligned(V, 16) || !aligned(idx, 4) || !aligned(score, 4) || !aligned(workspace, 256))
    return LRSA_ERR_INVALID_ARG;
  if (workspace_bytes < score_select_ws_bytes(g)) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  return run_score_select(params, g, static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V),
                          idx, score, workspace, static_cast<cudaStream_t>(cuda_stream));
}

int lrsa_attn_fwd(const lrsa_params_t* params, const void* Q, const void* K, const void* V,
                  const int32_t* idx, void* O, float* LSE, void* workspace, size_t workspace_bytes,
                  void* cuda_stream) {
  NvtxRange nvtx_range("lrsa_attn_fwd");
  launch_counter().n = 0;
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!Q || !K || !V || !O || !LSE || !workspace) return LRSA_ERR_INVALID_ARG;
  if (g.Wtot > 0 && !idx) return LRSA_ERR_INVALID_ARG;
  if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(LSE, 16) ||
      !aligned(idx, 4) || !aligned(workspace, 256))
    return LRSA_ERR_INVALID_ARG;
  if (workspace_bytes < fwd_ws_bytes(g)) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  auto st = static_cast<cudaStream_t>(cuda_stream);
  auto bf = [](const void* p) { return static_cast<const __nv_bfloat16*>(p); };
  if (g_impl == 0) return launch_attn_fwd_sm100(params, g, bf(Q), bf(K), bf(V), idx, static_cast<__nv_bfloat16*>(O), LSE, workspace, st);
  if (params->n_seqs > 0) return LRSA_ERR_UNSUPPORTED;   // the validation kernels take one sequence per row
  return launch_attn_ref_fwd(g, bf(Q), bf(K), bf(V), idx, static_cast<__nv_bfloat16*>(O), LSE, workspace, st);
}

int lrsa_attn_bwd(const lrsa_params_t* params, const void* Q, const void* K, const void* V,
                  const void* O, const void* dO, const float* LSE, const int32_t* idx, void* dQ,
                  void* dK, void* dV, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  NvtxRange nvtx_range("lrsa_attn_bwd");
  launch_counter().n = 0;
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!Q || !K || !V || !O || !dO || !LSE || !dQ || !dK || !dV || !workspace) return LRSA_ERR_INVALID_ARG;
  if (g.Wtot > 0 && !idx) return LRSA_ERR_INVALID_ARG;
  const void* ptrs[] = {Q, K, V, O, dO, LSE, dQ, dK, dV};
  for (const void* p : ptrs)
    if (!aligned(p, 16)) return LRSA_ERR_INVALID_ARG;
  if (!aligned(idx, 4) || !aligned(workspace, 256)) return LRSA_ERR_INVALID_ARG;
  if (workspace_bytes < bwd_ws_bytes(g)) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  auto st = static_cast<cudaStream_t>(cuda_stream);
  auto bf = [](const void* p) { return static_cast<const __nv_bfloat16*>(p); };
  if (g_impl == 0)
    return launch_attn_bwd_sm100(params, g, bf(Q), bf(K), bf(V), bf(O), bf(dO), LSE, idx, static_cast<__nv_bfloat16*>(dQ),
                                 static_cast<__nv_bfloat16*>(dK), static_cast<__nv_bfloat16*>(dV), workspace, st);
  if (params->n_seqs > 0) return LRSA_ERR_UNSUPPORTED;   // the validation kernels take one sequence per row
  return launch_attn_ref_bwd(g, bf(Q), bf(K), bf(V), bf(O), bf(dO), LSE, idx, static_cast<__nv_bfloat16*>(dQ),
                             static_cast<__nv_bfloat16*>(dK), static_cast<__nv_bfloat16*>(dV), workspace, st);
}

int lrsa_workspace_status(const void* workspace, void* cuda_stream) {
  if (!workspace) return LRSA_ERR_INVALID_ARG;
  int status = 0;
  auto st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return LRSA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LRSA_ERR_CUDA;
  return status == 0 ? LRSA_OK : LRSA_ERR_TIMEOUT;
}

const char* lrsa_status_string(int status) {
  switch (status) {
    case LRSA_OK: return "ok";
    case LRSA_ERR_INVALID_ARG: return "invalid argument";
    case LRSA_ERR_UNSUPPORTED: return "unsupported configuration";
    case LRSA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LRSA_ERR_CUDA: return "CUDA runtime error";
    case LRSA_ERR_TIMEOUT: return "bounded device-side wait expired";
    default: return "unknown status";
  }
}

int lrsa_last_launch_count(void) { return launch_counter().n; }

int lrsa_debug_set_wait_limit(int polls) {
  set_unit_wait_limit(polls == 0 ? (1 << 21) : polls);
  return LRSA_OK;
}

int lrsa_debug_set_impl(int impl) {
  if (impl != 0 && impl != 1) return LRSA_ERR_INVALID_ARG;
  g_impl = impl;
  return LRSA_OK;
}

}  // extern "C"
