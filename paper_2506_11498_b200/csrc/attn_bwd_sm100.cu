// LRSA attention backward: workspace layout and the sequence of launches.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

struct BwdWs {
  size_t kbar, dacc, zero_end, kc, vc, stats, dkv, total;
};
BwdWs bwd_ws_layout(const Geom& g) {
  BwdWs w;
  const size_t rc = g.Rc > 0 ? g.Rc : 1;
  const size_t cbytes = align_up((size_t)g.B * g.Hkv * rc * g.d * sizeof(__nv_bfloat16), 1024);
  size_t off = 1024;
  // cleared together with the header: the mean-key accumulator and the per-row D accumulator
  w.kbar = off; off += align_up((size_t)g.B * g.Hkv * g.d * sizeof(float), 1024);
  w.dacc = off; off += align_up((size_t)g.B * g.Hq * g.N * sizeof(float), 1024);
  w.zero_end = off;
  w.kc = off; off += cbytes;   // compact K/V for the query-outer dQ kernel
  w.vc = off; off += cbytes;
  w.stats = off; off += align_up((size_t)g.B * g.Hq * g.N * sizeof(float2), 1024);
  w.dkv = off; off += dkv_ws_bytes(g, nullptr);
  w.total = off;
  return w;
}

}  // namespace

size_t attn_bwd_ws_bytes(const Geom& g) { return bwd_ws_layout(g).total; }

int launch_attn_bwd_sm100(const lrsa_params_t* params, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                          const __nv_bfloat16* V, const __nv_bfloat16* O, const __nv_bfloat16* dO,
                          const float* LSE, const int32_t* idx, __nv_bfloat16* dQ, __nv_bfloat16* dK,
                          __nv_bfloat16* dV, void* ws, cudaStream_t st) {
  const BwdWs lay = bwd_ws_layout(g);
  unsigned char* base = static_cast<unsigned char*>(ws);
  LRSA_CUDA_CHECK(cudaMemsetAsync(base, 0, lay.zero_end, st));
  launch_counter().n++;
  __nv_bfloat16* Kc = reinterpret_cast<__nv_bfloat16*>(base + lay.kc);
  __nv_bfloat16* Vc = reinterpret_cast<__nv_bfloat16*>(base + lay.vc);
  float2* stats = reinterpret_cast<float2*>(base + lay.stats);
  float* kbar = reinterpret_cast<float*>(base + lay.kbar);
  float* Dacc = reinterpret_cast<float*>(base + lay.dacc);
  int* status = &reinterpret_cast<WsHeader*>(base)->status;
  // Per-row statistics and the mean key are taken over whole rows (the mean key is only a centring
  // vector: any constant works).  Then, sequence after sequence, the dK/dV kernel (which also produces
  // the accurate D of the sequence's rows) and the dQ kernel; bf16 dK, dV at the end.
  const __nv_bfloat16* Olo = static_cast<const __nv_bfloat16*>(params->o_residual);
  int rc = launch_bwd_prep(g, O, Olo, dO, LSE, K, stats, kbar, st);
  if (rc == LRSA_OK) rc = dkv_zero(g, base + lay.dkv, st);
  const int n_seqs = geom_n_seqs(params);
  int woff = 0;
  for (int s = 0; s < n_seqs && rc == LRSA_OK; ++s) {
    Geom gs;
    seq_geom(g, params->cu_seqlens, params->n_seqs, s, woff, &gs);
    woff += gs.Wsel;
    rc = launch_bwd_dkv_sm100(g, gs, Q, dO, K, V, stats, Dacc, idx, base + lay.dkv, status, st);
    if (rc == LRSA_OK) rc = launch_compact_kv(gs, K, V, idx, Kc, Vc, st);
    if (rc == LRSA_OK) rc = launch_bwd_dq_sm100(gs, Q, dO, K, V, Kc, Vc, stats, Dacc, kbar, dQ, status, st);
  }
  if (rc == LRSA_OK) rc = dkv_convert(g, base + lay.dkv, dK, dV, st);
  return rc;
}

}  // namespace lrsa
