// CUDA-core validation kernels for LRSA attention (Section 3.1 Eq. 3 under the chunked mask of
// Section 3.2): one warp per query row (forward, dQ) or per key row (dK, dV), fp32 throughout,
// reading the kept positions straight from idx.  Slow by design; they exist so that the
// tensor-core kernels can be compared on the GPU at sizes the CPU checker cannot reach, and are
// selected only through the library's validation switch.
#include "lrsa_internal.h"

namespace lrsa {
namespace {

struct RefArgs {
  const __nv_bfloat16 *Q, *K, *V, *O, *dO;
  const float* LSE;
  const int32_t* idx;
  __nv_bfloat16 *Oout, *dQ, *dK, *dV;
  float* LSEout;
  float* Dws;  // [B,Hq,N]
  int B, Hq, Hkv, G, N, L, Kk, S, ndp, W, C, Wsel;
  float scale;
};

__device__ __forceinline__ float wsum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D>
__device__ __forceinline__ void load_row(const __nv_bfloat16* p, int lane, float (&r)[D / 32]) {
#pragma unroll
  for (int i = 0; i < D / 32; ++i) r[i] = __bfloat162float(p[lane * (D / 32) + i]);
}
template <int D>
__device__ __forceinline__ float dot(const float (&a)[D / 32], const float (&b)[D / 32]) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < D / 32; ++i) s = fmaf(a[i], b[i], s);
  return wsum(s);
}

// The keys query t sees, as a list: sinks, kept positions of the compressed windows, then the
// contiguous range that ends at t.
struct KeyList {
  int n_front;      // sinks + kept entries
  int dense_start;  // first position of the contiguous range
  int n;            // total
  const int32_t* kept;
  int S;
  __device__ int pos(int i) const {
    if (i < S) return i;
    if (i < n_front) return kept[i - S];
    return dense_start + (i - n_front);
  }
};
__device__ __forceinline__ KeyList key_list(const RefArgs& a, int b, int hkv, int t) {
  KeyList kl;
  kl.S = a.S;
  kl.kept = a.idx + (size_t)(b * a.Hkv + hkv) * a.Wsel * a.Kk;
  if (t < a.S) {
    kl.S = 0; kl.n_front = 0; kl.dense_start = 0; kl.n = t + 1;
  } else {
    const int c = (t - a.S) / a.L;
    const int nh = n_hist_windows(c, a.ndp, a.Wsel);
    kl.n_front = a.S + nh * a.Kk;
    kl.dense_start = a.S + nh * a.L;
    kl.n = kl.n_front + (t - kl.dense_start + 1);
  }
  return kl;
}

template <int D>
__global__ void __launch_bounds__(256) ref_fwd_kernel(const RefArgs a) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= (long long)a.B * a.Hq * a.N) return;
  const int t = (int)(row % a.N), hq = (int)((row / a.N) % a.Hq), b = (int)(row / ((long long)a.N * a.Hq));
  const int hkv = hq / a.G;
  float q[D / 32], o[D / 32], x[D / 32];
  load_row<D>(a.Q + (size_t)row * D, lane, q);
#pragma unroll
  for (int i = 0; i < D / 32; ++i) o[i] = 0.f;
  const KeyList kl = key_list(a, b, hkv, t);
  const size_t kvbase = (size_t)(b * a.Hkv + hkv) * a.N;
  float m = -INFINITY, l = 0.f;
  for (int i = 0; i < kl.n; ++i) {
    const size_t j = kvbase + kl.pos(i);
    load_row<D>(a.K + j * D, lane, x);
    const float s = dot<D>(q, x) * a.scale;
    const float mn = fmaxf(m, s);
    const float corr = expf(m - mn), p = expf(s - mn);
    l = l * corr + p;
    load_row<D>(a.V + j * D, lane, x);
#pragma unroll
    for (int c = 0; c < D / 32; ++c) o[c] = o[c] * corr + p * x[c];
    m = mn;
  }
#pragma unroll
  for (int c = 0; c < D / 32; ++c) a.Oout[(size_t)row * D + lane * (D / 32) + c] = __float2bfloat16(o[c] / l);
  if (lane == 0) a.LSEout[row] = m + logf(l);
}

template <int D>
__global__ void __launch_bounds__(256) ref_bwd_dq_kernel(const RefArgs a) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= (long long)a.B * a.Hq * a.N) return;
  const int t = (int)(row % a.N), hq = (int)((row / a.N) % a.Hq), b = (int)(row / ((long long)a.N * a.Hq));
  const int hkv = hq / a.G;
  float q[D / 32], go[D / 32], x[D / 32], acc[D / 32];
  load_row<D>(a.Q + (size_t)row * D, lane, q);
  load_row<D>(a.dO + (size_t)row * D, lane, go);
  load_row<D>(a.O + (size_t)row * D, lane, x);
  const float Dt = dot<D>(go, x);
  if (lane == 0) a.Dws[row] = Dt;
  const float lse = a.LSE[row];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) acc[i] = 0.f;
  const KeyList kl = key_list(a, b, hkv, t);
  const size_t kvbase = (size_t)(b * a.Hkv + hkv) * a.N;
  for (int i = 0; i < kl.n; ++i) {
    const size_t j = kvbase + kl.pos(i);
    load_row<D>(a.V + j * D, lane, x);
    const float dp = dot<D>(go, x);
    load_row<D>(a.K + j * D, lane, x);
    const float p = expf(dot<D>(q, x) * a.scale - lse);
    const float ds = p * (dp - Dt);
#pragma unroll
    for (int c = 0; c < D / 32; ++c) acc[c] = fmaf(ds, x[c], acc[c]);
  }
#pragma unroll
  for (int c = 0; c < D / 32; ++c) a.dQ[(size_t)row * D + lane * (D / 32) + c] = __float2bfloat16(acc[c] * a.scale);
}

template <int D>
__global__ void __launch_bounds__(256) ref_bwd_dkv_kernel(const RefArgs a) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= (long long)a.B * a.Hkv * a.N) return;
  const int j = (int)(row % a.N), hkv = (int)((row / a.N) % a.Hkv), b = (int)(row / ((long long)a.N * a.Hkv));
  float k[D / 32], v[D / 32], q[D / 32], go[D / 32], dk[D / 32], dv[D / 32];
  load_row<D>(a.K + (size_t)row * D, lane, k);
  load_row<D>(a.V + (size_t)row * D, lane, v);
#pragma unroll
  for (int i = 0; i < D / 32; ++i) dk[i] = dv[i] = 0.f;
  // queries that see key j: [j, tsplit) uncompressed, then [tsplit, N) only if j is kept
  int tend = a.N;
  if (j >= a.S) {
    const int w = (j - a.S) / a.L;
    const int cc = first_compressed_chunk(w, a.ndp, a.Wsel, a.C);
    const int tsplit = cc >= a.C ? a.N : min(a.N, a.S + cc * a.L);
    bool kept = false;
    if (w < a.Wsel) {
      const int32_t* ix = a.idx + ((size_t)(b * a.Hkv + hkv) * a.Wsel + w) * a.Kk;
      int lo = 0, hi = a.Kk - 1;
      while (lo <= hi) {
        const int mid = (lo + hi) >> 1, val = ix[mid];
        if (val == j) { kept = true; break; }
        if (val < j) lo = mid + 1; else hi = mid - 1;
      }
    }
    if (!kept) tend = tsplit;
  }
  for (int g = 0; g < a.G; ++g) {
    const size_t qbase = (size_t)(b * a.Hq + hkv * a.G + g) * a.N;
    for (int t = j; t < tend; ++t) {
      load_row<D>(a.Q + (qbase + t) * D, lane, q);
      load_row<D>(a.dO + (qbase + t) * D, lane, go);
      const float p = expf(dot<D>(q, k) * a.scale - a.LSE[qbase + t]);
      const float ds = p * (dot<D>(go, v) - a.Dws[qbase + t]);
#pragma unroll
      for (int c = 0; c < D / 32; ++c) { dv[c] = fmaf(p, go[c], dv[c]); dk[c] = fmaf(ds, q[c], dk[c]); }
    }
  }
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
    a.dK[(size_t)row * D + lane * (D / 32) + c] = __float2bfloat16(dk[c] * a.scale);
    a.dV[(size_t)row * D + lane * (D / 32) + c] = __float2bfloat16(dv[c]);
  }
}

RefArgs make_args(const Geom& g) {
  RefArgs a{};
  a.B = g.B; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.N; a.L = g.L; a.Kk = g.K; a.S = g.S;
  a.ndp = g.ndp; a.W = g.W; a.C = g.C; a.Wsel = g.Wsel; a.scale = g.scale;
  return a;
}

}  // namespace

size_t attn_ref_fwd_ws_bytes(const Geom&) { return sizeof(WsHeader); }
size_t attn_ref_bwd_ws_bytes(const Geom& g) {
  return sizeof(WsHeader) + align_up((size_t)g.B * g.Hq * g.N * sizeof(float), 256);
}

int launch_attn_ref_fwd(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const int32_t* idx, __nv_bfloat16* O, float* LSE,
                        void* ws, cudaStream_t st) {
  LRSA_CUDA_CHECK(cudaMemsetAsync(ws, 0, sizeof(WsHeader), st));
  launch_counter().n++;
  RefArgs a = make_args(g);
  a.Q = Q; a.K = K; a.V = V; a.idx = idx; a.Oout = O; a.LSEout = LSE;
  const long long rows = (long long)g.B * g.Hq * g.N;
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  if (g.d == 128) ref_fwd_kernel<128><<<blocks, 256, 0, st>>>(a);
  else ref_fwd_kernel<64><<<blocks, 256, 0, st>>>(a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

int launch_attn_ref_bwd(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const __nv_bfloat16* O, const __nv_bfloat16* dO,
                        const float* LSE, const int32_t* idx, __nv_bfloat16* dQ, __nv_bfloat16* dK,
                        __nv_bfloat16* dV, void* ws, cudaStream_t st) {
  LRSA_CUDA_CHECK(cudaMemsetAsync(ws, 0, sizeof(WsHeader), st));
  launch_counter().n++;
  RefArgs a = make_args(g);
  a.Q = Q; a.K = K; a.V = V; a.O = O; a.dO = dO; a.LSE = LSE; a.idx = idx;
  a.dQ = dQ; a.dK = dK; a.dV = dV;
  a.Dws = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + sizeof(WsHeader));
  const long long qrows = (long long)g.B * g.Hq * g.N, krows = (long long)g.B * g.Hkv * g.N;
  const unsigned qb = (unsigned)((qrows + 7) / 8), kb = (unsigned)((krows + 7) / 8);
  if (g.d == 128) {
    ref_bwd_dq_kernel<128><<<qb, 256, 0, st>>>(a);
    ref_bwd_dkv_kernel<128><<<kb, 256, 0, st>>>(a);
  } else {
    ref_bwd_dq_kernel<64><<<qb, 256, 0, st>>>(a);
    ref_bwd_dkv_kernel<64><<<kb, 256, 0, st>>>(a);
  }
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n += 2;
  return LRSA_OK;
}

// dK, dV only, with D = rowsum(dO*O) supplied by the caller.
int launch_attn_ref_bwd_dkv(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                            const __nv_bfloat16* V, const __nv_bfloat16* dO, const float* LSE,
                            const int32_t* idx, const float* Dsum, __nv_bfloat16* dK, __nv_bfloat16* dV,
                            cudaStream_t st) {
  RefArgs a = make_args(g);
  a.Q = Q; a.K = K; a.V = V; a.dO = dO; a.LSE = LSE; a.idx = idx; a.dK = dK; a.dV = dV;
  a.Dws = const_cast<float*>(Dsum);
  const long long krows = (long long)g.B * g.Hkv * g.N;
  const unsigned kb = (unsigned)((krows + 7) / 8);
  if (g.d == 128) ref_bwd_dkv_kernel<128><<<kb, 256, 0, st>>>(a);
  else ref_bwd_dkv_kernel<64><<<kb, 256, 0, st>>>(a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

}  // namespace lrsa
