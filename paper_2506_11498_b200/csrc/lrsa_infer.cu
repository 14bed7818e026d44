// Inference side of LRSA (Section 3.2: the KV-cache update of Attn-Fill 1 / Attn-Fill 2 and the condensed
// cache of its last paragraph): a physically condensed KV cache that grows token by token, and decode
// attention over it.
//
// Cache of one (batch, KV head), all bf16:
//   list  [S + Wcap*K][d]  the sinks, then K kept rows of every compressed window, in window order
//   ring  [2L][d]          the uncompressed recent tokens: position p >= S sits at row (p - S) mod 2L
// for K and for V, plus idx [Wcap][K] (the kept positions, for inspection and parity).  A query of chunk
// c sees the sinks, windows 0..c-2 through their kept rows, window c-1 and its own chunk causally, so the
// ring only ever needs the last full window and the chunk being filled.  Window c-2 is scored (Eq. 4-8,
// with window c-1 as its reference) and its kept rows are appended to the list when the first token of
// chunk c arrives: not earlier, because the queries of chunk c-1 still see it whole.
//
// Decode attention reads the list prefix and the ring once per KV head for all query heads of the group
// (HBM-bound: 4*d bytes per key, a few FMAs per byte): the keys are split over CTAs, every warp keeps an
// online softmax per query head, and a second small kernel merges the partial results.
#include "lrsa_internal.h"
#include "sm100_ptx.h"

namespace lrsa {
namespace {

struct CacheLayout {
  int rows_list;   // S + Wcap*K
  int Wcap;        // windows that can ever be compressed with seq_len tokens of capacity
  size_t k_list, v_list, k_ring, v_ring, idx, total;
};

CacheLayout cache_layout(const Geom& g) {
  CacheLayout c;
  // the last token of the capacity sits in chunk (N-1-S)/L; windows up to that chunk minus two get compressed
  const int c_last = g.N > g.S ? (g.N - 1 - g.S) / g.L : 0;
  c.Wcap = c_last >= 2 ? c_last - 1 : 0;
  c.rows_list = g.S + c.Wcap * g.K;
  const size_t BH = (size_t)g.B * g.Hkv;
  const size_t list = align_up(BH * (c.rows_list > 0 ? c.rows_list : 1) * g.d * sizeof(__nv_bfloat16), 256);
  const size_t ring = align_up(BH * 2 * g.L * g.d * sizeof(__nv_bfloat16), 256);
  size_t off = 256;
  c.k_list = off; off += list;
  c.v_list = off; off += list;
  c.k_ring = off; off += ring;
  c.v_ring = off; off += ring;
  c.idx = off; off += align_up(BH * (c.Wcap > 0 ? c.Wcap : 1) * g.K * sizeof(int32_t), 256);
  c.total = off;
  return c;
}

// New tokens [p0, p1) of every (batch, KV head) into the sink rows of the list or into the ring.
// One warp per (head, token); src rows are [BH][n_new][d] with token p at row p - p_first.
__global__ void cache_insert_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                                    __nv_bfloat16* k_list, __nv_bfloat16* v_list, __nv_bfloat16* k_ring,
                                    __nv_bfloat16* v_ring, int BH, int n_new, int p_first, int p0, int p1, int S, int L,
                                    int rows_list, int d) {
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int n = p1 - p0;
  if (wid >= (long long)BH * n) return;
  const int bh = (int)(wid / n), p = p0 + (int)(wid % n), lane = threadIdx.x & 31;
  const size_t src = ((size_t)bh * n_new + (p - p_first)) * d;
  __nv_bfloat16 *kd, *vd;
  if (p < S) {
    kd = k_list + ((size_t)bh * rows_list + p) * d; vd = v_list + ((size_t)bh * rows_list + p) * d;
  } else {
    const size_t r = ((size_t)bh * 2 * L + (p - S) % (2 * L)) * d;
    kd = k_ring + r; vd = v_ring + r;
  }
  for (int c = lane * 2; c < d; c += 64) {
    *reinterpret_cast<uint32_t*>(kd + c) = *reinterpret_cast<const uint32_t*>(k_new + src + c);
    *reinterpret_cast<uint32_t*>(vd + c) = *reinterpret_cast<const uint32_t*>(v_new + src + c);
  }
}

// The K kept rows of window w, from the ring to rows S + w*K ... of the list.  One warp per (head, kept row).
__global__ void cache_keep_kernel(const int32_t* __restrict__ idx, const __nv_bfloat16* __restrict__ k_ring,
                                  const __nv_bfloat16* __restrict__ v_ring, __nv_bfloat16* k_list, __nv_bfloat16* v_list,
                                  int BH, int w, int Wcap, int K, int S, int L, int rows_list, int d) {
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= (long long)BH * K) return;
  const int bh = (int)(wid / K), r = (int)(wid % K), lane = threadIdx.x & 31;
  const int pos = idx[((size_t)bh * Wcap + w) * K + r];
  const size_t src = ((size_t)bh * 2 * L + (pos - S) % (2 * L)) * d;
  const size_t dst = ((size_t)bh * rows_list + S + (size_t)w * K + r) * d;
  for (int c = lane * 2; c < d; c += 64) {
    *reinterpret_cast<uint32_t*>(k_list + dst + c) = *reinterpret_cast<const uint32_t*>(k_ring + src + c);
    *reinterpret_cast<uint32_t*>(v_list + dst + c) = *reinterpret_cast<const uint32_t*>(v_ring + src + c);
  }
}


// ---- decode attention ----
constexpr int kDecThreads = 128;
constexpr int kDecHeads = 8;      // query heads of a group handled per pass over the keys
constexpr int kDecKeys = 128;     // keys per CTA, staged in shared memory by bulk copies

struct DecodeArgs {
  const __nv_bfloat16 *q, *k_list, *v_list, *k_ring, *v_ring;
  float* part;          // [BHkv][n_split][G][D + 2]: unnormalised output, running maximum (log2 domain), sum
  int* status;          // workspace status word
  int BHkv, Hq, Hkv, G, rows_list, L, S;
  int n_list, n_ring, ring0;   // keys: list rows [0, n_list), then n_ring ring rows starting at ring row ring0
  int n_split;
  float scale_log2;
};

__device__ __forceinline__ float bf_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Grid (n_split, BHkv).  The CTA's (at most) 128 keys are runs of consecutive rows of the list and of the
// ring (at most three runs: the ring wraps once); one thread fetches K and V of every run with bulk copies,
// so all of the CTA's bytes are in flight at once.  Then D/8 lanes share a key (16 bytes each), a warp works
// on 32/(D/8) keys at a time, and every such lane group keeps an online softmax (maximum, sum, 8 output
// channels per lane) per query head.
template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(const DecodeArgs a) {
  constexpr int LPK = D / 8, KPW = 32 / LPK;           // lanes per key, keys per warp step
  constexpr int kGroups = (kDecThreads / 32) * KPW;    // lane groups per CTA
  extern __shared__ __align__(128) unsigned char dec_smem[];   // K rows [kDecKeys][D], then V rows
  __shared__ __align__(8) uint64_t bar;
  __shared__ float red_m[kGroups][kDecHeads], red_l[kGroups][kDecHeads];
  __shared__ float red_o[kGroups][D];
  __shared__ int s_fail;
  const int bh = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPK, ch = (lane % LPK) * 8, grp = warp * KPW + sub;
  const int n_keys = a.n_list + a.n_ring;
  const int k_lo = split * kDecKeys, k_hi = min(n_keys, k_lo + kDecKeys), nk = k_hi - k_lo;
  const int b = bh / a.Hkv, hkv = bh % a.Hkv;
  __nv_bfloat16* sK = reinterpret_cast<__nv_bfloat16*>(dec_smem);
  __nv_bfloat16* sV = sK + kDecKeys * D;
  if (tid == 0) {
    s_fail = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_barrier_init();
    ptx::mbar_expect_tx(ptx::smem_u32(&bar), (uint32_t)nk * D * 2 * 2);
    const __nv_bfloat16* kl = a.k_list + (size_t)bh * a.rows_list * D;
    const __nv_bfloat16* vl = a.v_list + (size_t)bh * a.rows_list * D;
    const __nv_bfloat16* kr = a.k_ring + (size_t)bh * 2 * a.L * D;
    const __nv_bfloat16* vr = a.v_ring + (size_t)bh * 2 * a.L * D;
    int i = k_lo;
    while (i < k_hi) {
      const __nv_bfloat16 *ks, *vs;
      int run;
      if (i < a.n_list) {
        run = min(k_hi, a.n_list) - i;
        ks = kl + (size_t)i * D; vs = vl + (size_t)i * D;
      } else {
        const int r = (a.ring0 + (i - a.n_list)) % (2 * a.L);
        run = min(k_hi - i, 2 * a.L - r);
        ks = kr + (size_t)r * D; vs = vr + (size_t)r * D;
      }
      const uint32_t bytes = (uint32_t)run * D * 2;
      bulk_load(ptx::smem_u32(sK + (size_t)(i - k_lo) * D), ks, bytes, ptx::smem_u32(&bar));
      bulk_load(ptx::smem_u32(sV + (size_t)(i - k_lo) * D), vs, bytes, ptx::smem_u32(&bar));
      i += run;
    }
  }
  __syncthreads();
  {
    // bounded wait for the copies; a CTA that gives up records it and leaves its partial result empty
    bool ok = ptx::mbar_try_wait(ptx::smem_u32(&bar), 0);
    const long long t0 = clock64();
    while (!ok) {
      ok = ptx::mbar_try_wait(ptx::smem_u32(&bar), 0);
      if (!ok && clock64() - t0 > 4000000000LL) { s_fail = 1; break; }
    }
  }
  __syncthreads();
  const bool failed = s_fail != 0;
  if (failed && tid == 0) atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);

  for (int g0 = 0; g0 < a.G; g0 += kDecHeads) {
    const int ng = min(kDecHeads, a.G - g0);
    float q[kDecHeads][8], acc[kDecHeads][8], m[kDecHeads], l[kDecHeads];
#pragma unroll
    for (int g = 0; g < kDecHeads; ++g) {
      m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) { acc[g][e] = 0.f; q[g][e] = 0.f; }
      if (g < ng) {
        const uint4 x = *reinterpret_cast<const uint4*>(a.q + ((size_t)(b * a.Hq + hkv * a.G + g0 + g)) * D + ch);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) { q[g][2 * e] = bf_lo(w[e]) * a.scale_log2; q[g][2 * e + 1] = bf_hi(w[e]) * a.scale_log2; }
      }
    }
    for (int i0 = warp * KPW; i0 < nk && !failed; i0 += (kDecThreads / 32) * KPW) {
      const int i = i0 + sub;
      const bool live = i < nk;
      uint4 kx = make_uint4(0, 0, 0, 0), vx = make_uint4(0, 0, 0, 0);
      if (live) {
        kx = *reinterpret_cast<const uint4*>(sK + (size_t)i * D + ch);
        vx = *reinterpret_cast<const uint4*>(sV + (size_t)i * D + ch);
      }
      const uint32_t kw[4] = {kx.x, kx.y, kx.z, kx.w}, vw[4] = {vx.x, vx.y, vx.z, vx.w};
      float kf[8], vf[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kf[2 * e] = bf_lo(kw[e]); kf[2 * e + 1] = bf_hi(kw[e]);
        vf[2 * e] = bf_lo(vw[e]); vf[2 * e + 1] = bf_hi(vw[e]);
      }
#pragma unroll
      for (int g = 0; g < kDecHeads; ++g) {
        if (g < ng) {   // uniform over the CTA
          float s = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) s = fmaf(q[g][e], kf[e], s);
#pragma unroll
          for (int o = LPK / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if (live) {
            const float mn = fmaxf(m[g], s);
            const float f = exp2f(m[g] - mn), pr = exp2f(s - mn);   // exp2f(-inf) = 0 on the first key
            l[g] = l[g] * f + pr;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[g][e] = fmaf(acc[g][e], f, pr * vf[e]);
            m[g] = mn;
          }
        }
      }
    }
    // merge the lane groups of the CTA: one head at a time through shared memory
    for (int g = 0; g < ng; ++g) {
      __syncthreads();
      if (lane % LPK == 0) { red_m[grp][g] = m[g]; red_l[grp][g] = l[g]; }
#pragma unroll
      for (int e = 0; e < 8; ++e) red_o[grp][ch + e] = acc[g][e];
      __syncthreads();
      if (tid < D) {
        float M = -INFINITY;
        for (int r = 0; r < kGroups; ++r) M = fmaxf(M, red_m[r][g]);
        float o = 0.f, lsum = 0.f;
        for (int r = 0; r < kGroups; ++r) {
          const float f = red_m[r][g] == -INFINITY ? 0.f : exp2f(red_m[r][g] - M);
          o = fmaf(red_o[r][tid], f, o);
          lsum = fmaf(red_l[r][g], f, lsum);
        }
        float* dst = a.part + (((size_t)bh * a.n_split + split) * a.G + g0 + g) * (D + 2);
        dst[tid] = o;
        if (tid == 0) { dst[D] = M; dst[D + 1] = lsum; }
      }
    }
  }
}

// One CTA per (batch, query head): merges the partial results of the splits.  kMergeRows thread rows take
// alternate splits (so their loads are in flight together), then the rows are merged through shared memory.
constexpr int kMergeRows = 8;
template <int D>
__global__ void __launch_bounds__(kMergeRows * D) decode_merge_kernel(const float* __restrict__ part,
                                                                       __nv_bfloat16* __restrict__ o,
                                                                       float* __restrict__ lse, int Hq, int Hkv, int G,
                                                                       int n_split) {
  __shared__ float sm_m[kMergeRows], sm_l[kMergeRows], sm_o[kMergeRows][D];
  const int bhq = blockIdx.x, b = bhq / Hq, hq = bhq % Hq, hkv = hq / G, g = hq % G;
  const int c = threadIdx.x % D, row = threadIdx.x / D;
  const float* base = part + (((size_t)(b * Hkv + hkv) * n_split) * G + g) * (D + 2);
  const size_t stride = (size_t)G * (D + 2);
  float M = -INFINITY, acc = 0.f, l = 0.f;
  for (int s = row; s < n_split; s += kMergeRows) {
    const float ms = base[s * stride + D];
    if (ms == -INFINITY) continue;
    const float mn = fmaxf(M, ms), f0 = exp2f(M - mn), f1 = exp2f(ms - mn);
    acc = acc * f0 + base[s * stride + c] * f1;
    l = l * f0 + base[s * stride + D + 1] * f1;
    M = mn;
  }
  sm_o[row][c] = acc;
  if (c == 0) { sm_m[row] = M; sm_l[row] = l; }
  __syncthreads();
  if (row == 0) {
    float Mt = -INFINITY;
    for (int r = 0; r < kMergeRows; ++r) Mt = fmaxf(Mt, sm_m[r]);
    float at = 0.f, lt = 0.f;
    for (int r = 0; r < kMergeRows; ++r) {
      const float f = sm_m[r] == -INFINITY ? 0.f : exp2f(sm_m[r] - Mt);
      at = fmaf(sm_o[r][c], f, at);
      lt = fmaf(sm_l[r], f, lt);
    }
    o[(size_t)bhq * D + c] = __float2bfloat16(at / lt);
    if (c == 0 && lse) lse[bhq] = (Mt + log2f(lt)) * 0.6931471805599453f;
  }
}

int decode_splits(int n_keys) { return n_keys > 0 ? (n_keys + kDecKeys - 1) / kDecKeys : 1; }

}  // namespace
}  // namespace lrsa

using namespace lrsa;

extern "C" {

int lrsa_cache_bytes(const lrsa_params_t* params, size_t* cache_bytes, size_t* workspace_bytes) {
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (params->n_seqs > 0 || g.ndp != 1) return LRSA_ERR_UNSUPPORTED;
  if (cache_bytes) *cache_bytes = cache_layout(g).total;
  if (workspace_bytes) {
    // scoring scratch of a two-window problem, or the partial results of the decode kernel
    Geom two = g;
    two.N = two.Nrow = 2 * g.L; two.S = 0; two.W = 2; two.Wsel = 1; two.T = 0; two.C = 2;
    const size_t a = score_select_ws_bytes(two);
    // a sequence of N tokens never shows a query more than S + Wcap*K + 2L keys
    const size_t b = 256 + (size_t)g.B * g.Hkv * decode_splits(cache_layout(g).rows_list + 2 * g.L) * g.G * (g.d + 2) * sizeof(float);
    *workspace_bytes = a > b ? a : b;
  }
  return LRSA_OK;
}

int lrsa_cache_append(const lrsa_params_t* params, void* cache, size_t cache_bytes, const void* k_new,
                      const void* v_new, int32_t n_prev, int32_t n_new, void* workspace, size_t workspace_bytes,
                      void* cuda_stream) {
  NvtxRange nvtx_range("lrsa_cache_append");
  launch_counter().n = 0;
  Geom g;
  int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (params->n_seqs > 0 || g.ndp != 1) return LRSA_ERR_UNSUPPORTED;
  if (!cache || !k_new || !v_new || !workspace || n_prev < 0 || n_new < 1 || (long long)n_prev + n_new > g.N)
    return LRSA_ERR_INVALID_ARG;
  auto mis = [](const void* p, size_t al) { return reinterpret_cast<uintptr_t>(p) % al != 0; };
  if (mis(cache, 256) || mis(workspace, 256) || mis(k_new, 16) || mis(v_new, 16)) return LRSA_ERR_INVALID_ARG;
  const CacheLayout lay = cache_layout(g);
  size_t need_ws = 0;
  lrsa_cache_bytes(params, nullptr, &need_ws);
  if (cache_bytes < lay.total || workspace_bytes < need_ws) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  auto st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* cb = static_cast<unsigned char*>(cache);
  auto* k_list = reinterpret_cast<__nv_bfloat16*>(cb + lay.k_list);
  auto* v_list = reinterpret_cast<__nv_bfloat16*>(cb + lay.v_list);
  auto* k_ring = reinterpret_cast<__nv_bfloat16*>(cb + lay.k_ring);
  auto* v_ring = reinterpret_cast<__nv_bfloat16*>(cb + lay.v_ring);
  auto* idx = reinterpret_cast<int32_t*>(cb + lay.idx);
  const int BH = g.B * g.Hkv;
  LRSA_CUDA_CHECK(cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st));
  launch_counter().n++;
  int pos = n_prev;
  const int end = n_prev + n_new;
  while (pos < end) {
    int seg_end = end;
    if (pos < g.S) {
      seg_end = end < g.S ? end : g.S;
    } else {
      const int c = (pos - g.S) / g.L;
      if (pos == g.S + c * g.L && c >= 2) {
        // The first token of chunk c: window c-2 leaves the ring.  It is scored with window c-1 as its
        // reference (the two halves of the ring, in either order) and its kept rows join the list.
        const int w = c - 2;
        Geom two = g;
        two.N = 2 * g.L; two.Nrow = 2 * g.L; two.S = 0; two.W = 2; two.Wsel = 1; two.T = 0; two.C = 2;
        two.tok0 = (w % 2) * g.L;
        two.win_stride = (w % 2) ? -g.L : g.L;
        two.emit_off = g.S + w * g.L;
        two.Wtot = lay.Wcap; two.woff = w;
        rc = launch_score_select(two, k_ring, v_ring, idx, nullptr, workspace, st);
        if (rc != LRSA_OK) return rc;
        const long long warps = (long long)BH * g.K;
        cache_keep_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(idx, k_ring, v_ring, k_list, v_list, BH, w,
                                                                     lay.Wcap, g.K, g.S, g.L, lay.rows_list, g.d);
        LRSA_CUDA_CHECK(cudaGetLastError());
        launch_counter().n++;
      }
      const int next = g.S + (c + 1) * g.L;
      seg_end = end < next ? end : next;
    }
    const long long warps = (long long)BH * (seg_end - pos);
    cache_insert_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), k_list, v_list, k_ring,
        v_ring, BH, n_new, n_prev, pos, seg_end, g.S, g.L, lay.rows_list, g.d);
    LRSA_CUDA_CHECK(cudaGetLastError());
    launch_counter().n++;
    pos = seg_end;
  }
  return LRSA_OK;
}

int lrsa_cache_kept(const lrsa_params_t* params, const void* cache, const int32_t** idx, int32_t* w_cap) {
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!cache || !idx) return LRSA_ERR_INVALID_ARG;
  const CacheLayout lay = cache_layout(g);
  *idx = reinterpret_cast<const int32_t*>(static_cast<const unsigned char*>(cache) + lay.idx);
  if (w_cap) *w_cap = lay.Wcap;
  return LRSA_OK;
}

int lrsa_attn_decode(const lrsa_params_t* params, const void* cache, size_t cache_bytes, const void* q,
                     int32_t n_tokens, void* o, float* lse, void* workspace, size_t workspace_bytes,
                     void* cuda_stream) {
  NvtxRange nvtx_range("lrsa_attn_decode");
  launch_counter().n = 0;
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (params->n_seqs > 0 || g.ndp != 1) return LRSA_ERR_UNSUPPORTED;
  if (!cache || !q || !o || !workspace || n_tokens < 1 || n_tokens > g.N) return LRSA_ERR_INVALID_ARG;
  auto mis = [](const void* p, size_t al) { return reinterpret_cast<uintptr_t>(p) % al != 0; };
  if (mis(cache, 256) || mis(workspace, 256) || mis(q, 16) || mis(o, 16) || mis(lse, 4)) return LRSA_ERR_INVALID_ARG;
  const CacheLayout lay = cache_layout(g);
  size_t need_ws = 0;
  lrsa_cache_bytes(params, nullptr, &need_ws);
  if (cache_bytes < lay.total || workspace_bytes < need_ws) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  auto st = static_cast<cudaStream_t>(cuda_stream);
  const unsigned char* cb = static_cast<const unsigned char*>(cache);
  DecodeArgs a;
  a.q = static_cast<const __nv_bfloat16*>(q);
  a.k_list = reinterpret_cast<const __nv_bfloat16*>(cb + lay.k_list);
  a.v_list = reinterpret_cast<const __nv_bfloat16*>(cb + lay.v_list);
  a.k_ring = reinterpret_cast<const __nv_bfloat16*>(cb + lay.k_ring);
  a.v_ring = reinterpret_cast<const __nv_bfloat16*>(cb + lay.v_ring);
  a.part = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + 256);
  a.BHkv = g.B * g.Hkv; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.rows_list = lay.rows_list > 0 ? lay.rows_list : 1;
  a.L = g.L; a.S = g.S;
  // the keys the query at position t = n_tokens - 1 sees (Attn-Fill 1/2): a sink query its causal prefix;
  // otherwise the sinks, the kept rows of windows 0..c-2, and positions [S + (c-1)L, t] from the ring
  const int t = n_tokens - 1;
  if (t < g.S) {
    a.n_list = t + 1; a.n_ring = 0; a.ring0 = 0;
  } else {
    const int c = (t - g.S) / g.L, nc = c >= 1 ? c - 1 : 0;
    a.n_list = g.S + nc * g.K;
    a.n_ring = t - (g.S + nc * g.L) + 1;
    a.ring0 = (nc * g.L) % (2 * g.L);
  }
  a.n_split = decode_splits(a.n_list + a.n_ring);
  a.scale_log2 = g.scale * 1.4426950408889634f;
  a.status = &reinterpret_cast<WsHeader*>(workspace)->status;
  LRSA_CUDA_CHECK(cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st));
  launch_counter().n++;
  const dim3 grid(a.n_split, a.BHkv);
  const size_t smem = (size_t)2 * kDecKeys * g.d * sizeof(__nv_bfloat16);
  if (g.d == 128) {
    LRSA_CUDA_CHECK(cudaFuncSetAttribute(decode_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_partial_kernel<128><<<grid, kDecThreads, smem, st>>>(a);
  } else {
    LRSA_CUDA_CHECK(cudaFuncSetAttribute(decode_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_partial_kernel<64><<<grid, kDecThreads, smem, st>>>(a);
  }
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  if (g.d == 128)
    decode_merge_kernel<128><<<g.B * g.Hq, kMergeRows * 128, 0, st>>>(a.part, static_cast<__nv_bfloat16*>(o), lse, g.Hq, g.Hkv, g.G, a.n_split);
  else
    decode_merge_kernel<64><<<g.B * g.Hq, kMergeRows * 64, 0, st>>>(a.part, static_cast<__nv_bfloat16*>(o), lse, g.Hq, g.Hkv, g.G, a.n_split);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

}  // extern "C"
