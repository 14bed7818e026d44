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
constexpr int kDecHeads = 16;     // query heads of a group per pass over the keys (the M of the tensor-core product)
constexpr int kDecKeys = 128;     // keys per CTA (32 per warp), staged in shared memory

struct DecodeArgs {
  const __nv_bfloat16 *q, *k_list, *v_list, *k_ring, *v_ring;
  float* part;          // [BHkv][n_split][G][D + 2]: unnormalised output, running maximum (log2 domain), sum
  int* status;          // workspace status word
  int BHkv, Hq, Hkv, G, rows_list, L, S;
  int n_list, n_ring, ring0;   // keys: list rows [0, n_list), then n_ring ring rows starting at ring row ring0
  int n_split;
  float scale_log2;
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Grid (n_split, BHkv).  One query token per (batch, head) and a few hundred to a few thousand keys per KV head:
// the work is the transfer of K and V, so the CTA's (at most) 128 key rows are fetched at once (every thread
// issues one bulk copy for its row of K and one for its row of V) and everything after that has to be short.
// The query heads of the KV group form the rows of a small matrix product (GQA: 16 rows per pass, the unused
// ones zero), so S = Q K^T and O = P V run on the warp-level tensor-core instructions (m16n8k16, bf16 operands,
// fp32 accumulation; a 128-row tcgen05 product would be nine tenths padding here): a warp takes 32 keys, reads
// Q, K and V fragments with ldmatrix from rows padded by 16 bytes (rows 128 or 256 bytes apart would put the
// eight rows of a fragment on the same banks), forms the softmax of its 32 keys in registers and hands P over
// as the A operand of the second product.  The four warps' partial results are merged through shared memory;
// the splits by decode_merge_kernel.
template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(const DecodeArgs a) {
  constexpr int CPR = D / 8;                 // 16-byte chunks per row
  constexpr int KS = D / 16;                 // k-steps of Q K^T
  constexpr int NT = D / 8;                  // 8-channel tiles of the output
  constexpr int kRowBytes = D * 2, kStride = kRowBytes + 16;
  extern __shared__ __align__(128) unsigned char dec_smem[];   // K rows [kDecKeys], V rows [kDecKeys], Q rows [16]
  __shared__ __align__(8) uint64_t bar;
  __shared__ int s_fail;
  const int bh = blockIdx.y, split = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_keys = a.n_list + a.n_ring;
  const int k_lo = split * kDecKeys, k_hi = min(n_keys, k_lo + kDecKeys), nk = k_hi - k_lo;
  const int b = bh / a.Hkv, hkv = bh % a.Hkv;
  const uint32_t sK = ptx::smem_u32(dec_smem), sV = sK + kDecKeys * kStride, sQ = sV + kDecKeys * kStride;
  unsigned char* gQ = dec_smem + 2 * kDecKeys * kStride;
  // The merge kernel is launched as a programmatic dependent of this one: its CTAs may be scheduled from here
  // on and wait (griddepcontrol.wait) until this grid has completed and its stores are visible.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    s_fail = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_barrier_init();
    ptx::mbar_expect_tx(ptx::smem_u32(&bar), (uint32_t)nk * kRowBytes * 2);   // every row copy below reports here
    // the only writer of the status word before a wait below can expire (seconds later)
    if (split == 0 && bh == 0) *a.status = 0;
  }
  __syncthreads();
  {
    // this thread's row of K and of V
    const int r = tid;
    if (r < nk) {
      const int k = k_lo + r;
      const __nv_bfloat16 *ks, *vs;
      if (k < a.n_list) {
        const size_t off = ((size_t)bh * a.rows_list + k) * D;
        ks = a.k_list + off; vs = a.v_list + off;
      } else {
        const size_t off = ((size_t)bh * 2 * a.L + (a.ring0 + (k - a.n_list)) % (2 * a.L)) * D;
        ks = a.k_ring + off; vs = a.v_ring + off;
      }
      bulk_load(sK + r * kStride, ks, kRowBytes, ptx::smem_u32(&bar));
      bulk_load(sV + r * kStride, vs, kRowBytes, ptx::smem_u32(&bar));
    } else {
      // rows beyond the split's keys: their probabilities are zero, their V must not be NaN
#pragma unroll
      for (int c = 0; c < CPR; ++c) {
        *reinterpret_cast<uint4*>(dec_smem + r * kStride + c * 16) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(dec_smem + (kDecKeys + r) * kStride + c * 16) = make_uint4(0, 0, 0, 0);
      }
    }
  }

  const int row = lane >> 2, cpair = (lane & 3) * 2;   // fragment coordinates of this lane
  for (int g0 = 0; g0 < a.G; g0 += kDecHeads) {
    const int ng = min(kDecHeads, a.G - g0);
    // Q of this pass: 16 rows (heads g0 ..., zero beyond the group) into shared memory, 16 bytes per thread and step
    for (int i = tid; i < kDecHeads * CPR; i += kDecThreads) {
      const int g = i / CPR, cch = i % CPR;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (g < ng) v = *reinterpret_cast<const uint4*>(a.q + ((size_t)(b * a.Hq + hkv * a.G + g0 + g)) * D + cch * 8);
      *reinterpret_cast<uint4*>(gQ + g * kStride + cch * 16) = v;
    }
    if (g0 == 0) {
      // bounded wait for the copies; a CTA that gives up records it, waits once more for its copies (they write
      // this CTA's shared memory) and leaves its partial result empty
      bool got = ptx::mbar_try_wait(ptx::smem_u32(&bar), 0);
      const long long t0 = clock64();
      while (!got) {
        got = ptx::mbar_try_wait(ptx::smem_u32(&bar), 0);
        if (!got && clock64() - t0 > 4000000000LL) { s_fail = 1; break; }
      }
    }
    __syncthreads();
    if (s_fail) {
      if (tid == 0) {
        atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(ptx::smem_u32(&bar), 0) && clock64() - t0 < 4000000000LL) {}
      }
      __syncthreads();
      // empty partial results: maximum -inf, the merge kernel skips them
      for (int i = tid; i < ng; i += kDecThreads) {
        float* dst = a.part + (((size_t)bh * a.n_split + split) * a.G + g0 + i) * (D + 2);
        dst[D] = -INFINITY; dst[D + 1] = 0.f;
      }
      continue;
    }
    // Q as A fragments: matrices (heads 0-7, channels k..k+7), (heads 8-15, same), then channels k+8..k+15
    uint32_t qa[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
      ldmatrix_x4(sQ + ((lane & 7) + 8 * ((lane >> 3) & 1)) * kStride + (2 * ks + (lane >> 4)) * 16, qa[ks]);
    // S = Q K^T for this warp's 32 keys: four tiles of 8 keys
    float s[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
      const int key = warp * 32 + 8 * j + (lane & 7);
#pragma unroll
      for (int q4 = 0; q4 < CPR / 4; ++q4) {
        uint32_t kb[4];
        ldmatrix_x4(sK + key * kStride + (4 * q4 + (lane >> 3)) * 16, kb);
        mma_16816(s[j], qa[2 * q4], kb[0], kb[1]);
        mma_16816(s[j], qa[2 * q4 + 1], kb[2], kb[3]);
      }
    }
    // scale, mask the keys beyond the split, row maxima and sums (rows: head `row` -> index 0, `row + 8` -> 1)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = warp * 32 + 8 * j + cpair + (e & 1);
        s[j][e] = key < nk ? s[j][e] * a.scale_log2 : -INFINITY;
        mx[e >> 1] = fmaxf(mx[e >> 1], s[j][e]);
      }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
    }
    float sum[2] = {0.f, 0.f};
    uint32_t pa[2][4];   // P as A fragments of the two 16-key steps
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float pr[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        pr[e] = mx[e >> 1] == -INFINITY ? 0.f : exp2f(s[j][e] - mx[e >> 1]);
        sum[e >> 1] += pr[e];
      }
      pa[j >> 1][(j & 1) * 2 + 0] = ptx::pack_bf16(pr[0], pr[1]);
      pa[j >> 1][(j & 1) * 2 + 1] = ptx::pack_bf16(pr[2], pr[3]);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 1);
      sum[h] += __shfl_xor_sync(0xffffffffu, sum[h], 2);
    }
    // O = P V: V fragments transposed on the way out of shared memory (keys are the contraction index)
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
      uint32_t vb[4];
      ldmatrix_x4_trans(sV + (warp * 32 + lane) * kStride + nt * 16, vb);
      mma_16816(o[nt], pa[0], vb[0], vb[1]);
      mma_16816(o[nt], pa[1], vb[2], vb[3]);
    }
    // merge the four warps through shared memory (the K rows are no longer needed once every warp is here;
    // with more than one pass over the heads they are needed again, so the merge buffer then follows V)
    __syncthreads();
    float* mrg = reinterpret_cast<float*>(dec_smem + (a.G > kDecHeads ? (2 * kDecKeys + kDecHeads) * kStride : 0));
    float* mo = mrg;                                   // [4 warps][16 heads][D]
    float* mm_ = mrg + 4 * kDecHeads * D;              // [4][16] maxima
    float* ml = mm_ + 4 * kDecHeads;                   // [4][16] sums
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      *reinterpret_cast<float2*>(mo + ((warp * kDecHeads + row) * D + nt * 8 + cpair)) = make_float2(o[nt][0], o[nt][1]);
      *reinterpret_cast<float2*>(mo + ((warp * kDecHeads + row + 8) * D + nt * 8 + cpair)) = make_float2(o[nt][2], o[nt][3]);
    }
    if ((lane & 3) == 0) {
      mm_[warp * kDecHeads + row] = mx[0]; mm_[warp * kDecHeads + row + 8] = mx[1];
      ml[warp * kDecHeads + row] = sum[0]; ml[warp * kDecHeads + row + 8] = sum[1];
    }
    __syncthreads();
    for (int i = tid; i < ng * D; i += kDecThreads) {
      const int g = i / D, c = i % D;
      float M = -INFINITY;
#pragma unroll
      for (int w = 0; w < 4; ++w) M = fmaxf(M, mm_[w * kDecHeads + g]);
      float ov = 0.f, lsum = 0.f;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float mw = mm_[w * kDecHeads + g];
        const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
        ov = fmaf(mo[(w * kDecHeads + g) * D + c], f, ov);
        lsum = fmaf(ml[w * kDecHeads + g], f, lsum);
      }
      float* dst = a.part + (((size_t)bh * a.n_split + split) * a.G + g0 + g) * (D + 2);
      dst[c] = ov;
      if (c == 0) { dst[D] = M; dst[D + 1] = lsum; }
    }
    __syncthreads();   // the merge buffer is reused by the next pass
  }
}

// One CTA per (batch, query head): merges the partial results of the splits.  kMergeRows thread rows take
// alternate splits, four at a time with all their loads issued before the arithmetic (the kernel is a chain of
// L2 round trips otherwise), then the rows are merged through shared memory.
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
  constexpr int kBatch = 4;
  // launched as a programmatic dependent of the partial kernel: wait for its grid to complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int s0 = row; s0 < n_split; s0 += kMergeRows * kBatch) {
    float ms[kBatch], vs[kBatch], ls[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int s = s0 + u * kMergeRows;
      const bool in = s < n_split;
      ms[u] = in ? __ldcg(base + s * stride + D) : -INFINITY;
      vs[u] = in ? __ldcg(base + s * stride + c) : 0.f;
      ls[u] = in ? __ldcg(base + s * stride + D + 1) : 0.f;
    }
    float mn = M;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) mn = fmaxf(mn, ms[u]);
    if (mn == -INFINITY) continue;
    const float f0 = exp2f(M - mn);   // exp2f(-inf) = 0 while nothing has been merged
    acc *= f0; l *= f0;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const float f = exp2f(ms[u] - mn);
      acc = fmaf(vs[u], f, acc);
      l = fmaf(ls[u], f, l);
    }
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
  const dim3 grid(a.n_split, a.BHkv);
  // K and V rows; the merge buffer (4 warps x 16 heads x (d + 2) floats) lies over them, or behind them when the
  // group has more than 16 query heads and the rows are read again
  const size_t rows_bytes = (size_t)(2 * kDecKeys + kDecHeads) * (g.d * sizeof(__nv_bfloat16) + 16);   // K, V and Q rows, padded
  const size_t merge_bytes = (size_t)4 * kDecHeads * (g.d + 2) * sizeof(float);
  const size_t smem = g.G > kDecHeads ? rows_bytes + merge_bytes : (rows_bytes > merge_bytes ? rows_bytes : merge_bytes);
  if (g.d == 128) {
    LRSA_CUDA_CHECK(cudaFuncSetAttribute(decode_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_partial_kernel<128><<<grid, kDecThreads, smem, st>>>(a);
  } else {
    LRSA_CUDA_CHECK(cudaFuncSetAttribute(decode_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    decode_partial_kernel<64><<<grid, kDecThreads, smem, st>>>(a);
  }
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  {
    // programmatic dependent launch: the merge kernel's launch latency overlaps the partial kernel
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.B * g.Hq);
    cfg.blockDim = dim3(kMergeRows * g.d);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* part = a.part;
    __nv_bfloat16* op = static_cast<__nv_bfloat16*>(o);
    if (g.d == 128)
      LRSA_CUDA_CHECK(cudaLaunchKernelEx(&cfg, decode_merge_kernel<128>, part, op, lse, g.Hq, g.Hkv, g.G, a.n_split));
    else
      LRSA_CUDA_CHECK(cudaLaunchKernelEx(&cfg, decode_merge_kernel<64>, part, op, lse, g.Hq, g.Hkv, g.G, a.n_split));
  }
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

}  // extern "C"
