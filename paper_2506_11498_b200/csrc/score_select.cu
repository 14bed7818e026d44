// LagKV scoring and top-K selection (Section 3.2, Eq. 4-8 and the selection rule after Eq. 8).
//
// Two kernels, chosen by the lag window size:
//   * score_select_chain_kernel (lag windows of up to 4096 tokens: the hot path).  A CTA owns a run of
//     consecutive scored windows of one (batch, KV head), streams them downwards through a ring of bulk
//     copies and keeps statistics and spreads in shared memory; no traffic between CTAs.  Described in
//     front of the kernel below.
//   * score_select_kernel (longer windows).  The work unit is a slice of TOK tokens of one lag window; a
//     CTA takes one unit from a ticket counter in DESCENDING window order and keeps its slice of K and V
//     in registers for both phases:
//       phase 1  per-channel min/max of the slice (packed bf16x2 compares, exact), folded into the
//                window's statistics in global memory with order-preserving integer atomics, then
//                a release-increment of the window's `ready` counter            (Eq. 4, Eq. 5)
//       phase 2  wait (bounded) until the FOLLOWING window's statistics are complete, normalise
//                the slice held in registers (Eq. 6), per-token standard deviation over head_dim
//                (Eq. 7, inner part), written to a small fp32 scratch
//       select   the CTA that finishes a window last soft-maxes the window's K and V spreads
//                (Eq. 7), adds them (Eq. 8), radix-selects the top_k scores and emits the kept
//                positions in ascending order.
//     A unit of window w waits only on units of window w+1, all of which hold smaller tickets, were
//     therefore picked up by CTAs that already run, and publish before they wait on anything: the
//     wait always ends, whatever the number of resident CTAs.  It is bounded all the same.
// Both see one sequence: rows of N tokens per (batch, KV head), of which the sequence starts at token tok0
// (packed batches), windows win_stride tokens apart (negative for the two-window ring of the inference cache).
#include <stddef.h>

#include "lrsa_internal.h"
#include "sm100_ptx.h"

namespace lrsa {
namespace {

constexpr int kThreads = 256;
constexpr int kSteps = 4;  // 16-byte row chunks of K (and of V) each thread keeps in registers

struct ScoreArgs {
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  int32_t* idx;
  float* score;   // optional
  WsHeader* hdr;
  int* ready;     // [BH, W]     slices of window w whose min/max are folded in
  int* done;      // [BH, Wsel]  slices of window w whose spreads are written
  uint32_t* mm;   // [BH, W, 2 (K,V), 2 (min,max), d] order-preserving keys, zero = identity
  float* spread;  // [BH, Wsel, 2 (K,V), L]
  int BH, N, L, Kk, S, W, Wsel, n_slices, ddof;   // N: tokens per (batch, head) row of K and V (the row stride)
  int tok0, Wtot, woff;   // the sequence starts at token tok0 of the rows; its windows are [woff, woff + Wsel) of the
                          // Wtot windows per head of idx and score
  int emit_off;           // added to S + w*L + i when a position is written to idx
  int win_stride;         // tokens from window w to window w+1 in memory (L; -L or L for a two-window ring buffer)
  long long elems;        // elements of K (and of V)
  int clear_status;       // the chain kernel's first CTA clears the status word itself (saves a memset node)
  int unit_wait_limit;    // polls of the one-slice-per-CTA kernel's wait for the next window; negative: give up at once
  int spin_limit;
};

// fp32 bits -> uint32 whose unsigned order is the float order (and back).
__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

__device__ __forceinline__ uint32_t bmin2(uint32_t a, uint32_t b) {
  __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ float bf_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Top-K of the window by the last CTA to finish it.  smem: sk[L], sv[L] floats, then scratch.
// Bytes of the selection scratch: sk[L], sv[L], 256 histogram bins, 32 floats, 16 ints.
// Rounded up to 16 bytes: the chain kernel puts a buffer of 16-byte vectors right behind this scratch
// (an odd window length would leave it misaligned otherwise).
__host__ __device__ inline size_t select_scratch_bytes(int L) {
  return (((size_t)2 * L * 4 + 256 * 4 + 32 * 4 + 16 * 4) + 15) & ~(size_t)15;
}

// Barrier of the 256 scoring threads (named barrier 1): the whole block in the one-unit-per-CTA kernel,
// all warps but the producer in the streaming kernel.
__device__ __forceinline__ void scoring_warps_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// `in_smem`: the spreads are already in sk / sv (the chain kernel keeps them there) instead of in a.spread.
__device__ void select_window(const ScoreArgs& a, int bh, int w, unsigned char* smem, bool in_smem = false) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, L = a.L;
  float* sk = reinterpret_cast<float*>(smem);
  float* sv = sk + L;
  uint32_t* hist = reinterpret_cast<uint32_t*>(sv + L);  // 256 bins
  float* red = reinterpret_cast<float*>(hist + 256);     // 32 floats
  int* ibuf = reinterpret_cast<int*>(red + 32);          // 16 ints
  const float* gk = in_smem ? sk : a.spread + ((size_t)(bh * a.Wsel + w) * 2 + 0) * L;
  const float* gv = in_smem ? sv : gk + L;

  // Eq. 7: softmax over the L tokens of the window, for K and for V
  float mk = -INFINITY, mv = -INFINITY;
  for (int i = tid; i < L; i += kThreads) {
    const float x = in_smem ? sk[i] : __ldcg(gk + i), y = in_smem ? sv[i] : __ldcg(gv + i);
    sk[i] = x; sv[i] = y;
    mk = fmaxf(mk, x); mv = fmaxf(mv, y);
  }
  mk = warp_max(mk); mv = warp_max(mv);
  if (lane == 0) { red[warp] = mk; red[8 + warp] = mv; }
  scoring_warps_sync();
  mk = red[0]; mv = red[8];
#pragma unroll
  for (int i = 1; i < 8; ++i) { mk = fmaxf(mk, red[i]); mv = fmaxf(mv, red[8 + i]); }
  scoring_warps_sync();
  float ek = 0.f, ev = 0.f;
  for (int i = tid; i < L; i += kThreads) {
    const float x = expf(sk[i] - mk), y = expf(sv[i] - mv);
    sk[i] = x; sv[i] = y;
    ek += x; ev += y;
  }
  ek = warp_sum(ek); ev = warp_sum(ev);
  if (lane == 0) { red[warp] = ek; red[8 + warp] = ev; }
  scoring_warps_sync();
  ek = 0.f; ev = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) { ek += red[i]; ev += red[8 + i]; }
  // Eq. 8
  float* gs = a.score ? a.score + (size_t)(bh * a.Wtot + a.woff + w) * L : nullptr;
  uint32_t kmin = 0xffffffffu, kmax = 0u;   // range of the keys (scores are positive: bit order = value order)
  for (int i = tid; i < L; i += kThreads) {
    const float s = sk[i] / ek + sv[i] / ev;
    sk[i] = s;
    if (gs) gs[i] = s;
    kmin = min(kmin, __float_as_uint(s));
    kmax = max(kmax, __float_as_uint(s));
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  scoring_warps_sync();   // also: every read of red[] above is done
  uint32_t* kred = reinterpret_cast<uint32_t*>(red);
  if (lane == 0) { kred[warp] = kmin; kred[8 + warp] = kmax; }
  scoring_warps_sync();
#pragma unroll
  for (int i = 0; i < 8; ++i) { kmin = min(kmin, kred[i]); kmax = max(kmax, kred[8 + i]); }

  // radix select of the K-th largest score; scores are positive, so bit order = value order
  // The keys of a window share their leading bits (the scores of one window lie within a small factor of
  // each other): those bits are fixed at once, and the 8-bit passes start at the highest bit in which two
  // keys differ.  (A pass over shared bits would also send every key to one histogram bin: a thousand
  // serialised shared-memory atomics.)
  const uint32_t* key = reinterpret_cast<const uint32_t*>(sk);
  const uint32_t diff = kmin ^ kmax;
  const int top = diff ? 31 - __clz(diff) : -1;                  // highest differing bit, -1: all keys equal
  uint32_t mask = top >= 31 ? 0u : ~((2u << (top < 0 ? 0 : top)) - 1u);
  if (top < 0) mask = 0xffffffffu;
  uint32_t prefix = kmax & mask;
  int remaining = a.Kk;
  for (int shift = top < 0 ? -1 : max(top - 7, 0); shift >= 0; shift = shift == 0 ? -1 : max(shift - 8, 0)) {
    hist[tid] = 0;
    scoring_warps_sync();
    for (int i = tid; i < L; i += kThreads) {
      const uint32_t k = key[i];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 255u], 1u);
    }
    scoring_warps_sync();
    if (warp == 0) {
      // lane l owns bins 255-8l ... 248-8l, highest first
      uint32_t c[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c[j] = hist[255 - 8 * lane - j]; tot += c[j]; }
      uint32_t incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      uint32_t above = incl - tot;  // elements in bins above this lane's
      if (above < (uint32_t)remaining && (uint32_t)remaining <= incl) {
        int j = 0;
        while (above + c[j] < (uint32_t)remaining) { above += c[j]; ++j; }
        ibuf[0] = 255 - 8 * lane - j;
        ibuf[1] = remaining - (int)above;
        ibuf[2] = (int)c[j];   // keys in the chosen bin
      }
    }
    scoring_warps_sync();
    prefix |= (uint32_t)ibuf[0] << shift;
    mask |= 255u << shift;
    remaining = ibuf[1];
    // Every key of the chosen bin is kept: the remaining bits need not be resolved.  (With 8-bit digits a
    // thousand keys are alone in their bin after two passes, so this ends the search at half its length.)
    // The threshold is then the bin's lowest possible key: keys above it are kept as "greater", keys equal to
    // it as "equal", of which `remaining` is at least as many as exist.
    const bool whole_bin = ibuf[2] == remaining;
    scoring_warps_sync();
    if (whole_bin) break;
  }
  const uint32_t kth = prefix;    // K-th largest key
  const int need_eq = remaining;  // how many keys equal to it are kept (lowest positions first)

  // emit kept positions in ascending order: every thread takes a run of consecutive tokens, one block
  // scan gives the number of kept tokens before the run
  int32_t* out = a.idx + (size_t)(bh * a.Wtot + a.woff + w) * a.Kk;
  const int pos0 = a.emit_off + a.S + w * L;   // position of the window's first token
  const int per = (L + kThreads - 1) / kThreads;
  const int i_lo = min(L, tid * per), i_hi = min(L, i_lo + per);
  int packed = 0;   // tokens above the K-th score | tokens equal to it << 16
  for (int i = i_lo; i < i_hi; ++i) {
    const uint32_t k = key[i];
    packed += (k > kth ? 1 : 0) | (k == kth ? 1 << 16 : 0);
  }
  int incl = packed;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  int* wtot = ibuf;  // 8 warp totals (ibuf's last readers passed the barrier that ended the last pass)
  if (lane == 31) wtot[warp] = incl;
  scoring_warps_sync();
  int excl = incl - packed;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    if (j < warp) excl += wtot[j];
  int gt_before = excl & 0xffff, eq_before = excl >> 16;
  for (int i = i_lo; i < i_hi; ++i) {
    const uint32_t k = key[i];
    if (k > kth) {
      out[gt_before + min(eq_before, need_eq)] = pos0 + i;
      ++gt_before;
    } else if (k == kth) {
      if (eq_before < need_eq) out[gt_before + eq_before] = pos0 + i;
      ++eq_before;
    }
  }
  scoring_warps_sync();   // sk and ibuf may be reused by the caller
}

template <int D>
__global__ void __launch_bounds__(kThreads) score_select_kernel(const ScoreArgs a) {
  constexpr int LPR = D / 8;              // lanes per token row, 16 bytes each
  constexpr int RPS = kThreads / LPR;     // rows per step
  constexpr int TOK = kSteps * RPS;       // tokens per unit
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ int s_ticket, s_flag;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { s_ticket = atomicAdd(&a.hdr->ticket, 1); s_flag = 0; }
  __syncthreads();
  const int per_w = a.BH * a.n_slices;
  const int w = a.W - 1 - s_ticket / per_w;   // descending windows
  const int r = s_ticket % per_w;
  const int bh = r / a.n_slices, slice = r % a.n_slices;
  const int chunk = tid % LPR, row = tid / LPR;

  // the slice of K and of V, held in registers for both phases
  uint4 kq[kSteps], vq[kSteps];
  bool valid[kSteps];
  const long long row0 = (long long)bh * a.N + a.tok0 + a.S + (long long)w * a.win_stride;
#pragma unroll
  for (int s = 0; s < kSteps; ++s) {
    const int i = slice * TOK + s * RPS + row;
    valid[s] = i < a.L;
    if (valid[s]) {
      const long long off = (row0 + i) * D + chunk * 8;
      kq[s] = __ldcs(reinterpret_cast<const uint4*>(a.K + off));
      vq[s] = __ldcs(reinterpret_cast<const uint4*>(a.V + off));
    } else {
      kq[s] = make_uint4(0, 0, 0, 0);
      vq[s] = make_uint4(0, 0, 0, 0);
    }
  }

  // ---- phase 1: Eq. 4, Eq. 5 (window 0 is never a reference) ----
  if (w >= 1) {
    const uint32_t PINF = 0x7F807F80u, NINF = 0xFF80FF80u;
    uint32_t st[2][2][4];  // [K,V][min,max][4 bf16 pairs]
#pragma unroll
    for (int j = 0; j < 4; ++j) { st[0][0][j] = st[1][0][j] = PINF; st[0][1][j] = st[1][1][j] = NINF; }
#pragma unroll
    for (int s = 0; s < kSteps; ++s) {
      if (!valid[s]) continue;
      const uint32_t kk[4] = {kq[s].x, kq[s].y, kq[s].z, kq[s].w};
      const uint32_t vv[4] = {vq[s].x, vq[s].y, vq[s].z, vq[s].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        st[0][0][j] = bmin2(st[0][0][j], kk[j]); st[0][1][j] = bmax2(st[0][1][j], kk[j]);
        st[1][0][j] = bmin2(st[1][0][j], vv[j]); st[1][1][j] = bmax2(st[1][1][j], vv[j]);
      }
    }
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1)
#pragma unroll
      for (int z = 0; z < 2; ++z)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          st[z][0][j] = bmin2(st[z][0][j], __shfl_xor_sync(0xffffffffu, st[z][0][j], o));
          st[z][1][j] = bmax2(st[z][1][j], __shfl_xor_sync(0xffffffffu, st[z][1][j], o));
        }
    // cross-warp: smem [warp][z*2+stat][D] bf16
    __nv_bfloat16* sm = reinterpret_cast<__nv_bfloat16*>(smem);
    if (lane < LPR) {
#pragma unroll
      for (int z = 0; z < 2; ++z)
#pragma unroll
        for (int m = 0; m < 2; ++m)
          *reinterpret_cast<uint4*>(sm + ((warp * 4 + z * 2 + m) * D + lane * 8)) =
              make_uint4(st[z][m][0], st[z][m][1], st[z][m][2], st[z][m][3]);
    }
    __syncthreads();
    uint32_t* mm = a.mm + (size_t)(bh * a.W + w) * 4 * D;
    for (int v = tid; v < 4 * D; v += kThreads) {
      const int zs = v / D, ch = v % D;
      const bool is_max = zs & 1;
      float acc = __bfloat162float(sm[zs * D + ch]);
#pragma unroll
      for (int ww = 1; ww < kThreads / 32; ++ww) {
        const float x = __bfloat162float(sm[(ww * 4 + zs) * D + ch]);
        acc = is_max ? fmaxf(acc, x) : fminf(acc, x);
      }
      const uint32_t k = order_key(acc);
      atomicMax(mm + v, is_max ? k : ~k);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) atomicAdd(a.ready + bh * a.W + w, 1);
  }
  if (w >= a.Wsel) return;  // the last full window is a reference only

  // ---- phase 2: Eq. 6 and the per-token Std of Eq. 7 ----
  if (tid == 0) {
    const int* flag = a.ready + bh * a.W + w + 1;
    int it = 0;
    while (a.unit_wait_limit < 0 || ld_acquire(flag) < a.n_slices) {
      if (++it > a.unit_wait_limit) { s_flag = 1; atomicExch(&a.hdr->status, (int)LRSA_ERR_TIMEOUT); break; }
      __nanosleep(64);
    }
  }
  __syncthreads();
  if (s_flag) return;
  __threadfence();

  const uint32_t* mm = a.mm + (size_t)(bh * a.W + w + 1) * 4 * D;
  const float inv_dof = 1.0f / (float)(D - a.ddof);
#pragma unroll
  for (int z = 0; z < 2; ++z) {
    // z' = x*sa + sb = zbar - 1/2; a channel with zero range has zbar = 0
    float sa[8], sb[8];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint4 kmn = __ldcg(reinterpret_cast<const uint4*>(mm + (z * 2 + 0) * D + chunk * 8 + h * 4));
      const uint4 kmx = __ldcg(reinterpret_cast<const uint4*>(mm + (z * 2 + 1) * D + chunk * 8 + h * 4));
      const uint32_t a_mn[4] = {kmn.x, kmn.y, kmn.z, kmn.w}, a_mx[4] = {kmx.x, kmx.y, kmx.z, kmx.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float mn = key_to_float(~a_mn[j]), mx = key_to_float(a_mx[j]);
        const float range = mx - mn;
        const float inv = range > 0.f ? 1.0f / range : 0.f;
        sa[h * 4 + j] = inv;
        sb[h * 4 + j] = range > 0.f ? -(0.5f * (mn + mx)) * inv : -0.5f;
      }
    }
    float* out = a.spread + ((size_t)(bh * a.Wsel + w) * 2 + z) * a.L;
#pragma unroll
    for (int s = 0; s < kSteps; ++s) {
      const uint4 q = z == 0 ? kq[s] : vq[s];
      const uint32_t pk[4] = {q.x, q.y, q.z, q.w};
      float sum = 0.f, sq = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float z0 = fmaf(bf_lo(pk[j]), sa[2 * j], sb[2 * j]);
        const float z1 = fmaf(bf_hi(pk[j]), sa[2 * j + 1], sb[2 * j + 1]);
        sum += z0 + z1;
        sq = fmaf(z0, z0, sq);
        sq = fmaf(z1, z1, sq);
      }
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) {
        sum += __shfl_xor_sync(0xffffffffu, sum, o);
        sq += __shfl_xor_sync(0xffffffffu, sq, o);
      }
      if (chunk == 0 && valid[s]) {
        const float var = (sq - sum * sum * (1.0f / D)) * inv_dof;
        out[slice * TOK + s * RPS + row] = sqrtf(fmaxf(var, 0.f));
      }
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_flag = (atomicAdd(a.done + bh * a.Wsel + w, 1) == a.n_slices - 1) ? 2 : 0;
  __syncthreads();
  if (s_flag != 2) return;
  __threadfence();
  select_window(a, bh, w, smem);
}

// ---------------------------------------------------------------------------------------------
// Chain kernel (lag windows up to kChainMaxL tokens): no communication between CTAs at all.
//
// A CTA owns a run of consecutive scored windows [w_a, w_b) of one (batch, KV head) and walks it
// downwards.  It first streams window w_b only for its channel minima and maxima (Eq. 4-5); then for
// w = w_b-1 ... w_a every 16 KB slice of K and of V is normalised with the statistics of window w+1,
// already in shared memory (Eq. 6), reduced to per-token spreads (Eq. 7) that stay in shared memory,
// and folded into the running statistics of window w itself for the next step; at the end of a
// window the CTA soft-maxes, adds (Eq. 8) and selects.  A producer warp keeps a ring of slices in
// flight with bulk asynchronous copies, so the loads never wait for the arithmetic; two groups of
// eight scoring warps take alternate slices (the arithmetic of one slice is a chain of dependent
// shuffles and reductions, and one group alone leaves the SM idle most of the time).  Each group has
// its own ring of stages and waits for its slices in the order they were issued: a barrier is then
// never waited on two phases ahead (a parity wait cannot tell "two phases ahead" from "done"), which
// a shared ring allowed when one group ran ahead and bulk copies landed out of order.
// With one window per CTA (the 32K benchmark: 120 windows on 148 SMs) every window is streamed
// twice, by its own CTA and as the reference of the window before it; the second read comes a few
// microseconds after the first and is served by L2 as long as K and V fit there (67 MB of 126 MB).
// Longer runs per CTA (more windows than SMs) read 1 + 1/run of the data.
constexpr int kChainMaxRing = 3;   // stages per scoring group (2 when the selection scratch is large)
constexpr int kChainMaxL = 4096;
constexpr int kChainGroups = 2;                           // scoring groups of kThreads threads, alternating slices
constexpr int kChainThreads = kChainGroups * kThreads + 32;

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void all_groups_sync() {
  asm volatile("bar.sync 3, %0;" ::"n"(kChainGroups * kThreads) : "memory");
}
// Barriers that also OR a predicate over their threads: every thread leaves with the same verdict, so a
// group (or the whole CTA) takes the give-up branch together even if the flag was raised while some of
// its threads had already looked at it.
__device__ __forceinline__ bool bar_or(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ bool group_sync_or(int grp, bool pred) { return bar_or(grp + 1, kThreads, pred); }
__device__ __forceinline__ bool all_groups_sync_or(bool pred) { return bar_or(3, kChainGroups * kThreads, pred); }

// Bounded wait on a shared-memory barrier phase; false when it gave up.
__device__ __forceinline__ bool stage_wait(uint32_t bar, uint32_t parity, int limit) {
  for (int it = 0; it < limit; ++it)
    if (ptx::mbar_try_wait(bar, parity)) return true;
  return false;
}

template <int D>
__global__ void __launch_bounds__(kChainThreads, 1) score_select_chain_kernel(const ScoreArgs a, int run, int runs_per_bh,
                                                                              int ring) {
  constexpr int LPR = D / 8;              // lanes per token row, 16 bytes each
  constexpr int RPS = kThreads / LPR;     // rows per step
  constexpr int TOK = kSteps * RPS;       // tokens per slice
  constexpr int kSliceBytes = TOK * D * 2;
  constexpr int kStageBytes = 2 * kSliceBytes;   // K slice, then V slice
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ __align__(8) uint64_t full_bar[kChainGroups * kChainMaxRing], empty_bar[kChainGroups * kChainMaxRing];
  __shared__ int s_abort;
  // after the ring: scale/offset of the reference window [2 (K,V)][2 (sa,sb)][D], then the selection
  // scratch (spreads sk[L], sv[L], histogram...), whose tail doubles as the min/max reduction buffer
  float* sasb = reinterpret_cast<float*>(smem + kChainGroups * ring * kStageBytes);
  unsigned char* sel = reinterpret_cast<unsigned char*>(sasb + 4 * D);
  float* sk = reinterpret_cast<float*>(sel);
  float* sv = sk + a.L;
  __nv_bfloat16* red = reinterpret_cast<__nv_bfloat16*>(sel + select_scratch_bytes(a.L));   // [16 warps][4][D]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // A bounded wait needs seconds to expire, the first CTA of the grid starts with the launch: its clearing
  // of the status word cannot overwrite another CTA's verdict.
  if (a.clear_status && blockIdx.x == 0 && tid == 0) a.hdr->status = 0;
  if (tid == 0) {
    s_abort = 0;
    for (int i = 0; i < kChainGroups * kChainMaxRing; ++i) {
      ptx::mbar_init(ptx::smem_u32(&full_bar[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&empty_bar[i]), 1);
    }
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int bh = blockIdx.x / runs_per_bh, seg = blockIdx.x % runs_per_bh;
  const int w_a = seg * run, w_b = min(a.Wsel, w_a + run);   // scored windows [w_a, w_b); reference w_b <= W-1
  const int n_win = w_b - w_a + 1;                            // windows streamed, the reference first
  const int n_it = n_win * a.n_slices;
  volatile int* abort = &s_abort;

  if (warp == kChainGroups * kThreads / 32) {
    // ---------------- producer ----------------
    if (lane != 0) return;
    // slice i goes to group i % 2; it is that group's k-th slice and uses slot k % ring of its ring in
    // that slot's (k / ring)-th use.  All counters advance without divisions: one thread feeds the SM.
    static_assert(kChainGroups == 2, "slot bookkeeping below");
    int kr[2] = {0, 0}, use[2] = {0, 0};   // per group: k % ring and k / ring of its next slice
    int w = w_b, slice = 0;
    for (int i = 0; i < n_it; ++i) {
      const int g = i & 1, slot = g * ring + kr[g];
      if (use[g] > 0 && !stage_wait(ptx::smem_u32(&empty_bar[slot]), (use[g] - 1) & 1, a.spin_limit)) {
        *abort = 1;
        atomicExch(&a.hdr->status, (int)LRSA_ERR_TIMEOUT);
        break;
      }
      if (*abort) break;
      const int rows = min(TOK, a.L - slice * TOK);
      const uint32_t bytes = (uint32_t)rows * D * 2;
      const long long off = ((long long)bh * a.N + a.tok0 + a.S + (long long)w * a.win_stride + (long long)slice * TOK) * D;
      const uint32_t bar = ptx::smem_u32(&full_bar[slot]);
      const uint32_t dst = ptx::smem_u32(smem + slot * kStageBytes);
      // self-check: the slice lies inside the tensor and the copy is 16-byte granular; otherwise give up
      // (status word) instead of issuing it
      if (w < 0 || w >= a.W || rows <= 0 || off < 0 || off + (long long)rows * D > a.elems || (bytes & 15u) ||
          ((reinterpret_cast<uintptr_t>(a.K + off) | reinterpret_cast<uintptr_t>(a.V + off) | dst) & 15u)) {
        *abort = 1;
        atomicExch(&a.hdr->status, (int)LRSA_ERR_TIMEOUT);
        break;
      }
      ptx::mbar_expect_tx(bar, 2 * bytes);
      bulk_load(dst, a.K + off, bytes, bar);
      bulk_load(dst + kSliceBytes, a.V + off, bytes, bar);
      if (++kr[g] == ring) { kr[g] = 0; ++use[g]; }
      if (++slice == a.n_slices) { slice = 0; --w; }
    }
    // No copy may be in flight when the CTA's shared memory is released, whether the run completed or a
    // wait gave up: the producer leaves last, after the latest copy into every slot has landed (bounded).
    for (int g = 0; g < kChainGroups; ++g)
      for (int r = 0; r < ring; ++r) {
        const int u = r < kr[g] ? use[g] : use[g] - 1;   // latest use of the slot that was issued
        if (u >= 0) (void)stage_wait(ptx::smem_u32(&full_bar[g * ring + r]), u & 1, a.spin_limit);
      }
    return;
  }

  // ---------------- scoring warps ----------------
  const int grp = tid / kThreads, gt = tid % kThreads;   // group and thread within the group
  const int chunk = gt % LPR, row = gt / LPR;
  const float inv_dof = 1.0f / (float)(D - a.ddof);
  const uint32_t PINF = 0x7F807F80u, NINF = 0xFF80FF80u;
  uint32_t st[2][2][4];  // running [K,V][min,max][4 bf16 pairs] of this group's slices of the window
  int it_all = 0, ckr = 0, cuse = 0;   // slices streamed so far by both groups; this group's ring position
  for (int wi = 0; wi < n_win; ++wi) {
   const int w = w_b - wi;
   const bool scoring = wi > 0;          // the first window streamed is a reference only
   const bool want_stats = w > w_a;      // its statistics serve the next window of the run
   // scale and offset (Eq. 6) of this thread's eight channels, as packed pairs: [tensor][sa, sb][pair]
   uint64_t sab2[2][2][4];
   if (scoring) {
#pragma unroll
     for (int z = 0; z < 2; ++z)
#pragma unroll
       for (int m = 0; m < 2; ++m)
#pragma unroll
         for (int h = 0; h < 2; ++h) {
           const float4 v = *reinterpret_cast<const float4*>(sasb + (z * 2 + m) * D + chunk * 8 + h * 4);
           sab2[z][m][2 * h] = ptx::f2_pack(v.x, v.y);
           sab2[z][m][2 * h + 1] = ptx::f2_pack(v.z, v.w);
         }
   } else {
#pragma unroll
     for (int z = 0; z < 2; ++z)
#pragma unroll
       for (int m = 0; m < 2; ++m)
#pragma unroll
         for (int j = 0; j < 4; ++j) sab2[z][m][j] = 0ull;
   }
#pragma unroll
   for (int j = 0; j < 4; ++j) { st[0][0][j] = st[1][0][j] = PINF; st[0][1][j] = st[1][1][j] = NINF; }
   for (int slice = 0; slice < a.n_slices; ++slice, ++it_all) {
    if ((it_all & 1) != grp) continue;
    const int slot = grp * ring + ckr;   // this group's slice number k: ckr = k % ring, cuse = k / ring
    // One barrier per slice: a warp whose wait ran out skips the arithmetic (warp-uniform, the
    // arithmetic shuffles), raises the flag and still meets the group at the barrier below, after
    // which every thread of the group reads the same verdict.
    bool got = stage_wait(ptx::smem_u32(&full_bar[slot]), cuse & 1, a.spin_limit);
    got = __all_sync(0xffffffffu, got);
    if (!got) {
      *abort = 1;
      atomicExch(&a.hdr->status, (int)LRSA_ERR_TIMEOUT);
    }
    if (__all_sync(0xffffffffu, got && !*abort)) {
    const unsigned char* stage = smem + slot * kStageBytes;
    // this thread's rows of the slice: kSteps rows of K and of V, 16 bytes (8 channels) each
    uint4 kq[kSteps], vq[kSteps];
    bool valid[kSteps];
#pragma unroll
    for (int s = 0; s < kSteps; ++s) {
      const int t = s * RPS + row;
      valid[s] = slice * TOK + t < a.L;
      if (valid[s]) {
        kq[s] = *reinterpret_cast<const uint4*>(stage + (size_t)t * D * 2 + chunk * 16);
        vq[s] = *reinterpret_cast<const uint4*>(stage + kSliceBytes + (size_t)t * D * 2 + chunk * 16);
      } else {
        kq[s] = make_uint4(0, 0, 0, 0);
        vq[s] = make_uint4(0, 0, 0, 0);
      }
    }
    if (want_stats) {
      // Eq. 4, Eq. 5, folded into the running statistics
#pragma unroll
      for (int s = 0; s < kSteps; ++s) {
        if (!valid[s]) continue;
        const uint32_t kk[4] = {kq[s].x, kq[s].y, kq[s].z, kq[s].w}, vv[4] = {vq[s].x, vq[s].y, vq[s].z, vq[s].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          st[0][0][j] = bmin2(st[0][0][j], kk[j]); st[0][1][j] = bmax2(st[0][1][j], kk[j]);
          st[1][0][j] = bmin2(st[1][0][j], vv[j]); st[1][1][j] = bmax2(st[1][1][j], vv[j]);
        }
      }
    }
    if (scoring) {
      // Eq. 6 with the statistics of window w+1 (z' = x*sa + sb = zbar - 1/2) and the per-token Std of
      // Eq. 7.  Arithmetic on packed fp32 pairs; sa/sb of this thread's eight channels live in registers
      // for the whole window (sab2, loaded below the window loop's head).
      float part[2 * kSteps][2];   // [tensor * kSteps + step][sum, sum of squares] over this thread's 8 channels
#pragma unroll
      for (int z = 0; z < 2; ++z) {
#pragma unroll
        for (int s = 0; s < kSteps; ++s) {
          const uint4 q = z == 0 ? kq[s] : vq[s];
          const uint32_t pk[4] = {q.x, q.y, q.z, q.w};
          uint64_t sum2 = 0ull, sq2 = 0ull;   // (+0, +0)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint64_t z2 = ptx::f2_fma(ptx::f2_pack(bf_lo(pk[j]), bf_hi(pk[j])), sab2[z][0][j], sab2[z][1][j]);
            sum2 = ptx::f2_add(sum2, z2);
            sq2 = ptx::f2_fma(z2, z2, sq2);
          }
          float s0, s1, q0, q1;
          ptx::f2_unpack(sum2, s0, s1);
          ptx::f2_unpack(sq2, q0, q1);
          part[z * kSteps + s][0] = s0 + s1;
          part[z * kSteps + s][1] = q0 + q1;
        }
      }
      // Sum over the LPR lanes of a row.  Halving exchange: at every level a lane keeps half of its
      // entries and hands the other half to its partner, so 2*kSteps entries cost 2*(2*kSteps - 1)
      // shuffles instead of 2*kSteps*log2(LPR)*2; levels left over once one entry remains are plain
      // butterflies.  The lane ends with entry e(chunk) complete.
      int ent = 0;   // index of the entry this lane ends up with
      {
        int m = 2 * kSteps;   // entries still held
#pragma unroll
        for (int bit = LPR / 2; bit >= 1; bit >>= 1) {
          if (m > 1) {
            m >>= 1;
            const bool up = (chunk & bit) != 0;
#pragma unroll
            for (int e = 0; e < kSteps; ++e) {   // kSteps >= m at every level
              if (e < m) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                  const float send = up ? part[e][c] : part[e + m][c];
                  const float keep = up ? part[e + m][c] : part[e][c];
                  part[e][c] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
                }
              }
            }
            ent += up ? m : 0;
          } else {
            part[0][0] += __shfl_xor_sync(0xffffffffu, part[0][0], bit);
            part[0][1] += __shfl_xor_sync(0xffffffffu, part[0][1], bit);
          }
        }
      }
      {
        const int z = ent / kSteps, st_ = ent % kSteps;
        // lanes that differ only in the bits of the plain butterfly levels hold the same entry: one writes
        constexpr int kDup = LPR / (2 * kSteps) > 1 ? LPR / (2 * kSteps) : 1;
        const bool writer = (chunk & (kDup - 1)) == 0;
        const int tkn = slice * TOK + st_ * RPS + row;
        if (writer && tkn < a.L) {
          const float var = (part[0][1] - part[0][0] * part[0][0] * (1.0f / D)) * inv_dof;
          (z == 0 ? sk : sv)[tkn] = sqrtf(fmaxf(var, 0.f));
        }
      }
    }
    }
    // every read of the stage by this group is done; one verdict for the group
    if (group_sync_or(grp, *abort != 0)) break;
    if (gt == 0) ptx::mbar_arrive(ptx::smem_u32(&empty_bar[slot]));
    if (++ckr == ring) { ckr = 0; ++cuse; }
   }

   // ---- end of window w: both groups have written their spreads and hold their part of the statistics ----
   if (all_groups_sync_or(*abort != 0)) return;   // one verdict for the CTA
   if (scoring && grp == 0) select_window(a, bh, w, sel, true);   // group 0 only (its own barrier inside)
   if (want_stats) {
      // reduce the running statistics over the rows of a warp, then over the warps, and turn them
      // into the scale and offset the next window is normalised with
#pragma unroll
      for (int o = 16; o >= LPR; o >>= 1)
#pragma unroll
        for (int z = 0; z < 2; ++z)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            st[z][0][j] = bmin2(st[z][0][j], __shfl_xor_sync(0xffffffffu, st[z][0][j], o));
            st[z][1][j] = bmax2(st[z][1][j], __shfl_xor_sync(0xffffffffu, st[z][1][j], o));
          }
      if (lane < LPR) {
#pragma unroll
        for (int z = 0; z < 2; ++z)
#pragma unroll
          for (int m = 0; m < 2; ++m)
            *reinterpret_cast<uint4*>(red + ((warp * 4 + z * 2 + m) * D + lane * 8)) =
                make_uint4(st[z][m][0], st[z][m][1], st[z][m][2], st[z][m][3]);
      }
      all_groups_sync();
      for (int v = tid; v < 2 * D; v += kChainGroups * kThreads) {
        const int z = v / D, ch = v % D;
        float mn = __bfloat162float(red[(z * 2 + 0) * D + ch]), mx = __bfloat162float(red[(z * 2 + 1) * D + ch]);
#pragma unroll
        for (int ww = 1; ww < kChainGroups * kThreads / 32; ++ww) {
          mn = fminf(mn, __bfloat162float(red[(ww * 4 + z * 2 + 0) * D + ch]));
          mx = fmaxf(mx, __bfloat162float(red[(ww * 4 + z * 2 + 1) * D + ch]));
        }
        // a channel with zero range has zbar = 0, i.e. z' = -1/2
        const float range = mx - mn;
        const float inv = range > 0.f ? 1.0f / range : 0.f;
        sasb[(z * 2 + 0) * D + ch] = inv;
        sasb[(z * 2 + 1) * D + ch] = range > 0.f ? -(0.5f * (mn + mx)) * inv : -0.5f;
      }
   }
   all_groups_sync();   // the next window's slices may overwrite the spreads and read the new statistics
  }
}

template <int D>
constexpr int tok_per_unit() { return kSteps * (kThreads / (D / 8)); }

size_t select_smem_bytes(int L, int d) {
  const size_t phase1 = (size_t)(kThreads / 32) * 4 * d * sizeof(__nv_bfloat16);
  const size_t sel = (size_t)2 * L * sizeof(float) + 256 * 4 + 32 * 4 + 16 * 4;
  return phase1 > sel ? phase1 : sel;
}

// Polls the one-slice-per-CTA kernel grants its wait for the following window's statistics.  Test hook:
// a negative value makes that wait give up at once (the kernel holds its slice in registers and has no
// copy in flight, so every thread returns after the verdict).  The chain kernel's limits are not touched.
int g_unit_wait_limit = 1 << 21;

struct ScoreWs {
  size_t ready, done, mm, zero_bytes, spread, total;
};
ScoreWs score_ws_layout(const Geom& g) {
  ScoreWs w;
  const size_t BH = (size_t)g.B * g.Hkv;
  size_t off = sizeof(WsHeader);
  w.ready = off; off += align_up(BH * g.W * sizeof(int), 16);
  w.done = off;  off += align_up(BH * g.Wsel * sizeof(int), 16);
  w.mm = off;    off += align_up(BH * g.W * 4 * g.d * sizeof(uint32_t), 256);
  w.zero_bytes = off;   // everything up to here is cleared before the launch
  w.spread = off; off += align_up(BH * g.Wsel * 2 * g.L * sizeof(float), 256);
  w.total = off;
  return w;
}

}  // namespace

// The chain kernel uses nothing but the status header; the one-slice-per-CTA kernel needs its counters,
// statistics and spreads.
size_t score_select_ws_bytes(const Geom& g) { return g.L <= kChainMaxL ? sizeof(WsHeader) : score_ws_layout(g).total; }

void set_unit_wait_limit(int polls) { g_unit_wait_limit = polls; }

bool score_select_clears_status(const Geom& g) { return g.Wsel > 0 && g.L <= kChainMaxL; }

int launch_score_select(const Geom& g, const __nv_bfloat16* K, const __nv_bfloat16* V, int32_t* idx,
                        float* score, void* ws, cudaStream_t st, bool clear_status) {
  if (g.Wsel == 0) return LRSA_OK;  // nothing is scored
  const ScoreWs lay = score_ws_layout(g);
  unsigned char* base = static_cast<unsigned char*>(ws);
  // The status word (the header) is cleared once per call by the caller.  The chain kernel keeps everything
  // else on chip; the one-slice-per-CTA kernel needs its ticket, counters and statistics at zero.
  if (g.L > kChainMaxL) {
    LRSA_CUDA_CHECK(cudaMemsetAsync(base + offsetof(WsHeader, ticket), 0, lay.zero_bytes - offsetof(WsHeader, ticket), st));
    launch_counter().n++;
  }
  ScoreArgs a;
  a.K = K; a.V = V; a.idx = idx; a.score = score;
  a.hdr = reinterpret_cast<WsHeader*>(base);
  a.ready = reinterpret_cast<int*>(base + lay.ready);
  a.done = reinterpret_cast<int*>(base + lay.done);
  a.mm = reinterpret_cast<uint32_t*>(base + lay.mm);
  a.spread = reinterpret_cast<float*>(base + lay.spread);
  a.BH = g.B * g.Hkv; a.N = g.Nrow; a.L = g.L; a.Kk = g.K; a.S = g.S; a.W = g.W; a.Wsel = g.Wsel;
  a.tok0 = g.tok0; a.Wtot = g.Wtot; a.woff = g.woff; a.emit_off = g.emit_off; a.win_stride = g.win_stride;
  a.elems = (long long)g.B * g.Hkv * g.Nrow * g.d;
  a.ddof = g.ddof;
  a.clear_status = clear_status && score_select_clears_status(g) ? 1 : 0;
  a.spin_limit = 1 << 21;
  a.unit_wait_limit = g_unit_wait_limit;
  const int tok = g.d == 128 ? tok_per_unit<128>() : tok_per_unit<64>();
  a.n_slices = (g.L + tok - 1) / tok;
  const size_t smem = select_smem_bytes(g.L, g.d);
  if (smem > 200 * 1024) return LRSA_ERR_UNSUPPORTED;
  const long long units = (long long)a.BH * g.W * a.n_slices;
  if (units > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  if (g.L <= kChainMaxL) {
    // chain kernel: runs of consecutive windows per CTA, about one CTA per SM, no inter-CTA traffic
    int dev = 0, sms = 0;
    LRSA_CUDA_CHECK(cudaGetDevice(&dev));
    LRSA_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int run = (a.BH * g.Wsel + sms - 1) / sms;
    const int runs_per_bh = (g.Wsel + run - 1) / run;
    const size_t stage = (size_t)2 * tok * g.d * sizeof(__nv_bfloat16);
    const size_t rest = (size_t)4 * g.d * sizeof(float) + select_scratch_bytes(g.L) +
                        (size_t)(kChainGroups * kThreads / 32) * 4 * g.d * sizeof(__nv_bfloat16);
    const int ring = kChainGroups * kChainMaxRing * stage + rest <= 220 * 1024 ? kChainMaxRing : 2;
    const size_t bytes = (size_t)kChainGroups * ring * stage                             // rings
                         + (size_t)4 * g.d * sizeof(float)                               // scale / offset
                         + select_scratch_bytes(g.L)
                         + (size_t)(kChainGroups * kThreads / 32) * 4 * g.d * sizeof(__nv_bfloat16);   // min/max reduction
    auto ckern = g.d == 128 ? score_select_chain_kernel<128> : score_select_chain_kernel<64>;
    LRSA_CUDA_CHECK(cudaFuncSetAttribute(ckern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    ckern<<<(unsigned)(a.BH * runs_per_bh), kChainThreads, bytes, st>>>(a, run, runs_per_bh, ring);
    LRSA_CUDA_CHECK(cudaGetLastError());
    launch_counter().n++;
    return LRSA_OK;
  }
  auto kern = g.d == 128 ? score_select_kernel<128> : score_select_kernel<64>;
  LRSA_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(unsigned)units, kThreads, smem, st>>>(a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

}  // namespace lrsa
