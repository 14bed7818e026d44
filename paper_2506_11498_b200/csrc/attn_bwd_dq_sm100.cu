// LRSA attention backward, dQ part, on tcgen05 tensor cores.
//
// A CTA owns one 128-row query tile of one (batch, query head) and walks its key list (the same
// row-block decomposition as the forward) in 64-key tiles.  Q and dO are copied once into tensor
// memory, so every product takes its 128-row operand from TMEM and only the K_j / V_j tiles from
// shared memory (with both operands in shared memory the kernel is bound by shared-memory
// bandwidth, not by the tensor core).  Per key tile j:
//   S  = Q K_j^T          (TMEM x smem -> TMEM)      P  = exp2(S*c - LSE*log2e)
//   dP = dO V_j^T         (TMEM x smem -> TMEM)      dS = P * (dP - D)          (bf16, back into TMEM)
//   A += dS K_j           (TMEM x smem -> TMEM)      epilogue: dQ = scale * (A - r * kbar) -> bf16
// S/dP are double-buffered in TMEM, so the tensor core computes tile j+1 while tile j is in the
// softmax; both softmax warpgroups work on every tile (32 key columns each) to keep the latency
// between "S ready" and "dS ready" short.  Warps: 0 TMA producer, 1-3 tensor-core issuers (S, dP, A;
// no warp has more than eight tcgen05.mma per tile to issue), 4-11 softmax and epilogue.
//
// D_t = sum_j P_tj dP_tj comes from the dK/dV kernel, which runs first and accumulates it in fp32
// (rowsum(dO * O) of the bf16 O is not accurate enough: its error is multiplied by the
// softmax-averaged key, which is large when a few salient keys dominate a row).
// Rows of the exact dS sum to zero; after bf16 rounding they sum to r_t, which multiplies whatever
// constant vector the keys of a head share (outlier channels).  The epilogue subtracts r_t * kbar,
// kbar the mean key of the KV head; in exact arithmetic this subtracts zero.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

using namespace ptx;

constexpr int kKeys = 64;   // keys per tile in this kernel

template <int D>
struct DqCfg {
  static constexpr int kSub = D / 64;
  static constexpr int kQSubBytes = kTile * 128;           // 128 query rows x 128 bytes
  static constexpr int kQTileBytes = kSub * kQSubBytes;    // the Q or the dO tile
  static constexpr int kKSubBytes = kKeys * 128;           // 64 key rows x 128 bytes
  static constexpr int kKTileBytes = kSub * kKSubBytes;    // one K or V tile
  static constexpr int kStages = D == 128 ? 9 : 16;        // ring slots, K and V tiles alternate
  static constexpr int kSmem = 2 * kQTileBytes + kStages * kKTileBytes + 1024;
  static constexpr int kThreads = 384;
  // TMEM columns: Q and dO as packed bf16 (D/2 columns each), accumulator A at D, then buffer b with
  // S at 256 + 128b and dP 64 columns further
  static constexpr uint32_t kColQ = 0, kColdO = D / 2, kColA = D, kColBuf = 256, kColP = 64;
};

struct DqArgs {
  BlockPlan plan;
  int BH, Hq, Hkv, G, N;   // N: tokens per (batch, head) row of stats, Dacc and dQ (the row stride)
  const float2* stats;   // per query row: (-LSE*log2e, D~); only the first component is used here
  const float* Dacc;     // per query row: D = sum_j P dP
  const float* kbar;     // [B*Hkv][D] mean key
  __nv_bfloat16* dQ;
  float scale, scale_log2;
  int* status;
};

struct DqBars {
  uint64_t q_full, qt_ready, acc_done;
  uint64_t kv_full[16], kv_empty[16];
  uint64_t s_full[2], p_full[2], buf_free[2];
};

template <int D>
__global__ void __launch_bounds__(DqCfg<D>::kThreads, 1)
lrsa_bwd_dq_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
                   const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                   const __grid_constant__ CUtensorMap mapKc, const __grid_constant__ CUtensorMap mapVc,
                   const DqArgs a) {
  using Cfg = DqCfg<D>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) DqBars bars;
  __shared__ float red_s[2][kTile];   // [column half][row] sums of the rounded dS
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0, sdO = smem0 + Cfg::kQTileBytes, sRing = smem0 + 2 * Cfg::kQTileBytes;

  const int bh = blockIdx.x % a.BH, blk = blockIdx.x / a.BH;
  const RowBlock rb = decode_block(a.plan, blk);
  const int bh_kv = (bh / a.Hq) * a.Hkv + (bh % a.Hq) / a.G;
  const int n_ct = (rb.n_front + kKeys - 1) / kKeys;
  const int n = n_ct + (rb.q_end - 1 - rb.dense_start) / kKeys + 1;   // key tiles of this block (>= 1)

  if (tid == 0) {
    abort_s = 0;
    mbar_init(smem_u32(&bars.q_full), 1);
    mbar_init(smem_u32(&bars.qt_ready), 256);
    mbar_init(smem_u32(&bars.acc_done), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.s_full[b]), 2);      // the S issuer and the dP issuer
      mbar_init(smem_u32(&bars.p_full[b]), 256);    // every softmax thread
      mbar_init(smem_u32(&bars.buf_free[b]), 1);
    }
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_s), 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_base_s;
  volatile int* abort = &abort_s;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapQ); prefetch_tensormap(&mapdO); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
      prefetch_tensormap(&mapKc); prefetch_tensormap(&mapVc);
      mbar_expect_tx(smem_u32(&bars.q_full), 2 * Cfg::kQTileBytes);
      for (int h = 0; h < Cfg::kSub; ++h) {
        tma_load_3d(sQ + h * Cfg::kQSubBytes, &mapQ, h * 64, rb.q0, bh, smem_u32(&bars.q_full));
        tma_load_3d(sdO + h * Cfg::kQSubBytes, &mapdO, h * 64, rb.q0, bh, smem_u32(&bars.q_full));
      }
      int it = 0;
      bool ok = true;
      for (int j = 0; j < n && ok; ++j) {
        for (int which = 0; which < 2 && ok; ++which, ++it) {
          const int slot = it % NS, use = it / NS;
          if (use > 0) ok = mbar_wait(smem_u32(&bars.kv_empty[slot]), (use - 1) & 1, abort);
          if (!ok) break;
          const uint32_t full = smem_u32(&bars.kv_full[slot]);
          mbar_expect_tx(full, Cfg::kKTileBytes);
          const bool compact = j < n_ct;
          const CUtensorMap* map = compact ? (which ? &mapVc : &mapKc) : (which ? &mapV : &mapK);
          const int row = compact ? j * kKeys : rb.dense_start + (j - n_ct) * kKeys;
          for (int h = 0; h < Cfg::kSub; ++h)
            tma_load_3d(sRing + slot * Cfg::kKTileBytes + h * Cfg::kKSubBytes, map, h * 64, row, bh_kv, full);
        }
      }
      if (!ok) {
        // give loads already in flight a bounded chance to land before the CTA's smem is released
        for (int back = 1; back <= NS && back <= it; ++back) {
          const int i2 = it - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&bars.kv_full[i2 % NS]), (i2 / NS) & 1) && clock64() - t0 < 2000000) {}
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ---------------- S issuer (warp 1: Q K_j^T) and dP issuer (warp 2: dO V_j^T) ----------------
    // Each issuing warp runs its loop with all lanes (uniform control flow, descriptors computed once)
    // and elects one lane per instruction.
    const int which = warp - 1;                                          // 0: K tiles, 1: V tiles
    constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kKeys, 0, 0);   // 128 x 64
    const uint64_t descR = make_smem_desc_sw128(sRing, 16, 1024);       // K-major K_j / V_j
    const uint32_t a_tmem = tmem + (which == 0 ? Cfg::kColQ : Cfg::kColdO);
    bool ok = mbar_wait_warp(smem_u32(&bars.qt_ready), 0, abort);   // Q and dO are in tensor memory
    for (int j = 0; j < n && ok; ++j) {
      const int it = 2 * j + which, b = j & 1;   // ring order: K_j at 2j, V_j at 2j+1
      ok = mbar_wait_warp(smem_u32(&bars.kv_full[it % NS]), (it / NS) & 1, abort);
      if (ok && j >= 2) ok = mbar_wait_warp(smem_u32(&bars.buf_free[b]), ((j >> 1) - 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem + Cfg::kColBuf + b * 128 + which * Cfg::kColP;
      const uint64_t dT = desc_advance(descR, (it % NS) * Cfg::kKTileBytes);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint64_t bd = desc_advance(dT, (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32);
        if (elect_one()) umma_ts(d_tmem, a_tmem + kk * 8, bd, idesc_s, kk > 0 ? 1u : 0u);
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bars.s_full[b]));
        if (which == 1) umma_commit(smem_u32(&bars.kv_empty[it % NS]));   // V_j is used by dP only
      }
      __syncwarp();
    }
  } else if (warp == 3) {
    // ---------------- A issuer: A += dS K_j ----------------
    constexpr uint32_t idesc_a = make_idesc_bf16(kTile, D, 0, 1);                  // 128 x D, B = K_j MN-major
    const uint64_t descRmn = make_smem_desc_sw128(sRing, Cfg::kKSubBytes, 1024);
    bool ok = true;
    for (int j = 0; j < n && ok; ++j) {
      const int b = j & 1, itK = 2 * j;
      const uint32_t buf = tmem + Cfg::kColBuf + b * 128;
      ok = mbar_wait_warp(smem_u32(&bars.p_full[b]), (j >> 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t dKj = desc_advance(descRmn, (itK % NS) * Cfg::kKTileBytes);
      const uint32_t acc0 = j > 0 ? 1u : 0u;
      // packed dS: keys [0,32) in columns [0,16) of the S region, keys [32,64) in columns [32,48)
#pragma unroll
      for (int kk = 0; kk < kKeys / 16; ++kk) {
        const uint64_t bd = desc_advance(dKj, kk * 2048);
        if (elect_one()) umma_ts(tmem + Cfg::kColA, buf + (kk >> 1) * 32 + (kk & 1) * 8, bd, idesc_a, kk > 0 ? 1u : acc0);
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bars.kv_empty[itK % NS]));   // K_j: S (before the softmax) and A are done
        umma_commit(smem_u32(&bars.buf_free[b]));          // tile j+2 may overwrite the buffer
      }
      __syncwarp();
    }
    if (ok && elect_one()) umma_commit(smem_u32(&bars.acc_done));
    __syncwarp();
  } else {
    // ---------------- softmax warps: warpgroup `half` takes key columns [32*half, 32*half+32) ----------------
    const int half = (warp - 4) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int qpos = rb.q0 + row;
    const bool live = qpos < rb.q_end;
    const float c = a.scale_log2;
    // rows outside the block get lse = +inf so that P = 0
    const float nl2 = live ? a.stats[(size_t)bh * a.N + qpos].x : -INFINITY;
    const float Dt = live ? a.Dacc[(size_t)bh * a.N + qpos] : 0.f;
    float rsum = 0.f;
    // copy this thread's row of Q (warpgroup 0) or dO (warpgroup 1) from the swizzled shared-memory
    // tile into tensor memory: 16-byte chunk c of row r of a 64-column sub-tile sits at chunk c ^ (r & 7)
    bool ok = mbar_wait(smem_u32(&bars.q_full), 0, abort);
    if (ok) {
      const unsigned char* src = smem_raw + ((half == 0 ? sQ : sdO) - smem_u32(smem_raw)) + row * 128;
      const uint32_t dst = tmem + lane_addr + (half == 0 ? Cfg::kColQ : Cfg::kColdO);
#pragma unroll
      for (int h = 0; h < Cfg::kSub; ++h) {
        uint32_t v[32];
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          const uint4 x = *reinterpret_cast<const uint4*>(src + h * Cfg::kQSubBytes + ((ch ^ (row & 7)) << 4));
          v[4 * ch] = x.x; v[4 * ch + 1] = x.y; v[4 * ch + 2] = x.z; v[4 * ch + 3] = x.w;
        }
        tmem_st32(dst + h * 32, v);
      }
      tmem_wait_st();
    }
    tc_fence_before_sync();
    mbar_arrive(smem_u32(&bars.qt_ready));   // also when the wait gave up: the issuers then see abort
    for (int j = 0; j < n && ok; ++j) {
      const int b = j & 1;
      ok = mbar_wait(smem_u32(&bars.s_full[b]), (j >> 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t S_addr = tmem + lane_addr + Cfg::kColBuf + b * 128 + half * 32;
      uint32_t s[32], dp[32];
      tmem_ld32(S_addr, s);
      tmem_ld32(S_addr + Cfg::kColP, dp);
      tmem_wait_ld();
      const int limit = (j < n_ct ? rb.n_front - j * kKeys : qpos - (rb.dense_start + (j - n_ct) * kKeys) + 1) - half * 32;
      if (limit < 32) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i >= limit) s[i] = 0xff800000u;
      }
      uint32_t ds[16];
      float r0, r1;
      {
        // packed fp32 pairs: one issue slot for two elements of the scale-and-shift, of dP - D, of the
        // product and of the row sum of the rounded dS
        const uint64_t c2 = f2_pack(c, c), nl22 = f2_pack(nl2, nl2), nD2 = f2_pack(-Dt, -Dt);
        uint64_t r2 = f2_pack(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float x0, x1, d0, d1;
          f2_unpack(f2_fma(f2_pack(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, nl22), x0, x1);
          const float p0 = ex2(x0), p1 = ex2(x1);
          const uint64_t g2 = f2_add(f2_pack(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])), nD2);
          f2_unpack(f2_mul(f2_pack(p0, p1), g2), d0, d1);
          ds[i] = pack_bf16(d0, d1);
          r2 = f2_add(r2, f2_pack(__uint_as_float(ds[i] << 16), __uint_as_float(ds[i] & 0xffff0000u)));
        }
        f2_unpack(r2, r0, r1);
      }
      rsum += r0 + r1;
      tmem_st16(S_addr, ds);   // over the first half of this warpgroup's own S columns
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[b]));
    }
    red_s[half][row] = rsum;
    asm volatile("bar.sync 1, 256;" ::: "memory");   // the eight softmax warps, whether or not a wait gave up
    if (ok) ok = mbar_wait(smem_u32(&bars.acc_done), 0, abort);
    // The dQ rows go through shared memory (the Q and dO tiles are idle since their copy into tensor
    // memory) and leave as one bulk copy per row: per-thread 16-byte stores to rows 256 bytes apart cost
    // a transaction each.  Rows are padded by 16 bytes so that a warp's stores spread over the banks.
    constexpr int kRowBytes = D * 2, kStageStride = kRowBytes + 16;
    unsigned char* stage_out = smem_raw + (sQ - smem_u32(smem_raw));
    if (ok) {
      tc_fence_after_sync();
      const float r = red_s[0][row] + red_s[1][row];
      constexpr int CH = D / 2;   // output columns of this warpgroup
      const uint32_t A_addr = tmem + lane_addr + Cfg::kColA + half * CH;
      const float* kb = a.kbar + (size_t)bh_kv * D + half * CH;
      unsigned char* srow = stage_out + row * kStageStride + half * (kRowBytes / 2);
#pragma unroll
      for (int q = 0; q < CH / 32; ++q) {
        uint32_t o[32];
        tmem_ld32(A_addr + q * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e)
            f[e] = fmaf(-r, __ldg(kb + q * 32 + 8 * v + e), __uint_as_float(o[8 * v + e])) * a.scale;
          uint4 w;
          w.x = pack_bf16(f[0], f[1]); w.y = pack_bf16(f[2], f[3]);
          w.z = pack_bf16(f[4], f[5]); w.w = pack_bf16(f[6], f[7]);
          *reinterpret_cast<uint4*>(srow + (q * 4 + v) * 16) = w;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads these stores
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");   // both halves of every row are staged (or a wait gave up)
    if (half == 0 && live && !*abort) {
      __nv_bfloat16* orow = a.dQ + ((size_t)bh * a.N + qpos) * D;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(orow),
                   "r"(smem_u32(stage_out + row * kStageStride)), "r"((uint32_t)kRowBytes)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory is released at exit
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
  if (tid == 0 && abort_s) atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);
}

// Per query row: D~_t = sum_c dO[t,c] * O[t,c] and -LSE_t * log2(e).  d/8 lanes share a row (16 bytes
// each) and a warp takes kPrepUnroll groups of 256/d rows with all loads issued before the arithmetic:
// the kernel only streams O and dO once and should run at memory speed.  With the rounding remainder of O
// (Olo, optional) the sum runs over O + Olo, which is O to fp32 accuracy.
constexpr int kPrepUnroll = 4;
__global__ void bwd_prep_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ Olo,
                                const __nv_bfloat16* __restrict__ dO, const float* __restrict__ LSE,
                                float2* __restrict__ stats, long long rows, int d) {
  const int lane = threadIdx.x & 31;
  const int lpr = d >> 3, rpw = 32 / lpr;   // lanes per row, rows per warp-wide load (d = 64: 8, 4; d = 128: 16, 2)
  const long long warp_id = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long row0 = warp_id * (kPrepUnroll * rpw) + lane / lpr;
  const int c = (lane % lpr) * 8;
  uint4 o[kPrepUnroll], l[kPrepUnroll], g[kPrepUnroll];
#pragma unroll
  for (int u = 0; u < kPrepUnroll; ++u) {
    const long long row = row0 + u * rpw;
    o[u] = l[u] = g[u] = make_uint4(0, 0, 0, 0);
    if (row < rows) {
      o[u] = *reinterpret_cast<const uint4*>(O + row * d + c);
      g[u] = *reinterpret_cast<const uint4*>(dO + row * d + c);
      if (Olo) l[u] = *reinterpret_cast<const uint4*>(Olo + row * d + c);
    }
  }
#pragma unroll
  for (int u = 0; u < kPrepUnroll; ++u) {
    const uint32_t ow[4] = {o[u].x, o[u].y, o[u].z, o[u].w}, gw[4] = {g[u].x, g[u].y, g[u].z, g[u].w};
    const uint32_t lw[4] = {l[u].x, l[u].y, l[u].z, l[u].w};
    float acc = 0.f, acc_lo = 0.f;   // the remainder's products are 2^-9 of the others: summed apart, added last
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc = fmaf(__uint_as_float(ow[j] << 16), __uint_as_float(gw[j] << 16), acc);
      acc = fmaf(__uint_as_float(ow[j] & 0xffff0000u), __uint_as_float(gw[j] & 0xffff0000u), acc);
      acc_lo = fmaf(__uint_as_float(lw[j] << 16), __uint_as_float(gw[j] << 16), acc_lo);
      acc_lo = fmaf(__uint_as_float(lw[j] & 0xffff0000u), __uint_as_float(gw[j] & 0xffff0000u), acc_lo);
    }
    acc += acc_lo;
    for (int off = lpr >> 1; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    const long long row = row0 + u * rpw;
    if ((lane % lpr) == 0 && row < rows) stats[row] = make_float2(-LSE[row] * 1.4426950408889634f, acc);
  }
}

// kbar[bh][c] += (1/N) * sum of K[bh][t][c] over this block's rows (kbar zeroed beforehand).
__global__ void __launch_bounds__(256) kbar_kernel(const __nv_bfloat16* __restrict__ K, float* __restrict__ kbar,
                                                   int N, int d, int rows_per_block) {
  __shared__ float red[256 * 8];
  const int bh = blockIdx.y, tid = threadIdx.x;
  const int lpr = d / 8, rps = 256 / lpr;          // lanes per row (16 bytes each), rows per step
  const int chunk = tid % lpr, r_in = tid / lpr;
  const int r0 = blockIdx.x * rows_per_block, r1 = min(N, r0 + rows_per_block);
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  for (int r = r0 + r_in; r < r1; r += rps) {
    const uint4 q = *reinterpret_cast<const uint4*>(K + ((size_t)bh * N + r) * d + chunk * 8);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[2 * e] += __uint_as_float(w[e] << 16);
      acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) red[tid * 8 + e] = acc[e];
  __syncthreads();
  if (tid < d) {
    const int ch = tid / 8, e = tid % 8;
    float sum = 0.f;
    for (int r = 0; r < rps; ++r) sum += red[(r * lpr + ch) * 8 + e];
    atomicAdd(kbar + (size_t)bh * d + tid, sum / (float)N);
  }
}

}  // namespace

int launch_bwd_prep(const Geom& g, const __nv_bfloat16* O, const __nv_bfloat16* Olo, const __nv_bfloat16* dO,
                    const float* LSE, const __nv_bfloat16* K, float2* stats, float* kbar, cudaStream_t st) {
  const long long rows = (long long)g.B * g.Hq * g.N;
  const long long rows_per_block = 8LL * kPrepUnroll * (32 / (g.d >> 3));
  bwd_prep_kernel<<<(unsigned)((rows + rows_per_block - 1) / rows_per_block), 256, 0, st>>>(O, Olo, dO, LSE, stats, rows, g.d);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  const int nsplit = 64, rpb = (g.N + nsplit - 1) / nsplit;
  kbar_kernel<<<dim3(nsplit, g.B * g.Hkv), 256, 0, st>>>(K, kbar, g.N, g.d, rpb);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

template <int D>
static int launch_dq_t(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO, const __nv_bfloat16* K,
                       const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, const float2* stats,
                       const float* Dacc, const float* kbar, __nv_bfloat16* dQ, int* status, cudaStream_t st) {
  using Cfg = DqCfg<D>;
  CUtensorMap mQ, mdO, mK, mV, mKc, mVc;
  const long long rc = g.Rc > 0 ? g.Rc : 1;
  // the sequence starts at token tok0 of rows of Nrow tokens: shifted bases, rows beyond its end read as zero
  const size_t sh = (size_t)g.tok0 * D;
  int r = make_tmap_bf16(&mQ, Q + sh, D, g.N, (long long)g.B * g.Hq, kTile, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&mdO, dO + sh, D, g.N, (long long)g.B * g.Hq, kTile, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&mK, K + sh, D, g.N, (long long)g.B * g.Hkv, kKeys, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&mV, V + sh, D, g.N, (long long)g.B * g.Hkv, kKeys, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&mKc, Kc, D, rc, (long long)g.B * g.Hkv, kKeys);
  if (r == LRSA_OK) r = make_tmap_bf16(&mVc, Vc, D, rc, (long long)g.B * g.Hkv, kKeys);
  if (r != LRSA_OK) return r;
  DqArgs a;
  a.plan = make_plan(g, kTile);
  a.BH = g.B * g.Hq; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.Nrow;
  a.stats = stats + g.tok0; a.Dacc = Dacc + g.tok0; a.kbar = kbar; a.dQ = dQ + sh;
  a.scale = g.scale; a.scale_log2 = g.scale * 1.4426950408889634f;
  a.status = status;
  const long long grid = (long long)a.plan.total * a.BH;
  if (grid > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  auto kern = lrsa_bwd_dq_kernel<D>;
  LRSA_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem));
  kern<<<(unsigned)grid, Cfg::kThreads, Cfg::kSmem, st>>>(mQ, mdO, mK, mV, mKc, mVc, a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

int launch_bwd_dq_sm100(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO, const __nv_bfloat16* K,
                        const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, const float2* stats,
                        const float* Dacc, const float* kbar, __nv_bfloat16* dQ, int* status, cudaStream_t st) {
  return g.d == 128 ? launch_dq_t<128>(g, Q, dO, K, V, Kc, Vc, stats, Dacc, kbar, dQ, status, st)
                    : launch_dq_t<64>(g, Q, dO, K, V, Kc, Vc, stats, Dacc, kbar, dQ, status, st);
}

}  // namespace lrsa
