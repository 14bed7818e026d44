// LRSA attention backward, dQ part, on tcgen05 tensor cores.
//
// Same row-block decomposition as the forward: a CTA owns 256 query rows (two 128-row tiles) of one
// (batch, query head) and walks their key list in 64-key tiles.  Per tile and key tile j:
//   S  = Q K_j^T          (smem x smem -> TMEM)      P  = exp2(S*c - LSE*log2e)
//   dP = dO V_j^T         (smem x smem -> TMEM)      dS = P * (dP - D)          (bf16, back into TMEM)
//   dQ += dS K_j          (TMEM x smem -> TMEM)      epilogue: dQ * scale -> bf16
// D = rowsum(dO * O) comes from a small preparation kernel.  dQ never leaves TMEM until the end, so
// the result does not depend on any accumulation order.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

using namespace ptx;

constexpr int kKeys = 64;   // keys per tile in this kernel

template <int D>
struct DqCfg {
  static constexpr int kSub = D / 64;
  static constexpr int kQSubBytes = kTile * 128;           // 128 query rows x 128 bytes
  static constexpr int kQTileBytes = kSub * kQSubBytes;    // one Q or dO tile
  static constexpr int kKSubBytes = kKeys * 128;           // 64 key rows x 128 bytes
  static constexpr int kKTileBytes = kSub * kKSubBytes;    // one K or V tile
  static constexpr int kStages = D == 128 ? 6 : 12;
  static constexpr int kSmem = 4 * kQTileBytes + kStages * kKTileBytes + 1024;
  static constexpr int kThreads = 320;
  // TMEM columns per query tile t: S at t*128, dP at t*128+64, dQ at 256 + t*D
  static constexpr uint32_t kColS = 0, kColP = 64, kColQ = 256;
};

struct DqArgs {
  BlockPlan plan;
  int BH, Hq, Hkv, G, N;
  const float* LSE;
  const float* Dsum;
  __nv_bfloat16* dQ;
  float scale, scale_log2;
  int* status;
};

struct DqBars {
  uint64_t q_full;
  uint64_t kv_full[12], kv_empty[12];
  uint64_t s_full[2], p_full[2], acc_done[2];
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
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0, sdO = smem0 + 2 * Cfg::kQTileBytes, sRing = smem0 + 4 * Cfg::kQTileBytes;

  const int bh = blockIdx.x % a.BH, blk = blockIdx.x / a.BH;
  const RowBlock rb = decode_block(a.plan, blk);
  const int bh_kv = (bh / a.Hq) * a.Hkv + (bh % a.Hq) / a.G;
  const int n_ct = (rb.n_front + kKeys - 1) / kKeys;
  int n_t[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int first = rb.q0 + t * kTile;
    n_t[t] = first >= rb.q_end ? 0 : n_ct + (min(first + kTile - 1, rb.q_end - 1) - rb.dense_start) / kKeys + 1;
  }
  const int n_max = max(n_t[0], n_t[1]);

  if (tid == 0) {
    abort_s = 0;
    mbar_init(smem_u32(&bars.q_full), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.p_full[t]), 128);
      mbar_init(smem_u32(&bars.acc_done[t]), 1);
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
    if (lane == 0) {
      prefetch_tensormap(&mapQ); prefetch_tensormap(&mapdO); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
      prefetch_tensormap(&mapKc); prefetch_tensormap(&mapVc);
      mbar_expect_tx(smem_u32(&bars.q_full), 4 * Cfg::kQTileBytes);
      for (int t = 0; t < 2; ++t)
        for (int h = 0; h < Cfg::kSub; ++h) {
          tma_load_3d(sQ + t * Cfg::kQTileBytes + h * Cfg::kQSubBytes, &mapQ, h * 64, rb.q0 + t * kTile, bh,
                      smem_u32(&bars.q_full));
          tma_load_3d(sdO + t * Cfg::kQTileBytes + h * Cfg::kQSubBytes, &mapdO, h * 64, rb.q0 + t * kTile, bh,
                      smem_u32(&bars.q_full));
        }
      int it = 0;
      bool ok = true;
      for (int j = 0; j < n_max && ok; ++j) {
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
        for (int back = 1; back <= NS && back <= it; ++back) {
          const int i2 = it - back;
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&bars.kv_full[i2 % NS]), (i2 / NS) & 1) && clock64() - t0 < 2000000) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kKeys, 0, 0);   // S, dP : 128 x 64
      constexpr uint32_t idesc_q = make_idesc_bf16(kTile, D, 0, 1);       // dQ    : 128 x D, B = K_j MN-major
      bool ok = mbar_wait(smem_u32(&bars.q_full), 0, abort);
      for (int j = 0; j <= n_max && ok; ++j) {
        // ring order: K_j at 2j, V_j at 2j+1.  Iteration j issues S/dP for tile j and dQ for tile j-1.
        const int itK = 2 * j, itV = 2 * j + 1, itKp = 2 * j - 2;
        if (j < n_max) {
          ok = mbar_wait(smem_u32(&bars.kv_full[itK % NS]), (itK / NS) & 1, abort);
          if (ok) ok = mbar_wait(smem_u32(&bars.kv_full[itV % NS]), (itV / NS) & 1, abort);
        }
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t sK = sRing + (itK % NS) * Cfg::kKTileBytes;
        const uint32_t sV = sRing + (itV % NS) * Cfg::kKTileBytes;
        const uint32_t sKp = sRing + ((itKp + 2 * NS) % NS) * Cfg::kKTileBytes;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const bool do_s = j < n_t[t], do_q = j >= 1 && (j - 1) < n_t[t];
          if (do_q) {
            ok = mbar_wait(smem_u32(&bars.p_full[t]), (j - 1) & 1, abort);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < kKeys / 16; ++kk)
              umma_ts(tmem + Cfg::kColQ + t * D, tmem + t * kTile + Cfg::kColS + kk * 8,
                      make_smem_desc_sw128(sKp + kk * 2048, Cfg::kKSubBytes, 1024), idesc_q,
                      (j - 1 > 0 || kk > 0) ? 1u : 0u);
            umma_commit(smem_u32(&bars.acc_done[t]));
          }
          if (do_s) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t qoff = (kk >> 2) * Cfg::kQSubBytes + (kk & 3) * 32;
              const uint32_t koff = (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32;
              umma_ss(tmem + t * kTile + Cfg::kColS, make_smem_desc_sw128(sQ + t * Cfg::kQTileBytes + qoff, 16, 1024),
                      make_smem_desc_sw128(sK + koff, 16, 1024), idesc_s, kk > 0 ? 1u : 0u);
            }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t qoff = (kk >> 2) * Cfg::kQSubBytes + (kk & 3) * 32;
              const uint32_t koff = (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32;
              umma_ss(tmem + t * kTile + Cfg::kColP, make_smem_desc_sw128(sdO + t * Cfg::kQTileBytes + qoff, 16, 1024),
                      make_smem_desc_sw128(sV + koff, 16, 1024), idesc_s, kk > 0 ? 1u : 0u);
            }
            umma_commit(smem_u32(&bars.s_full[t]));
          }
        }
        if (!ok) break;
        if (j < n_max) umma_commit(smem_u32(&bars.kv_empty[itV % NS]));   // V_j: used by dP only
        if (j >= 1) umma_commit(smem_u32(&bars.kv_empty[(itKp + 2 * NS) % NS]));  // K_{j-1}: S and dQ done
      }
    }
  } else {
    const int t = (warp - 2) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t S_addr = tmem + lane_addr + t * kTile + Cfg::kColS;
    const uint32_t P_addr = tmem + lane_addr + t * kTile + Cfg::kColP;
    const uint32_t Q_addr = tmem + lane_addr + Cfg::kColQ + t * D;
    const int qpos = rb.q0 + t * kTile + row;
    const int n = n_t[t];
    const float c = a.scale_log2;
    const bool live = qpos < rb.q_end;
    // exp2(s*c - lse*log2e); rows outside the block get lse = +inf so that P = 0
    const float nl2 = live ? -a.LSE[(size_t)bh * a.N + qpos] * 1.4426950408889634f : -INFINITY;
    const float Dt = live ? a.Dsum[(size_t)bh * a.N + qpos] : 0.f;
    bool ok = true;
    for (int j = 0; j < n; ++j) {
      ok = mbar_wait(smem_u32(&bars.s_full[t]), j & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      uint32_t s[64], dp[64];
      tmem_ld32(S_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
      tmem_ld32(S_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
      tmem_ld32(P_addr, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
      tmem_ld32(P_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
      tmem_wait_ld();
      const int limit = j < n_ct ? rb.n_front - j * kKeys : qpos - (rb.dense_start + (j - n_ct) * kKeys) + 1;
      if (limit < kKeys) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= limit) s[i] = 0xff800000u;
      }
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int e = q * 32 + 2 * i;
          const float p0 = ex2(fmaf(__uint_as_float(s[e]), c, nl2));
          const float p1 = ex2(fmaf(__uint_as_float(s[e + 1]), c, nl2));
          pk[i] = pack_bf16(p0 * (__uint_as_float(dp[e]) - Dt), p1 * (__uint_as_float(dp[e + 1]) - Dt));
        }
        // 16 columns of packed dS
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
            ::"r"(S_addr + q * 16), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]),
              "r"(pk[7]), "r"(pk[8]), "r"(pk[9]), "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15])
            : "memory");
      }
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[t]));
    }
    if (ok && n > 0) {
      ok = mbar_wait(smem_u32(&bars.acc_done[t]), (n - 1) & 1, abort);
      if (ok) {
        tc_fence_after_sync();
        __nv_bfloat16* orow = a.dQ + ((size_t)bh * a.N + qpos) * D;
#pragma unroll
        for (int q = 0; q < D / 32; ++q) {
          uint32_t o[32];
          tmem_ld32(Q_addr + q * 32, o);
          tmem_wait_ld();
          if (live) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * a.scale, __uint_as_float(o[8 * v + 1]) * a.scale);
              w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * a.scale, __uint_as_float(o[8 * v + 3]) * a.scale);
              w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * a.scale, __uint_as_float(o[8 * v + 5]) * a.scale);
              w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * a.scale, __uint_as_float(o[8 * v + 7]) * a.scale);
              *reinterpret_cast<uint4*>(orow + q * 32 + v * 8) = w;
            }
          }
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
  if (tid == 0 && abort_s) atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);
}

// D_t = sum_c dO[t,c] * O[t,c], one warp per query row.
__global__ void bwd_prep_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO,
                                float* __restrict__ Dsum, long long rows, int d) {
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  float acc = 0.f;
  for (int c = lane * 2; c < d; c += 64) {
    const __nv_bfloat162 o = *reinterpret_cast<const __nv_bfloat162*>(O + row * d + c);
    const __nv_bfloat162 g = *reinterpret_cast<const __nv_bfloat162*>(dO + row * d + c);
    acc += __bfloat162float(o.x) * __bfloat162float(g.x) + __bfloat162float(o.y) * __bfloat162float(g.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) Dsum[row] = acc;
}

}  // namespace

int launch_bwd_prep(const Geom& g, const __nv_bfloat16* O, const __nv_bfloat16* dO, float* Dsum, cudaStream_t st) {
  const long long rows = (long long)g.B * g.Hq * g.N;
  bwd_prep_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(O, dO, Dsum, rows, g.d);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

template <int D>
static int launch_dq_t(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO, const __nv_bfloat16* K,
                       const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, const float* LSE,
                       const float* Dsum, __nv_bfloat16* dQ, int* status, cudaStream_t st) {
  using Cfg = DqCfg<D>;
  CUtensorMap mQ, mdO, mK, mV, mKc, mVc;
  const long long rc = g.Rc > 0 ? g.Rc : 1;
  int r = make_tmap_bf16(&mQ, Q, D, g.N, (long long)g.B * g.Hq, kTile);
  if (r == LRSA_OK) r = make_tmap_bf16(&mdO, dO, D, g.N, (long long)g.B * g.Hq, kTile);
  if (r == LRSA_OK) r = make_tmap_bf16(&mK, K, D, g.N, (long long)g.B * g.Hkv, kKeys);
  if (r == LRSA_OK) r = make_tmap_bf16(&mV, V, D, g.N, (long long)g.B * g.Hkv, kKeys);
  if (r == LRSA_OK) r = make_tmap_bf16(&mKc, Kc, D, rc, (long long)g.B * g.Hkv, kKeys);
  if (r == LRSA_OK) r = make_tmap_bf16(&mVc, Vc, D, rc, (long long)g.B * g.Hkv, kKeys);
  if (r != LRSA_OK) return r;
  DqArgs a;
  a.plan = make_plan(g, 2 * kTile);
  a.BH = g.B * g.Hq; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.N;
  a.LSE = LSE; a.Dsum = Dsum; a.dQ = dQ;
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
                        const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, const float* LSE,
                        const float* Dsum, __nv_bfloat16* dQ, int* status, cudaStream_t st) {
  return g.d == 128 ? launch_dq_t<128>(g, Q, dO, K, V, Kc, Vc, LSE, Dsum, dQ, status, st)
                    : launch_dq_t<64>(g, Q, dO, K, V, Kc, Vc, LSE, Dsum, dQ, status, st);
}

}  // namespace lrsa
