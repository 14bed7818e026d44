// LRSA attention backward, dQ part, on tcgen05 tensor cores.
//
// A CTA owns one 128-row query tile of one (batch, query head) and walks its key list (the same
// row-block decomposition as the forward) in 64-key tiles.  Per key tile j:
//   S  = Q K_j^T          (smem x smem -> TMEM)      P  = exp2(S*c - LSE*log2e)
//   dP = dO V_j^T         (smem x smem -> TMEM)      dS = P * (dP - D~)         (bf16, back into TMEM)
//   A += dS K_j           (TMEM x smem -> TMEM)      M += P K_j                 (TMEM x smem -> TMEM)
// S/dP are double-buffered in TMEM: the two softmax warpgroups alternate over key tiles, so the
// tensor core computes S/dP of tile j+1 while tile j is in the softmax.
//
// D~ = rowsum(dO * O) comes from the bf16 O and is therefore only approximate; its error, and the
// bf16 rounding of dS, would be multiplied by the softmax-averaged key M_t = sum_j P_tj k_j, which is
// large when keys have outlier channels or a few salient keys dominate the row.  Rows of the exact dS
// sum to zero, so the epilogue removes whatever the rounded rows sum to:
//   dQ_t = scale * (A_t - r_t * M_t),  r_t = sum_j bf16(dS_tj)       (= scale * sum_j dS_tj (k_j - M_t))
// which cancels the error of D~ exactly and centres the rounding errors.  The kernel also writes the
// accurate D_t = sum_j P_tj dP_tj (fp32, thread-local) for the dK/dV kernel that runs after it.
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
  static constexpr int kThreads = 320;
  // TMEM columns: buffer b holds S at b*128 and dP at b*128+64; accumulators A at 256, M at 256+D
  static constexpr uint32_t kColP = 64, kColA = 256, kColM = 256 + D;
};

struct DqArgs {
  BlockPlan plan;
  int BH, Hq, Hkv, G, N;
  float2* stats;   // per query row: in (-LSE*log2e, D~); out: .y replaced by the accurate D
  __nv_bfloat16* dQ;
  float scale, scale_log2;
  int* status;
};

struct DqBars {
  uint64_t q_full, acc_done;
  uint64_t kv_full[16], kv_empty[16];
  uint64_t s_full[2], p_full[2];
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
  __shared__ float red_s[2][2][kTile];   // [warpgroup][D partial, r partial][row]
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
    mbar_init(smem_u32(&bars.acc_done), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&bars.s_full[b]), 1); mbar_init(smem_u32(&bars.p_full[b]), 128); }
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
  } else if (warp == 1) {
    // ---------------- MMA issuer: the whole warp runs the loop, one elected lane issues ----------------
    constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kKeys, 0, 0);   // S, dP : 128 x 64
    constexpr uint32_t idesc_a = make_idesc_bf16(kTile, D, 0, 1);       // A, M  : 128 x D, B = K_j MN-major
    const uint64_t descQ = make_smem_desc_sw128(sQ, 16, 1024), descdO = make_smem_desc_sw128(sdO, 16, 1024);
    const uint64_t descR = make_smem_desc_sw128(sRing, 16, 1024);                  // K-major K_j / V_j
    const uint64_t descRmn = make_smem_desc_sw128(sRing, Cfg::kKSubBytes, 1024);   // MN-major K_j
    bool ok = mbar_wait_warp(smem_u32(&bars.q_full), 0, abort);
    // ring order: K_j at 2j, V_j at 2j+1.  Iteration j issues S/dP of tile j, then A/M of tile j-1.
    for (int j = 0; j <= n && ok; ++j) {
      if (j < n) {
        const int itK = 2 * j, itV = 2 * j + 1, b = j & 1;
        ok = mbar_wait_warp(smem_u32(&bars.kv_full[itK % NS]), (itK / NS) & 1, abort);
        if (ok) ok = mbar_wait_warp(smem_u32(&bars.kv_full[itV % NS]), (itV / NS) & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t dK = desc_advance(descR, (itK % NS) * Cfg::kKTileBytes);
        const uint64_t dV = desc_advance(descR, (itV % NS) * Cfg::kKTileBytes);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t qoff = (kk >> 2) * Cfg::kQSubBytes + (kk & 3) * 32;
          const uint32_t koff = (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32;
          const uint64_t ad = desc_advance(descQ, qoff), bd = desc_advance(dK, koff);
          if (elect_one()) umma_ss(tmem + b * kTile, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t qoff = (kk >> 2) * Cfg::kQSubBytes + (kk & 3) * 32;
          const uint32_t koff = (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32;
          const uint64_t ad = desc_advance(descdO, qoff), bd = desc_advance(dV, koff);
          if (elect_one()) umma_ss(tmem + b * kTile + Cfg::kColP, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
        }
        if (elect_one()) {
          umma_commit(smem_u32(&bars.s_full[b]));
          umma_commit(smem_u32(&bars.kv_empty[itV % NS]));   // V_j is used by dP only
        }
        __syncwarp();
      }
      if (j >= 1) {
        const int pj = j - 1, b = pj & 1, itKp = 2 * pj;
        ok = mbar_wait_warp(smem_u32(&bars.p_full[b]), (pj >> 1) & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t dKp = desc_advance(descRmn, (itKp % NS) * Cfg::kKTileBytes);
        const uint32_t acc0 = pj > 0 ? 1u : 0u;
        // dS sits in columns [0,32) of the buffer's S region, P in columns [32,64), packed bf16 pairs
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          const uint64_t bd = desc_advance(dKp, kk * 2048);
          if (elect_one()) umma_ts(tmem + Cfg::kColA, tmem + b * kTile + kk * 8, bd, idesc_a, kk > 0 ? 1u : acc0);
        }
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          const uint64_t bd = desc_advance(dKp, kk * 2048);
          if (elect_one()) umma_ts(tmem + Cfg::kColM, tmem + b * kTile + 32 + kk * 8, bd, idesc_a, kk > 0 ? 1u : acc0);
        }
        if (elect_one()) umma_commit(smem_u32(&bars.kv_empty[itKp % NS]));   // K_{j-1}: S, A and M are done
        __syncwarp();
      }
    }
    if (ok && elect_one()) umma_commit(smem_u32(&bars.acc_done));
    __syncwarp();
  } else {
    // ---------------- softmax warpgroups (wg 0: even key tiles, wg 1: odd) + epilogue ----------------
    const int wg = (warp - 2) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t S_addr = tmem + lane_addr + wg * kTile;
    const uint32_t P_addr = S_addr + Cfg::kColP;
    const int qpos = rb.q0 + row;
    const bool live = qpos < rb.q_end;
    const float c = a.scale_log2;
    // rows outside the block get lse = +inf so that P = 0
    const float2 st = live ? a.stats[(size_t)bh * a.N + qpos] : make_float2(-INFINITY, 0.f);
    const float nl2 = st.x, Dt = st.y;
    float Dsum = 0.f, rsum = 0.f;
    bool ok = true;
    for (int j = wg; j < n; j += 2) {
      ok = mbar_wait(smem_u32(&bars.s_full[wg]), (j >> 1) & 1, abort);
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
      uint32_t ds[32], pp[32];
      float d0 = 0.f, d1 = 0.f, r0 = 0.f, r1 = 0.f;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float p0 = ex2(fmaf(__uint_as_float(s[2 * i]), c, nl2));
        const float p1 = ex2(fmaf(__uint_as_float(s[2 * i + 1]), c, nl2));
        const float g0 = __uint_as_float(dp[2 * i]), g1 = __uint_as_float(dp[2 * i + 1]);
        d0 = fmaf(p0, g0, d0);
        d1 = fmaf(p1, g1, d1);
        pp[i] = pack_bf16(p0, p1);
        ds[i] = pack_bf16(p0 * (g0 - Dt), p1 * (g1 - Dt));
        r0 += __uint_as_float(ds[i] << 16);
        r1 += __uint_as_float(ds[i] & 0xffff0000u);
      }
      Dsum += d0 + d1;
      rsum += r0 + r1;
      tmem_st32(S_addr, ds);
      tmem_st32(S_addr + 32, pp);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[wg]));
    }
    red_s[wg][0][row] = Dsum;
    red_s[wg][1][row] = rsum;
    asm volatile("bar.sync 1, 256;" ::: "memory");   // the eight softmax warps, whether or not a wait gave up
    if (ok) ok = mbar_wait(smem_u32(&bars.acc_done), 0, abort);
    if (ok) {
      tc_fence_after_sync();
      const float r = red_s[0][1][row] + red_s[1][1][row];
      if (wg == 0 && live) a.stats[(size_t)bh * a.N + qpos].y = red_s[0][0][row] + red_s[1][0][row];
      constexpr int CH = D / 2;   // output columns of this warpgroup
      const uint32_t A_addr = tmem + lane_addr + Cfg::kColA + wg * CH;
      const uint32_t M_addr = tmem + lane_addr + Cfg::kColM + wg * CH;
      __nv_bfloat16* orow = a.dQ + ((size_t)bh * a.N + qpos) * D + wg * CH;
#pragma unroll
      for (int q = 0; q < CH / 32; ++q) {
        uint32_t o[32], mk[32];
        tmem_ld32(A_addr + q * 32, o);
        tmem_ld32(M_addr + q * 32, mk);
        tmem_wait_ld();
        if (live) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              f[e] = fmaf(-r, __uint_as_float(mk[8 * v + e]), __uint_as_float(o[8 * v + e])) * a.scale;
            uint4 w;
            w.x = pack_bf16(f[0], f[1]); w.y = pack_bf16(f[2], f[3]);
            w.z = pack_bf16(f[4], f[5]); w.w = pack_bf16(f[6], f[7]);
            *reinterpret_cast<uint4*>(orow + q * 32 + v * 8) = w;
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

// Per query row: D~_t = sum_c dO[t,c] * O[t,c] and -LSE_t * log2(e), one warp per row.
__global__ void bwd_prep_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO,
                                const float* __restrict__ LSE, float2* __restrict__ stats, long long rows, int d) {
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
  if (lane == 0) stats[row] = make_float2(-LSE[row] * 1.4426950408889634f, acc);
}

}  // namespace

int launch_bwd_prep(const Geom& g, const __nv_bfloat16* O, const __nv_bfloat16* dO, const float* LSE,
                    float2* stats, cudaStream_t st) {
  const long long rows = (long long)g.B * g.Hq * g.N;
  bwd_prep_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(O, dO, LSE, stats, rows, g.d);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

template <int D>
static int launch_dq_t(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO, const __nv_bfloat16* K,
                       const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, float2* stats,
                       __nv_bfloat16* dQ, int* status, cudaStream_t st) {
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
  a.plan = make_plan(g, kTile);
  a.BH = g.B * g.Hq; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.N;
  a.stats = stats; a.dQ = dQ;
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
                        const __nv_bfloat16* V, const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, float2* stats,
                        __nv_bfloat16* dQ, int* status, cudaStream_t st) {
  return g.d == 128 ? launch_dq_t<128>(g, Q, dO, K, V, Kc, Vc, stats, dQ, status, st)
                    : launch_dq_t<64>(g, Q, dO, K, V, Kc, Vc, stats, dQ, status, st);
}

}  // namespace lrsa
