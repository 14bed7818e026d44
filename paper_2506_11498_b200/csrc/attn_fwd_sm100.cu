// LRSA attention forward on tcgen05 tensor cores (Section 3.1 Eq. 3 under the chunked mask of
// Section 3.2).
//
// A CTA owns up to 256 query rows of one (batch, query head) that share a key list (two 128-row tiles of
// one query chunk) and walks the list (first n_front rows of the compact sinks+kept buffer, then a contiguous
// range of original positions up to the diagonal) in 128-key tiles; every K_j / V_j tile in shared memory
// serves both query tiles.  Roles:
//   warp 0      TMA producer: the Q tiles once, then K_j, V_j tiles through a ring of shared-memory slots
//   warp 1      issues S_t = Q_t K_j^T (both operands in shared memory) into the tile's TMEM region; owns
//               the TMEM allocation
//   warp 2      issues O_t += P_t V_j with P_t read from tensor memory
//   warps 4-7   softmax of query tile 0, warps 8-11 of query tile 1: one thread per row, S from TMEM, online
//               softmax in fp32 with the maximum only raised when it grew by more than 2^8 (then O_t is
//               rescaled in TMEM), P written back over S as packed bf16
// The two tiles take turns on the tensor core: while one tile's scores are in its softmax warpgroup the
// products of the other run.  A row belongs to one thread from its scores to its output, so the softmax
// threads exchange nothing.  The issuing warps run their loops with all lanes and elect one lane per
// instruction.  All mbarrier waits are bounded; on expiry the CTA records LRSA_ERR_TIMEOUT in the workspace
// header and leaves.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

using namespace ptx;

template <int D>
struct FwdCfg {
  static constexpr int kSub = D / 64;                 // 64-column (128-byte) sub-tiles per tile
  static constexpr int kSubBytes = kTile * 128;       // 16 KB
  static constexpr int kTileBytes = kSub * kSubBytes; // one Q / K / V tile
  // A Q tile is followed by 2 KB so that the output rows of the tile can be staged there with 16 bytes of
  // padding per row (128 rows x (2D + 16) bytes = tile + 2 KB); the next tile stays 1024-byte aligned.
  static constexpr int kQRegion = kTileBytes + 2048;
  static constexpr int kStages = D == 128 ? 4 : 10;   // K/V ring slots
  static constexpr int kSmem = 2 * kQRegion + kStages * kTileBytes + 1024;
  static constexpr int kThreads = 384;
  // TMEM columns: accumulator O of query tile t at 128t, its S (and, packed over it, P) at 256 + 128t
  static constexpr uint32_t kColO = 0, kColS = 256;
};

struct FwdArgs {
  BlockPlan plan;          // blocks of up to 256 query rows (two tiles)
  int BH, Hq, Hkv, G, N;   // N: tokens per (batch, head) row of O and LSE (the row stride)
  __nv_bfloat16* O;
  __nv_bfloat16* Olo;        // optional: receives bf16(O_fp32 - O), the part of the output the bf16 O cannot hold
  float* LSE;
  float scale, scale_log2;   // softmax scale, and scale * log2(e)
  int* status;
};

struct FwdBars {
  uint64_t q_full;
  uint64_t kv_full[12], kv_empty[12];
  uint64_t s_full[2], p_full[2], buf_free[2], pv_done[2];   // per query tile
};

template <int D>
__global__ void __launch_bounds__(FwdCfg<D>::kThreads, 1)
lrsa_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapKc,
                const __grid_constant__ CUtensorMap mapVc, const FwdArgs a) {
  using Cfg = FwdCfg<D>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) FwdBars bars;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0, sRing = smem0 + 2 * Cfg::kQRegion;

  const int bh = blockIdx.x % a.BH, blk = blockIdx.x / a.BH;
  const RowBlock rb = decode_block(a.plan, blk);
  const int bh_kv = (bh / a.Hq) * a.Hkv + (bh % a.Hq) / a.G;
  const int n_ct = (rb.n_front + kTile - 1) / kTile;
  // key tiles of query tile t: the list, then the dense range up to the tile's last row (0: the tile is empty)
  const int n0 = n_ct + (min(rb.q_end, rb.q0 + kTile) - 1 - rb.dense_start) / kTile + 1;
  const int n1 = rb.q0 + kTile < rb.q_end ? n_ct + (rb.q_end - 1 - rb.dense_start) / kTile + 1 : 0;
  const int n = max(n0, n1);

  if (tid == 0) {
    abort_s = 0;
    mbar_init(smem_u32(&bars.q_full), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(smem_u32(&bars.s_full[t]), 1);
      mbar_init(smem_u32(&bars.p_full[t]), 128);    // every softmax thread of the tile's warpgroup
      mbar_init(smem_u32(&bars.buf_free[t]), 1);
      mbar_init(smem_u32(&bars.pv_done[t]), 1);
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
      prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
      prefetch_tensormap(&mapKc); prefetch_tensormap(&mapVc);
      mbar_expect_tx(smem_u32(&bars.q_full), (n1 > 0 ? 2 : 1) * Cfg::kTileBytes);
      for (int t = 0; t < (n1 > 0 ? 2 : 1); ++t)
        for (int h = 0; h < Cfg::kSub; ++h)
          tma_load_3d(sQ + t * Cfg::kQRegion + h * Cfg::kSubBytes, &mapQ, h * 64, rb.q0 + t * kTile, bh, smem_u32(&bars.q_full));
      int it = 0;
      bool ok = true;
      for (int j = 0; j < n && ok; ++j) {
        for (int which = 0; which < 2 && ok; ++which, ++it) {
          const int slot = it % NS, use = it / NS;
          if (use > 0) ok = mbar_wait(smem_u32(&bars.kv_empty[slot]), (use - 1) & 1, abort);
          if (!ok) break;
          const uint32_t full = smem_u32(&bars.kv_full[slot]);
          mbar_expect_tx(full, Cfg::kTileBytes);
          const bool compact = j < n_ct;
          const CUtensorMap* map = compact ? (which ? &mapVc : &mapKc) : (which ? &mapV : &mapK);
          const int row = compact ? j * kTile : rb.dense_start + (j - n_ct) * kTile;
          for (int h = 0; h < Cfg::kSub; ++h)
            tma_load_3d(sRing + slot * Cfg::kTileBytes + h * Cfg::kSubBytes, map, h * 64, row, bh_kv, full);
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
    // ---------------- S issuer: S_t = Q_t K_j^T for both query tiles ----------------
    constexpr uint32_t idesc_qk = make_idesc_bf16(kTile, kTile, 0, 0);
    const uint64_t descK0 = make_smem_desc_sw128(sRing, 16, 1024);
    const uint64_t descQ0 = make_smem_desc_sw128(sQ, 16, 1024);
    bool ok = mbar_wait_warp(smem_u32(&bars.q_full), 0, abort);
    for (int j = 0; j < n && ok; ++j) {
      const int it = 2 * j;   // ring order: K_j at 2j, V_j at 2j+1
      ok = mbar_wait_warp(smem_u32(&bars.kv_full[it % NS]), (it / NS) & 1, abort);
      const uint64_t dK = desc_advance(descK0, (it % NS) * Cfg::kTileBytes);
      for (int t = 0; t < 2 && ok; ++t) {
        if (j >= (t == 0 ? n0 : n1)) continue;
        // S_t is also where P_t lives: the tile's previous O += P V must have read it
        if (j >= 1) ok = mbar_wait_warp(smem_u32(&bars.buf_free[t]), (j - 1) & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t dQ = desc_advance(descQ0, t * Cfg::kQRegion);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * Cfg::kSubBytes + (kk & 3) * 32;
          const uint64_t ad = desc_advance(dQ, off), bd = desc_advance(dK, off);
          if (elect_one()) umma_ss(tmem + Cfg::kColS + t * kTile, ad, bd, idesc_qk, kk > 0 ? 1u : 0u);
        }
        if (elect_one()) umma_commit(smem_u32(&bars.s_full[t]));
        __syncwarp();
      }
      if (ok && elect_one()) umma_commit(smem_u32(&bars.kv_empty[it % NS]));   // K_j is used by the S products only
      __syncwarp();
    }
  } else if (warp == 2) {
    // ---------------- O issuer: O_t += P_t V_j ----------------
    constexpr uint32_t idesc_pv = make_idesc_bf16(kTile, D, 0, 1);
    const uint64_t descV0 = make_smem_desc_sw128(sRing, Cfg::kSubBytes, 1024);   // V_j MN-major
    bool ok = true;
    for (int j = 0; j < n && ok; ++j) {
      const int it = 2 * j + 1;
      ok = mbar_wait_warp(smem_u32(&bars.kv_full[it % NS]), (it / NS) & 1, abort);
      const uint64_t dV = desc_advance(descV0, (it % NS) * Cfg::kTileBytes);
      for (int t = 0; t < 2 && ok; ++t) {
        if (j >= (t == 0 ? n0 : n1)) continue;
        ok = mbar_wait_warp(smem_u32(&bars.p_full[t]), j & 1, abort);
        if (!ok) break;
        tc_fence_after_sync();
        // packed P_t: keys [16k, 16k+16) in columns [8k, 8k+8) of the tile's S region
#pragma unroll
        for (int kk = 0; kk < kTile / 16; ++kk) {
          const uint64_t bd = desc_advance(dV, kk * 2048);
          if (elect_one())
            umma_ts(tmem + Cfg::kColO + t * kTile, tmem + Cfg::kColS + t * kTile + kk * 8, bd, idesc_pv,
                    (kk > 0 || j > 0) ? 1u : 0u);
        }
        if (elect_one()) {
          umma_commit(smem_u32(&bars.buf_free[t]));    // S_t of the next key tile may overwrite P_t
          umma_commit(smem_u32(&bars.pv_done[t]));     // phase j: O_t holds key tiles 0..j
        }
        __syncwarp();
      }
      if (ok && elect_one()) umma_commit(smem_u32(&bars.kv_empty[it % NS]));
      __syncwarp();
    }
  } else if (warp >= 4) {
    // ---------------- softmax + epilogue: warpgroup t owns query tile t, one thread per row ----------------
    const int t = (warp - 4) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t S_addr = tmem + lane_addr + Cfg::kColS + t * kTile;
    const uint32_t O_addr = tmem + lane_addr + Cfg::kColO + t * kTile;
    const int nt = t == 0 ? n0 : n1;
    const int qpos = rb.q0 + t * kTile + row;
    const float c = a.scale_log2;
    float m = 0.f, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nt && ok; ++j) {
      ok = mbar_wait(smem_u32(&bars.s_full[t]), j & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      // keys of the tile this row may see: the first `limit`
      const int limit = j < n_ct ? rb.n_front - j * kTile : qpos - (rb.dense_start + (j - n_ct) * kTile) + 1;
      // Row maximum over the 128 columns, 64 at a time; the second half stays in registers for its
      // exponentials, the first half is read again afterwards (a second read of tensor memory is cheaper than
      // 64 more live registers).
      uint32_t s[64];
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        tmem_ld32(S_addr + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tmem_ld32(S_addr + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tmem_wait_ld();
        if (limit < kTile) {
          const int lim = limit - h * 64;
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (i >= lim) s[i] = 0xff800000u;  // -inf
        }
#pragma unroll
        for (int i = 0; i < 64; i += 4) {
          mx0 = fmaxf(mx0, __uint_as_float(s[i]));
          mx1 = fmaxf(mx1, __uint_as_float(s[i + 1]));
          mx2 = fmaxf(mx2, __uint_as_float(s[i + 2]));
          mx3 = fmaxf(mx3, __uint_as_float(s[i + 3]));
        }
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      if (j == 0) {
        m = mx == -INFINITY ? 0.f : mx;
      } else {
        // the maximum is only raised when it grew by more than 2^8 (then O is rescaled in tensor memory)
        const bool need = (mx - m) * c > 8.f;
        if (__any_sync(0xffffffffu, need)) {
          // O must hold every earlier tile before it is rescaled; the O issuer cannot start tile j before
          // this thread has arrived on p_full, so the rescale cannot race with it
          ok = mbar_wait(smem_u32(&bars.pv_done[t]), (j - 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          const float f = need ? ex2((m - mx) * c) : 1.f;
#pragma unroll
          for (int q = 0; q < D / 32; ++q) {
            uint32_t o[32];
            tmem_ld32(O_addr + q * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
            tmem_st32(O_addr + q * 32, o);
          }
          tmem_wait_st();
          l *= f;
          if (need) m = mx;
        }
      }
      const float nmc = -m * c;
      const uint64_t c2 = f2_pack(c, c), nmc2 = f2_pack(nmc, nmc);
      uint64_t sum2 = f2_pack(0.f, 0.f);
      // exponentials of 64 columns held in s[]: scale and shift as packed pairs (one issue slot for two
      // elements); one exponential in eight on the FMA pipe, the rest on the MUFU pipe
      auto exps = [&](uint32_t (&pk)[32]) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float x0, x1;
          f2_unpack(f2_fma(f2_pack(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, nmc2), x0, x1);
          const float p0 = ex2(x0);
          const float p1 = (i & 3) == 3 ? ex2_fma(x1) : ex2(x1);
          sum2 = f2_add(sum2, f2_pack(p0, p1));
          pk[i] = pack_bf16(p0, p1);
        }
      };
      uint32_t pk_hi[32], pk_lo[32];
      exps(pk_hi);   // s[] holds columns 64..127 (masked)
      tmem_ld32(S_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
      tmem_ld32(S_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
      tmem_wait_ld();
      if (limit < 64) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= limit) s[i] = 0xff800000u;
      }
      exps(pk_lo);
      float sum0, sum1;
      f2_unpack(sum2, sum0, sum1);
      l += sum0 + sum1;
      // P as packed bf16 over the first 64 columns of the tile's S (this thread's own lane: nobody else reads it)
      tmem_st32(S_addr, pk_lo);
      tmem_st32(S_addr + 32, pk_hi);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[t]));
    }
    if (ok && nt > 0) ok = mbar_wait(smem_u32(&bars.pv_done[t]), (nt - 1) & 1, abort);
    // The output rows go through shared memory (the tile's Q region, idle once its last S product is done,
    // which pv_done implies) and leave as one bulk copy per row: per-thread 16-byte stores to rows 256 bytes
    // apart cost a transaction each.  Rows are padded by 16 bytes so that a warp's stores spread over the banks.
    constexpr int kRowBytes = D * 2, kStageStride = kRowBytes + 16;
    static_assert(kTile * kStageStride <= Cfg::kQRegion, "staging fits the Q region");
    unsigned char* stage_out = smem_raw + (sQ - smem_u32(smem_raw)) + t * Cfg::kQRegion;
    const bool store = qpos < rb.q_end && nt > 0;
    if (ok && nt > 0) {
      tc_fence_after_sync();
      const float inv = 1.0f / l;
      unsigned char* srow = stage_out + row * kStageStride;
      // the remainder goes straight to global memory (contiguous bytes per thread, written once)
      __nv_bfloat16* lo_row = a.Olo && store ? a.Olo + ((size_t)bh * a.N + qpos) * D : nullptr;
#pragma unroll
      for (int q = 0; q < D / 32; ++q) {
        uint32_t o[32];
        tmem_ld32(O_addr + q * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(o[8 * v + e]) * inv;
          uint4 w;
          w.x = pack_bf16(f[0], f[1]); w.y = pack_bf16(f[2], f[3]);
          w.z = pack_bf16(f[4], f[5]); w.w = pack_bf16(f[6], f[7]);
          *reinterpret_cast<uint4*>(srow + (q * 4 + v) * 16) = w;
          if (lo_row) {
            const uint32_t hw[4] = {w.x, w.y, w.z, w.w};
            uint32_t lw[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              lw[e] = pack_bf16(f[2 * e] - __uint_as_float(hw[e] << 16), f[2 * e + 1] - __uint_as_float(hw[e] & 0xffff0000u));
            *reinterpret_cast<uint4*>(lo_row + q * 32 + v * 8) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
          }
        }
      }
      if (store) a.LSE[(size_t)bh * a.N + qpos] = m * a.scale + logf(l);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads this thread's stores
      if (store && !*abort) {
        __nv_bfloat16* orow = a.O + ((size_t)bh * a.N + qpos) * D;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(orow),
                     "r"(smem_u32(srow)), "r"((uint32_t)kRowBytes)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory is released at exit
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
  if (tid == 0 && abort_s) atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);
}

// K, V point at the sequence's first token; `kept` entries are positions in the whole row (tok0 + local).
__global__ void compact_kv_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                                  const int32_t* __restrict__ idx, __nv_bfloat16* __restrict__ Kc,
                                  __nv_bfloat16* __restrict__ Vc, int BHkv, int Nrow, int d, int S, int Rc, int tok0,
                                  int kept_stride, int kept_off) {
  // one warp per compact row; a row is d*2 bytes = 8 (d=128) or 4 (d=64) bytes per lane
  const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= (long long)BHkv * Rc) return;
  const int bh = (int)(wid / Rc), r = (int)(wid % Rc), lane = threadIdx.x & 31;
  const int pos = r < S ? r : idx[(size_t)bh * kept_stride + kept_off + (r - S)] - tok0;
  const size_t src = ((size_t)bh * Nrow + pos) * d, dst = ((size_t)bh * Rc + r) * d;
  if (d == 128) {
    reinterpret_cast<uint2*>(Kc + dst)[lane] = reinterpret_cast<const uint2*>(K + src)[lane];
    reinterpret_cast<uint2*>(Vc + dst)[lane] = reinterpret_cast<const uint2*>(V + src)[lane];
  } else {
    reinterpret_cast<uint32_t*>(Kc + dst)[lane] = reinterpret_cast<const uint32_t*>(K + src)[lane];
    reinterpret_cast<uint32_t*>(Vc + dst)[lane] = reinterpret_cast<const uint32_t*>(V + src)[lane];
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

struct FwdWs {
  size_t kc, vc, total;
};
FwdWs fwd_ws_layout(const Geom& g) {
  FwdWs w;
  const size_t rc = g.Rc > 0 ? g.Rc : 1;
  const size_t bytes = align_up((size_t)g.B * g.Hkv * rc * g.d * sizeof(__nv_bfloat16), 1024);
  w.kc = 1024;
  w.vc = w.kc + bytes;
  w.total = w.vc + bytes;
  return w;
}

}  // namespace

int make_tmap_bf16(CUtensorMap* map, const void* base, int d, long long rows, long long outer, int box_rows,
                   long long row_stride) {
  EncodeFn fn = encode_fn();
  if (!fn) return LRSA_ERR_CUDA;
  if (row_stride <= 0) row_stride = rows;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)outer};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * (cuuint64_t)row_stride};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LRSA_OK : LRSA_ERR_CUDA;
}

int make_tmap_bf16_rows(CUtensorMap* map, const void* base, int d, long long rows) {
  EncodeFn fn = encode_fn();
  if (!fn) return LRSA_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  cuuint32_t box[2] = {64, 1};
  cuuint32_t es[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? LRSA_OK : LRSA_ERR_CUDA;
}

int launch_compact_kv(const Geom& g, const __nv_bfloat16* K, const __nv_bfloat16* V, const int32_t* idx,
                      __nv_bfloat16* Kc, __nv_bfloat16* Vc, cudaStream_t st) {
  if (g.Rc == 0) return LRSA_OK;
  const long long warps = (long long)g.B * g.Hkv * g.Rc;
  const unsigned blocks = (unsigned)((warps + 7) / 8);
  const size_t sh = (size_t)g.tok0 * g.d;
  compact_kv_kernel<<<blocks, 256, 0, st>>>(K + sh, V + sh, idx, Kc, Vc, g.B * g.Hkv, g.Nrow, g.d, g.S, g.Rc, g.tok0,
                                            g.Wtot * g.K, g.woff * g.K);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

size_t attn_fwd_ws_bytes(const Geom& g) { return fwd_ws_layout(g).total; }

template <int D>
static int launch_fwd_t(const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K, const __nv_bfloat16* V,
                        const __nv_bfloat16* Kc, const __nv_bfloat16* Vc, __nv_bfloat16* O, __nv_bfloat16* Olo, float* LSE,
                        int* status, cudaStream_t st) {
  using Cfg = FwdCfg<D>;
  CUtensorMap mQ, mK, mV, mKc, mVc;
  const long long rc = g.Rc > 0 ? g.Rc : 1;
  // the sequence starts at token tok0 of rows of Nrow tokens: shifted bases, rows beyond its end read as zero
  const size_t sh = (size_t)g.tok0 * D;
  int rc_ = make_tmap_bf16(&mQ, Q + sh, D, g.N, (long long)g.B * g.Hq, kTile, g.Nrow);
  if (rc_ == LRSA_OK) rc_ = make_tmap_bf16(&mK, K + sh, D, g.N, (long long)g.B * g.Hkv, kTile, g.Nrow);
  if (rc_ == LRSA_OK) rc_ = make_tmap_bf16(&mV, V + sh, D, g.N, (long long)g.B * g.Hkv, kTile, g.Nrow);
  if (rc_ == LRSA_OK) rc_ = make_tmap_bf16(&mKc, Kc, D, rc, (long long)g.B * g.Hkv, kTile);
  if (rc_ == LRSA_OK) rc_ = make_tmap_bf16(&mVc, Vc, D, rc, (long long)g.B * g.Hkv, kTile);
  if (rc_ != LRSA_OK) return rc_;
  FwdArgs a;
  a.plan = make_plan(g, 2 * kTile);
  a.BH = g.B * g.Hq; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.Nrow;
  a.O = O + sh; a.Olo = Olo ? Olo + sh : nullptr; a.LSE = LSE + g.tok0; a.scale = g.scale; a.scale_log2 = g.scale * 1.4426950408889634f;
  a.status = status;
  const long long grid = (long long)a.plan.total * a.BH;
  if (grid > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  auto kern = lrsa_fwd_kernel<D>;
  LRSA_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem));
  kern<<<(unsigned)grid, Cfg::kThreads, Cfg::kSmem, st>>>(mQ, mK, mV, mKc, mVc, a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

int launch_attn_fwd_sm100(const lrsa_params_t* params, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* K,
                          const __nv_bfloat16* V, const int32_t* idx, __nv_bfloat16* O, float* LSE, void* ws,
                          cudaStream_t st) {
  const FwdWs lay = fwd_ws_layout(g);
  unsigned char* base = static_cast<unsigned char*>(ws);
  LRSA_CUDA_CHECK(cudaMemsetAsync(base, 0, sizeof(WsHeader), st));
  launch_counter().n++;
  __nv_bfloat16* Kc = reinterpret_cast<__nv_bfloat16*>(base + lay.kc);
  __nv_bfloat16* Vc = reinterpret_cast<__nv_bfloat16*>(base + lay.vc);
  int* status = &reinterpret_cast<WsHeader*>(base)->status;
  __nv_bfloat16* Olo = static_cast<__nv_bfloat16*>(params->o_residual);
  // sequence after sequence (one for an unpacked batch); the compact buffers are reused in stream order
  const int n_seqs = geom_n_seqs(params);
  int woff = 0;
  for (int s = 0; s < n_seqs; ++s) {
    Geom gs;
    seq_geom(g, params->cu_seqlens, params->n_seqs, s, woff, &gs);
    woff += gs.Wsel;
    int rc = launch_compact_kv(gs, K, V, idx, Kc, Vc, st);
    if (rc == LRSA_OK)
      rc = gs.d == 128 ? launch_fwd_t<128>(gs, Q, K, V, Kc, Vc, O, Olo, LSE, status, st)
                       : launch_fwd_t<64>(gs, Q, K, V, Kc, Vc, O, Olo, LSE, status, st);
    if (rc != LRSA_OK) return rc;
  }
  return LRSA_OK;
}

}  // namespace lrsa
