// LRSA attention forward on tcgen05 tensor cores (Section 3.1 Eq. 3 under the chunked mask of
// Section 3.2).
//
// A CTA owns one 128-row query tile of one (batch, query head) and walks its key list (first n_front
// rows of the compact sinks+kept buffer, then a contiguous range of original positions up to the
// diagonal) in 128-key tiles.  Q is copied once into tensor memory, so both products take their
// 128-row operand from TMEM and only K_j / V_j from shared memory.  Roles:
//   warp 0      TMA producer: the Q tile once, then K_j, V_j tiles through a ring of shared-memory slots
//   warp 1      issues S_j = Q K_j^T into one of two TMEM buffers; owns the TMEM allocation
//   warp 2      issues O += P_j V_j with P_j read from tensor memory
//   warps 4-11  softmax: both warpgroups work on every tile, 64 key columns each; S from TMEM, online
//               softmax in fp32 with the maximum only raised when it grew by more than 2^8 (then O is
//               rescaled in TMEM), P written back over S as packed bf16
// S is double-buffered, so the tensor core computes S_{j+1} while tile j is in the softmax.  The
// issuing warps run their loops with all lanes and elect one lane per instruction.  All mbarrier
// waits are bounded; on expiry the CTA records LRSA_ERR_TIMEOUT in the workspace header and leaves.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

using namespace ptx;

template <int D>
struct FwdCfg {
  static constexpr int kSub = D / 64;                 // 64-column (128-byte) sub-tiles per tile
  static constexpr int kSubBytes = kTile * 128;       // 16 KB
  static constexpr int kTileBytes = kSub * kSubBytes; // one Q / K / V tile
  static constexpr int kStages = D == 128 ? 6 : 12;   // K/V ring slots
  static constexpr int kSmem = (1 + kStages) * kTileBytes + 1024;
  static constexpr int kThreads = 384;
  // TMEM columns: Q as packed bf16 (D/2 columns), the accumulator O at 64, S buffer b at 256 + 128b
  static constexpr uint32_t kColQ = 0, kColO = 64, kColS = 256;
};

struct FwdArgs {
  BlockPlan plan;
  int BH, Hq, Hkv, G, N;   // N: tokens per (batch, head) row of O and LSE (the row stride)
  __nv_bfloat16* O;
  __nv_bfloat16* Olo;        // optional: receives bf16(O_fp32 - O), the part of the output the bf16 O cannot hold
  float* LSE;
  float scale, scale_log2;   // softmax scale, and scale * log2(e)
  int* status;
};

struct FwdBars {
  uint64_t q_full, qt_ready, pv_done;
  uint64_t kv_full[12], kv_empty[12];
  uint64_t s_full[2], p_full[2], buf_free[2];
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
  __shared__ float red_s[2][kTile];   // [column half][row] partial row sums
  __shared__ unsigned short loaded_s[2][kTile];   // [column half][row] tiles whose S this softmax thread has read
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem0, sRing = smem0 + Cfg::kTileBytes;

  const int bh = blockIdx.x % a.BH, blk = blockIdx.x / a.BH;
  const RowBlock rb = decode_block(a.plan, blk);
  const int bh_kv = (bh / a.Hq) * a.Hkv + (bh % a.Hq) / a.G;
  const int n_ct = (rb.n_front + kTile - 1) / kTile;
  const int n = n_ct + (rb.q_end - 1 - rb.dense_start) / kTile + 1;   // key tiles of this block (>= 1)

  if (tid == 0) {
    abort_s = 0;
    mbar_init(smem_u32(&bars.q_full), 1);
    mbar_init(smem_u32(&bars.qt_ready), 256);
    mbar_init(smem_u32(&bars.pv_done), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.kv_full[i]), 1); mbar_init(smem_u32(&bars.kv_empty[i]), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.s_full[b]), 1);
      mbar_init(smem_u32(&bars.p_full[b]), 256);    // every softmax thread
      mbar_init(smem_u32(&bars.buf_free[b]), 1);
    }
    fence_barrier_init();
  }
  if (tid < 2 * kTile) (&loaded_s[0][0])[tid] = 0;
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
      mbar_expect_tx(smem_u32(&bars.q_full), Cfg::kTileBytes);
      for (int h = 0; h < Cfg::kSub; ++h)
        tma_load_3d(sQ + h * Cfg::kSubBytes, &mapQ, h * 64, rb.q0, bh, smem_u32(&bars.q_full));
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
    // ---------------- S issuer: S_j = Q K_j^T into buffer j & 1 ----------------
    constexpr uint32_t idesc_qk = make_idesc_bf16(kTile, kTile, 0, 0);
    const uint64_t descK0 = make_smem_desc_sw128(sRing, 16, 1024);
    bool ok = mbar_wait_warp(smem_u32(&bars.qt_ready), 0, abort);   // Q is in tensor memory
    for (int j = 0; j < n && ok; ++j) {
      const int it = 2 * j, b = j & 1;   // ring order: K_j at 2j, V_j at 2j+1
      ok = mbar_wait_warp(smem_u32(&bars.kv_full[it % NS]), (it / NS) & 1, abort);
      if (ok && j >= 2) ok = mbar_wait_warp(smem_u32(&bars.buf_free[b]), ((j >> 1) - 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t dK = desc_advance(descK0, (it % NS) * Cfg::kTileBytes);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint64_t bd = desc_advance(dK, (kk >> 2) * Cfg::kSubBytes + (kk & 3) * 32);
        if (elect_one()) umma_ts(tmem + Cfg::kColS + b * kTile, tmem + Cfg::kColQ + kk * 8, bd, idesc_qk, kk > 0 ? 1u : 0u);
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bars.s_full[b]));
        umma_commit(smem_u32(&bars.kv_empty[it % NS]));   // K_j is used by S_j only
      }
      __syncwarp();
    }
  } else if (warp == 2) {
    // ---------------- O issuer: O += P_j V_j ----------------
    constexpr uint32_t idesc_pv = make_idesc_bf16(kTile, D, 0, 1);
    const uint64_t descV0 = make_smem_desc_sw128(sRing, Cfg::kSubBytes, 1024);   // V_j MN-major
    bool ok = true;
    for (int j = 0; j < n && ok; ++j) {
      const int it = 2 * j + 1, b = j & 1;
      ok = mbar_wait_warp(smem_u32(&bars.kv_full[it % NS]), (it / NS) & 1, abort);
      if (ok) ok = mbar_wait_warp(smem_u32(&bars.p_full[b]), (j >> 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t dV = desc_advance(descV0, (it % NS) * Cfg::kTileBytes);
      const uint32_t acc0 = j > 0 ? 1u : 0u;
      // packed P: keys [0,64) in columns [0,32) of the buffer, keys [64,128) in columns [64,96)
#pragma unroll
      for (int kk = 0; kk < kTile / 16; ++kk) {
        const uint64_t bd = desc_advance(dV, kk * 2048);
        if (elect_one())
          umma_ts(tmem + Cfg::kColO, tmem + Cfg::kColS + b * kTile + (kk >> 2) * 64 + (kk & 3) * 8, bd, idesc_pv,
                  kk > 0 ? 1u : acc0);
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bars.kv_empty[it % NS]));
        umma_commit(smem_u32(&bars.buf_free[b]));     // tile j+2 may overwrite the buffer
        umma_commit(smem_u32(&bars.pv_done));         // phase j: O holds tiles 0..j
      }
      __syncwarp();
    }
  } else if (warp >= 4) {
    // ---------------- softmax + epilogue: warpgroup `half` takes key columns [64*half, 64*half+64) ----------------
    const int half = (warp - 4) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t O_addr = tmem + lane_addr + Cfg::kColO + half * (D / 2);   // this thread's half of the O columns
    const int qpos = rb.q0 + row;
    const float c = a.scale_log2;
    // copy this thread's row of one 64-column sub-tile of Q from the swizzled shared-memory tile into
    // tensor memory: 16-byte chunk ch of row r sits at chunk ch ^ (r & 7)
    bool ok = mbar_wait(smem_u32(&bars.q_full), 0, abort);
    if (ok && half < Cfg::kSub) {
      const unsigned char* src = smem_raw + (sQ - smem_u32(smem_raw)) + half * Cfg::kSubBytes + row * 128;
      uint32_t v[32];
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 x = *reinterpret_cast<const uint4*>(src + ((ch ^ (row & 7)) << 4));
        v[4 * ch] = x.x; v[4 * ch + 1] = x.y; v[4 * ch + 2] = x.z; v[4 * ch + 3] = x.w;
      }
      tmem_st32(tmem + lane_addr + Cfg::kColQ + half * 32, v);
      tmem_wait_st();
    }
    tc_fence_before_sync();
    mbar_arrive(smem_u32(&bars.qt_ready));   // also when the wait gave up: the issuers then see abort
    float m = -INFINITY, l = 0.f;
    volatile unsigned short* my_loaded = &loaded_s[half][row];
    volatile unsigned short* partner_loaded = &loaded_s[1 - half][row];
    for (int j = 0; j < n && ok; ++j) {
      const int b = j & 1;
      ok = mbar_wait(smem_u32(&bars.s_full[b]), (j >> 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t S_own = tmem + lane_addr + Cfg::kColS + b * kTile + half * 64;
      const uint32_t S_oth = tmem + lane_addr + Cfg::kColS + b * kTile + (1 - half) * 64;
      uint32_t s[64], t[64];
      tmem_ld32(S_own, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
      tmem_ld32(S_own + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
      tmem_ld32(S_oth, *reinterpret_cast<uint32_t(*)[32]>(&t[0]));
      tmem_ld32(S_oth + 32, *reinterpret_cast<uint32_t(*)[32]>(&t[32]));
      tmem_wait_ld();
      *my_loaded = (unsigned short)(j + 1);   // the partner may now overwrite its S columns of this tile with P
      // keys of the tile this row may see: the first `limit`
      const int limit = j < n_ct ? rb.n_front - j * kTile : qpos - (rb.dense_start + (j - n_ct) * kTile) + 1;
      if (limit < kTile) {
        const int lim_own = limit - half * 64, lim_oth = limit - (1 - half) * 64;
#pragma unroll
        for (int i = 0; i < 64; ++i) {
          if (i >= lim_own) s[i] = 0xff800000u;  // -inf
          if (i >= lim_oth) t[i] = 0xff800000u;
        }
      }
      // row maximum over all 128 columns: both threads of a row compute the same value
      float mx0 = fmaxf(__uint_as_float(s[0]), __uint_as_float(t[0])), mx1 = fmaxf(__uint_as_float(s[1]), __uint_as_float(t[1]));
      float mx2 = fmaxf(__uint_as_float(s[2]), __uint_as_float(t[2])), mx3 = fmaxf(__uint_as_float(s[3]), __uint_as_float(t[3]));
#pragma unroll
      for (int i = 4; i < 64; i += 4) {
        mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(t[i]));
        mx1 = max3(mx1, __uint_as_float(s[i + 1]), __uint_as_float(t[i + 1]));
        mx2 = max3(mx2, __uint_as_float(s[i + 2]), __uint_as_float(t[i + 2]));
        mx3 = max3(mx3, __uint_as_float(s[i + 3]), __uint_as_float(t[i + 3]));
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      if (j == 0) {
        m = mx == -INFINITY ? 0.f : mx;
      } else {
        const bool need = (mx - m) * c > 8.f;
        if (__any_sync(0xffffffffu, need)) {
          // O must hold every earlier tile before it is rescaled; the O issuer cannot start tile j before
          // this thread has arrived on p_full, so the rescale cannot race with it
          ok = mbar_wait(smem_u32(&bars.pv_done), (j - 1) & 1, abort);
          if (!ok) break;
          tc_fence_after_sync();
          const float f = need ? ex2((m - mx) * c) : 1.f;
#pragma unroll
          for (int q = 0; q < D / 64; ++q) {
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
      float sum0, sum1;
      uint32_t pk[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        // scale and shift as packed pairs (one issue slot for two elements); one exponential in eight on
        // the FMA pipe, the rest on the MUFU pipe (measured optimum: the polynomial costs issue slots)
        float x0, x1;
        f2_unpack(f2_fma(f2_pack(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, nmc2), x0, x1);
        const float p0 = ex2(x0);
        const float p1 = (i & 3) == 3 ? ex2_fma(x1) : ex2(x1);
        sum2 = f2_add(sum2, f2_pack(p0, p1));
        pk[i] = pack_bf16(p0, p1);
      }
      f2_unpack(sum2, sum0, sum1);
      l += sum0 + sum1;
      // The two threads of a row read each other's S columns above and overwrite their own with P below:
      // a thread stores only after its partner has published that it has loaded this tile.  By now the
      // partner has had a whole tile of arithmetic to do so, so the check practically never waits.
      if ((int)*partner_loaded <= j) {
        const long long t0 = clock64();
        while ((int)*partner_loaded <= j) {
          if (*abort) { ok = false; break; }
          if (clock64() - t0 > kWaitCycles) { *abort = 1; ok = false; break; }
        }
      }
      ok = __all_sync(0xffffffffu, ok);   // one verdict per warp: the store below is warp-wide
      if (!ok) break;
      tmem_st32(S_own, pk);   // over the first half of this warpgroup's own S columns
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[b]));
    }
    red_s[half][row] = l;
    asm volatile("bar.sync 1, 256;" ::: "memory");   // the eight softmax warps, whether or not a wait gave up
    if (ok) ok = mbar_wait(smem_u32(&bars.pv_done), (n - 1) & 1, abort);
    // The output rows go through shared memory (the Q tile and the first ring slot are idle by now) and
    // leave as one bulk copy per row: per-thread 16-byte stores to rows 256 bytes apart cost a
    // transaction each.  Rows are padded by 16 bytes so that a warp's stores spread over the banks.
    constexpr int kRowBytes = D * 2, kStageStride = kRowBytes + 16;
    unsigned char* stage_out = smem_raw + (sQ - smem_u32(smem_raw));
    const bool store = qpos < rb.q_end;
    if (ok) {
      tc_fence_after_sync();
      const float lt = red_s[0][row] + red_s[1][row];
      const float inv = 1.0f / lt;
      unsigned char* srow = stage_out + row * kStageStride + half * (kRowBytes / 2);
      // the remainder goes straight to global memory (64 or 128 contiguous bytes per thread, written once)
      __nv_bfloat16* lo_row = a.Olo && store ? a.Olo + ((size_t)bh * a.N + qpos) * D + half * (D / 2) : nullptr;
#pragma unroll
      for (int q = 0; q < D / 64; ++q) {
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
      if (store && half == 0) a.LSE[(size_t)bh * a.N + qpos] = m * a.scale + logf(lt);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads these stores
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");   // both halves of every row are staged (or a wait gave up)
    if (half == 0 && store && !*abort) {
      __nv_bfloat16* orow = a.O + ((size_t)bh * a.N + qpos) * D;
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
  a.plan = make_plan(g, kTile);
  a.BH = g.B * g.Hq; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.N = g.Nrow;
  a.O = O + sh; a.Olo = Olo ? Olo + sh : nullptr; a.LSE = LSE + g.tok0; a.scale = g.scale; a.scale_log2 = g.scale * 1.4426950408889634f;
  a.status = status;
  const long long grid = (long long)a.plan.total * a.BH;
  if (grid > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  if (g.N / kTile + 4 > 0xffff) return LRSA_ERR_UNSUPPORTED;   // 16-bit tile counters of the softmax threads
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
