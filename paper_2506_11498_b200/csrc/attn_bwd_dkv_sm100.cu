// LRSA attention backward, dK / dV part, on tcgen05 tensor cores (key-outer).
//
// The keys of one (batch, KV head) are cut into 128-row tiles of two kinds:
//   compact tiles : 128 consecutive entries of the sinks + kept-positions list (the condensed KV cache
//                   of Section 3.2, gathered from K and V by position when the CTA starts); seen by
//                   every query of the chunks that see those windows compressed
//   dense tiles   : original positions of one window (or of the sink region / the tail); seen
//                   causally by the queries from the diagonal to the end of the last chunk that
//                   still sees that window uncompressed
// A CTA takes one tile and a segment of its (64-row query tile, query head of the group) list:
//   S^T  = K_j Q_i^T     (smem x smem -> TMEM, keys on lanes)     P^T  = exp2(S^T*c - LSE_i*log2e)
//   dP^T = V_j dO_i^T    (smem x smem -> TMEM)                    dS^T = P^T * (dP^T - D_i)
//   dV  += P^T dO_i      (TMEM x smem -> TMEM)
//   dK  += dS^T Q_i      (TMEM x smem -> TMEM)
// P^T and dS^T are written back over S^T and dP^T as packed bf16; both are double-buffered so the
// tensor core computes the next S^T/dP^T while the current pair is in the softmax, on which both
// warpgroups work (32 query columns each).  Warps: 0 producer, 1-3 tensor-core issuers (S^T, dP^T,
// dV/dK), 4-11 softmax and epilogue.  The softmax warps also sum P^T * dP^T over the keys (through
// spare tensor-memory columns and a transposing load shape) and add it to a per-query-row accumulator:
// D_i = sum_j P_ij dP_ij, the accurate replacement of rowsum(dO * O) that the dQ kernel (which runs
// afterwards) needs.  The list of a tile runs from the last query tile backwards with the heads
// innermost, and compact tiles are launched segment by segment, so that the CTAs resident at one time
// read the same Q_i / dO_i tiles (L2 hits instead of one DRAM pass per key tile).  At the end
// the accumulators are added (fp32 atomics) to a zeroed workspace indexed by original position: a
// row of a compact tile goes to the position it was gathered from, so a kept key's compressed and
// uncompressed contributions meet in one row.  A small kernel then converts to bf16.
#include "attn_common_sm100.h"

namespace lrsa {
namespace {

using namespace ptx;

constexpr int kQRows = 64;    // query rows per inner tile
constexpr int kSeg = 256;     // inner iterations per CTA at most

struct DkvPlan {
  int S, L, K, N, W, T, C, Wsel, ndp, Rc, G;
  int n_cmp;       // compact tiles
  int n_sink;      // dense tiles of the sink region
  int per_win;     // dense tiles per full window
  int per_tail;    // dense tiles of the tail
  int n_tiles;
};

struct KvTile {
  int kind;      // 0 compact, 1 dense
  int row0;      // first compact row / first key position
  int key_end;   // rows at or beyond this are not part of the tile
  int qb, qend;  // query positions [qb, qend) see (part of) the tile
  int nq;        // 64-row query tiles per head
};

inline DkvPlan make_dkv_plan(const Geom& g) {
  DkvPlan p;
  p.S = g.S; p.L = g.L; p.K = g.K; p.N = g.N; p.W = g.W; p.T = g.T; p.C = g.C; p.Wsel = g.Wsel;
  p.ndp = g.ndp; p.Rc = g.Rc; p.G = g.G;
  p.n_cmp = (g.Rc + kTile - 1) / kTile;
  p.n_sink = (g.S + kTile - 1) / kTile;
  p.per_win = (g.L + kTile - 1) / kTile;
  p.per_tail = (g.T + kTile - 1) / kTile;
  p.n_tiles = p.n_cmp + p.n_sink + g.W * p.per_win + p.per_tail;
  return p;
}

__host__ __device__ inline KvTile describe_tile(const DkvPlan& p, int tile) {
  KvTile t;
  if (tile < p.n_cmp) {
    t.kind = 0;
    t.row0 = tile * kTile;
    t.key_end = p.Rc;
    int cmin = 0;
    if (t.row0 >= p.S) cmin = first_compressed_chunk((t.row0 - p.S) / p.K, p.ndp, p.Wsel, p.C);
    t.qb = p.S + cmin * p.L;
    t.qend = cmin >= p.C ? t.qb : p.N;
  } else {
    t.kind = 1;
    int d = tile - p.n_cmp;
    if (d < p.n_sink) {
      t.row0 = d * kTile; t.key_end = p.S; t.qend = p.S;
    } else {
      d -= p.n_sink;
      int w;
      if (d < p.W * p.per_win) {
        w = d / p.per_win;
        t.row0 = p.S + w * p.L + (d % p.per_win) * kTile;
        t.key_end = p.S + (w + 1) * p.L;
      } else {
        w = p.W;
        t.row0 = p.S + p.W * p.L + (d - p.W * p.per_win) * kTile;
        t.key_end = p.N;
      }
      const int cc = first_compressed_chunk(w, p.ndp, p.Wsel, p.C);
      t.qend = cc >= p.C ? p.N : (p.S + cc * p.L < p.N ? p.S + cc * p.L : p.N);
    }
    t.qb = t.row0;
  }
  t.nq = t.qend > t.qb ? (t.qend - t.qb + kQRows - 1) / kQRows : 0;
  return t;
}

__host__ __device__ inline int tile_segments(const DkvPlan& p, const KvTile& t) {
  return (p.G * t.nq + kSeg - 1) / kSeg;
}

// Launch order of the (tile, segment) pairs (one block).  Iteration i of a tile is query tile
// nq-1 - i/G (counted from the last query) of head i%G, so segment s of every compact tile covers the
// same queries of the same heads.  Compact tiles are therefore issued segment-major: the CTAs that run at
// the same time then stream the same Q_i / dO_i tiles and share them through L2 instead of fetching
// them from DRAM once per key tile.  Dense tiles (short lists, neighbours already overlap) follow in
// position order.  seg_cnt: scratch of n_tiles + 1 ints; seg_map[x] = (tile, segment of the tile).
constexpr int kMaxSegsPerTile = 2048;
__global__ void dkv_setup_kernel(const DkvPlan p, int* seg_cnt, int2* seg_map) {
  __shared__ int off[kMaxSegsPerTile + 1];   // off[s] = pairs of compact tiles with a segment index below s
  __shared__ int s_mode, s_cmp_total;
  __shared__ int run_sum[256];   // blockDim.x = 256
  for (int i = threadIdx.x; i < p.n_tiles; i += blockDim.x) seg_cnt[i] = tile_segments(p, describe_tile(p, i));
  __syncthreads();
  if (threadIdx.x == 0) {
    // segment-major order needs the compact tiles' segment counts to be non-increasing (later rows are
    // seen by later chunks only) and few enough for the table; otherwise keep tile-major order
    bool mono = p.n_cmp > 0 && seg_cnt[0] <= kMaxSegsPerTile;
    for (int c = 1; c < p.n_cmp && mono; ++c) mono = seg_cnt[c] <= seg_cnt[c - 1];
    int total = 0;
    if (mono) {
      int c = p.n_cmp;   // tiles [0, c) have more than s segments
      const int maxs = seg_cnt[0];
      for (int sgm = 0; sgm < maxs; ++sgm) {
        while (c > 0 && seg_cnt[c - 1] <= sgm) --c;
        off[sgm] = total;
        total += c;
      }
    } else {
      for (int c = 0; c < p.n_cmp; ++c) {
        for (int sgm = 0; sgm < seg_cnt[c]; ++sgm) seg_map[total + sgm] = make_int2(c, sgm);
        total += seg_cnt[c];
      }
    }
    s_mode = mono ? 1 : 0;
    s_cmp_total = total;
  }
  // dense tiles, position order: every thread takes a run of consecutive tiles
  const int nd = p.n_tiles - p.n_cmp, per = (nd + (int)blockDim.x - 1) / (int)blockDim.x;
  const int d_lo = min(p.n_tiles, p.n_cmp + (int)threadIdx.x * per), d_hi = min(p.n_tiles, d_lo + per);
  int mine = 0;
  for (int t = d_lo; t < d_hi; ++t) mine += seg_cnt[t];
  run_sum[threadIdx.x] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    int acc = s_cmp_total;
    for (int i = 0; i < (int)blockDim.x; ++i) { const int v = run_sum[i]; run_sum[i] = acc; acc += v; }
  }
  __syncthreads();
  {
    int pos = run_sum[threadIdx.x];
    for (int t = d_lo; t < d_hi; ++t) {
      for (int sgm = 0; sgm < seg_cnt[t]; ++sgm) seg_map[pos + sgm] = make_int2(t, sgm);
      pos += seg_cnt[t];
    }
  }
  if (s_mode) {
    for (int c = threadIdx.x; c < p.n_cmp; c += blockDim.x)
      for (int sgm = 0; sgm < seg_cnt[c]; ++sgm) seg_map[off[sgm] + c] = make_int2(c, sgm);
  }
}

template <int D>
struct DkvCfg {
  static constexpr int kSub = D / 64;
  static constexpr int kKSubBytes = kTile * 128;            // 128 key rows x 128 bytes
  static constexpr int kKTileBytes = kSub * kKSubBytes;     // K_j or V_j
  static constexpr int kQSubBytes = kQRows * 128;           // 64 query rows x 128 bytes
  static constexpr int kQTileBytes = kSub * kQSubBytes;     // Q_i or dO_i
  static constexpr int kStageBytes = 2 * kQTileBytes;       // Q_i + dO_i
  static constexpr int kStages = D == 128 ? 4 : 8;
  static constexpr int kSmem = 2 * kKTileBytes + kStages * kStageBytes + 1024;
  static constexpr int kThreads = 384;   // producer, three MMA issuers, eight softmax warps
  static constexpr uint32_t kColS = 0, kColP = 128, kColK = 256, kColV = 256 + D;
};

struct DkvArgs {
  DkvPlan plan;
  int BHkv, Hq, Hkv, total_segs;
  const int32_t* idx;    // kept positions of this sequence's windows: head bh at idx + bh * kept_stride
  int kept_stride;       // Wtot * K entries per (batch, KV head)
  int Nrow, tok0;        // tokens per (batch, head) row (the stride of every tensor); first token of the sequence
  const float2* stats;   // per query row: (-LSE * log2(e), D~ = rowsum(dO * O) from the bf16 O)
  float* Dacc;           // [B*Hq][N], zeroed: receives sum_j P_tj dP_tj, the accurate D for the dQ kernel
  const int2* seg_map;   // launch order: (tile, segment of the tile)
  float* dKf;   // [BHkv][N][D] fp32, zeroed
  float* dVf;
  float scale, scale_log2;
  int* status;
};

struct DkvBars {
  uint64_t kv_full, acc_done;
  uint64_t ring_full[8], ring_empty[8];
  uint64_t s_full[2], p_full[2], buf_free[2], red_done[2];
};

__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int D>
__global__ void __launch_bounds__(DkvCfg<D>::kThreads, 1)
lrsa_bwd_dkv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapdO,
                    const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                    const __grid_constant__ CUtensorMap mapKg, const __grid_constant__ CUtensorMap mapVg,
                    const DkvArgs a) {
  using Cfg = DkvCfg<D>;
  constexpr int NS = Cfg::kStages;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) DkvBars bars;
  __shared__ __align__(16) float st_nl2[NS][kQRows];   // -LSE*log2(e) per query row of the stage (-inf: not seen)
  __shared__ __align__(16) float st_D[NS][kQRows];
  __shared__ int st_meta[NS][4];             // compact tiles: compact rows visible to the stage's first chunk,
                                             // first column of its second chunk, rows visible to that chunk
  __shared__ int st_q0[NS], st_hq[NS];       // first query position and query head of the stage (computed once,
                                             // by the producer: an integer division per thread and tile is costly)
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sK = smem0, sV = smem0 + Cfg::kKTileBytes, sRing = smem0 + 2 * Cfg::kKTileBytes;

  // ---- which tile, which segment ----
  const DkvPlan& p = a.plan;
  const int bh_kv = blockIdx.x % a.BHkv, seg = blockIdx.x / a.BHkv;
  const int2 ts = a.seg_map[seg];
  const KvTile kt = describe_tile(p, ts.x);
  const int it_begin = ts.y * kSeg;
  const int n = min(kSeg, p.G * kt.nq - it_begin);
  const int hq0 = (bh_kv / a.Hkv) * a.Hq + (bh_kv % a.Hkv) * p.G;   // first query head of the group

  if (tid == 0) {
    abort_s = 0;
    mbar_init(smem_u32(&bars.kv_full), 1);
    mbar_init(smem_u32(&bars.acc_done), 1);
    for (int i = 0; i < NS; ++i) { mbar_init(smem_u32(&bars.ring_full[i]), 1); mbar_init(smem_u32(&bars.ring_empty[i]), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars.s_full[b]), 2);      // the S^T issuer and the dP^T issuer
      mbar_init(smem_u32(&bars.p_full[b]), 256);    // every softmax thread
      mbar_init(smem_u32(&bars.buf_free[b]), 1);
      mbar_init(smem_u32(&bars.red_done[b]), 256);  // every softmax thread has read its scratch columns back
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
    // ---------------- producer (whole warp: lanes stage LSE and D, lane 0 drives TMA) ----------------
    if (lane == 0) {
      prefetch_tensormap(&mapQ); prefetch_tensormap(&mapdO);
      mbar_expect_tx(smem_u32(&bars.kv_full), 2 * Cfg::kKTileBytes);
    }
    __syncwarp();
    if (kt.kind == 0) {
      // every lane gathers four rows of the list tile from their positions in K and V
      const int32_t* kept = a.idx + (size_t)bh_kv * a.kept_stride;
      int pos[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        pos[i] = bh_kv * a.Nrow + compact_row_pos(kept, p.S, p.Rc, kt.row0 + 4 * lane + i, a.tok0);
      for (int h = 0; h < Cfg::kSub; ++h) {
        tma_gather4_2d(sK + h * Cfg::kKSubBytes + lane * 512, &mapKg, h * 64, pos[0], pos[1], pos[2], pos[3], smem_u32(&bars.kv_full));
        tma_gather4_2d(sV + h * Cfg::kKSubBytes + lane * 512, &mapVg, h * 64, pos[0], pos[1], pos[2], pos[3], smem_u32(&bars.kv_full));
      }
    } else if (lane == 0) {
      for (int h = 0; h < Cfg::kSub; ++h) {
        tma_load_3d(sK + h * Cfg::kKSubBytes, &mapK, h * 64, kt.row0, bh_kv, smem_u32(&bars.kv_full));
        tma_load_3d(sV + h * Cfg::kKSubBytes, &mapV, h * 64, kt.row0, bh_kv, smem_u32(&bars.kv_full));
      }
    }
    bool ok = true;
    int it = 0;
    // per-row statistics of a stage are fetched one stage ahead, so that their latency overlaps the
    // wait for a free slot instead of adding to it
    // iteration gi: query tile nq-1 - gi/G (from the last query backwards) of head gi % G
    int qt = kt.nq - 1 - it_begin / p.G, hd = it_begin % p.G;
    auto fetch = [&](int qt_, int hd_, float2 (&v)[kQRows / 32]) {
      const int hq = hq0 + hd_, q0 = kt.qb + qt_ * kQRows;
#pragma unroll
      for (int k = 0; k < kQRows / 32; ++k) {
        const int q = q0 + lane + 32 * k;
        v[k] = q < kt.qend ? __ldg(a.stats + (size_t)hq * a.Nrow + q) : make_float2(-INFINITY, 0.f);
      }
    };
    float2 cur[kQRows / 32], nxt[kQRows / 32];
    if (n > 0) fetch(qt, hd, cur);
    for (; it < n; ++it) {
      const int slot = it % NS, use = it / NS;
      int qt_n = qt, hd_n = hd + 1;
      if (hd_n == p.G) { hd_n = 0; --qt_n; }
      if (it + 1 < n) fetch(qt_n, hd_n, nxt);
      if (use > 0 && lane == 0) ok = mbar_wait(smem_u32(&bars.ring_empty[slot]), (use - 1) & 1, abort);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const int hq = hq0 + hd, q0 = kt.qb + qt * kQRows;
#pragma unroll
      for (int k = 0; k < kQRows / 32; ++k) {
        st_nl2[slot][lane + 32 * k] = cur[k].x;
        st_D[slot][lane + 32 * k] = cur[k].y;
        cur[k] = nxt[k];
      }
      if (lane == 0) { st_q0[slot] = q0; st_hq[slot] = hq; }
      if (lane == 0 && kt.kind == 0) {
        const int cch = (q0 - p.S) / p.L;
        st_meta[slot][0] = p.S + n_hist_windows(cch, p.ndp, p.Wsel) * p.K;
        st_meta[slot][1] = min(kQRows, p.S + (cch + 1) * p.L - q0);
        st_meta[slot][2] = p.S + n_hist_windows(cch + 1, p.ndp, p.Wsel) * p.K;
      }
      __syncwarp();
      if (lane == 0) {
        const uint32_t full = smem_u32(&bars.ring_full[slot]);
        mbar_expect_tx(full, Cfg::kStageBytes);
        const uint32_t dst = sRing + slot * Cfg::kStageBytes;
        for (int h = 0; h < Cfg::kSub; ++h) {
          tma_load_3d(dst + h * Cfg::kQSubBytes, &mapQ, h * 64, q0, hq, full);
          tma_load_3d(dst + Cfg::kQTileBytes + h * Cfg::kQSubBytes, &mapdO, h * 64, q0, hq, full);
        }
      }
      qt = qt_n; hd = hd_n;
    }
    if (!ok && lane == 0) {
      for (int back = 1; back <= NS && back <= it; ++back) {
        const int i2 = it - back;
        const long long t0 = clock64();
        while (!mbar_try_wait(smem_u32(&bars.ring_full[i2 % NS]), (i2 / NS) & 1) && clock64() - t0 < 2000000) {}
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ---------------- S^T issuer (warp 1: K_j Q_i^T) and dP^T issuer (warp 2: V_j dO_i^T) ----------------
    // Each issuing warp runs its loop with all lanes (uniform control flow, descriptors computed once)
    // and elects one lane per instruction.
    const int which = warp - 1;
    constexpr uint32_t idesc_s = make_idesc_bf16(kTile, kQRows, 0, 0);  // 128 keys x 64 queries
    const uint64_t descA = make_smem_desc_sw128(which == 0 ? sK : sV, 16, 1024);
    const uint64_t descR = make_smem_desc_sw128(sRing + which * Cfg::kQTileBytes, 16, 1024);   // K-major Q_i / dO_i
    bool ok = mbar_wait_warp(smem_u32(&bars.kv_full), 0, abort);
    for (int it = 0; it < n && ok; ++it) {
      const int slot = it % NS, b = it & 1;
      ok = mbar_wait_warp(smem_u32(&bars.ring_full[slot]), (it / NS) & 1, abort);
      if (ok && it >= 2) ok = mbar_wait_warp(smem_u32(&bars.buf_free[b]), ((it >> 1) - 1) & 1, abort);
      if (ok && it >= 2) ok = mbar_wait_warp(smem_u32(&bars.red_done[b]), ((it >> 1) - 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem + (which == 0 ? Cfg::kColS : Cfg::kColP) + b * kQRows;
      const uint64_t dB = desc_advance(descR, slot * Cfg::kStageBytes);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t koff = (kk >> 2) * Cfg::kKSubBytes + (kk & 3) * 32;
        const uint32_t qoff = (kk >> 2) * Cfg::kQSubBytes + (kk & 3) * 32;
        const uint64_t ad = desc_advance(descA, koff), bd = desc_advance(dB, qoff);
        if (elect_one()) umma_ss(d_tmem, ad, bd, idesc_s, kk > 0 ? 1u : 0u);
      }
      if (elect_one()) umma_commit(smem_u32(&bars.s_full[b]));
      __syncwarp();
    }
  } else if (warp == 3) {
    // ---------------- dV / dK issuer ----------------
    constexpr uint32_t idesc_a = make_idesc_bf16(kTile, D, 0, 1);       // 128 keys x D
    const uint64_t descRmn = make_smem_desc_sw128(sRing, Cfg::kQSubBytes, 1024);     // MN-major Q_i / dO_i
    bool ok = true;
    for (int it = 0; it < n && ok; ++it) {
      const int slot = it % NS, b = it & 1;
      ok = mbar_wait_warp(smem_u32(&bars.p_full[b]), (it >> 1) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint64_t dQi = desc_advance(descRmn, slot * Cfg::kStageBytes);
      const uint64_t ddOi = desc_advance(dQi, Cfg::kQTileBytes);
      const uint32_t acc0 = it > 0 ? 1u : 0u;
      // packed P^T / dS^T: queries [0,32) in columns [0,16) of the buffer, queries [32,64) in columns [32,48)
#pragma unroll
      for (int kk = 0; kk < kQRows / 16; ++kk) {
        const uint64_t bd = desc_advance(ddOi, kk * 2048);
        if (elect_one())
          umma_ts(tmem + Cfg::kColV, tmem + Cfg::kColS + b * kQRows + (kk >> 1) * 32 + (kk & 1) * 8, bd, idesc_a,
                  kk > 0 ? 1u : acc0);
      }
#pragma unroll
      for (int kk = 0; kk < kQRows / 16; ++kk) {
        const uint64_t bd = desc_advance(dQi, kk * 2048);
        if (elect_one())
          umma_ts(tmem + Cfg::kColK, tmem + Cfg::kColP + b * kQRows + (kk >> 1) * 32 + (kk & 1) * 8, bd, idesc_a,
                  kk > 0 ? 1u : acc0);
      }
      if (elect_one()) {
        umma_commit(smem_u32(&bars.ring_empty[slot]));
        umma_commit(smem_u32(&bars.buf_free[b]));      // tile it+2 may overwrite the buffer
      }
      __syncwarp();
    }
    if (ok && elect_one()) umma_commit(smem_u32(&bars.acc_done));
    __syncwarp();
  } else {
    // ---------------- P^T / dS^T: warpgroup `wg` takes query columns [32*wg, 32*wg+32) of every tile ----------------
    const int wg = (warp - 4) >> 2, quad = warp & 3;
    const int r = quad * 32 + lane;            // key row of this thread inside the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const float c = a.scale_log2;
    const bool key_ok = kt.row0 + r < kt.key_end;
    bool ok = true;
    for (int it = 0; it < n; ++it) {
      const int slot = it % NS, b = it & 1;
      ok = mbar_wait(smem_u32(&bars.s_full[b]), (it >> 1) & 1, abort);
      if (ok) ok = mbar_wait(smem_u32(&bars.ring_full[slot]), (it / NS) & 1, abort);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t S_addr = tmem + lane_addr + Cfg::kColS + b * kQRows + wg * 32;
      const uint32_t P_addr = tmem + lane_addr + Cfg::kColP + b * kQRows + wg * 32;
      uint32_t s[32], dp[32];
      tmem_ld32(S_addr, s);
      tmem_ld32(P_addr, dp);
      tmem_wait_ld();
      // first query column of this tile that sees this thread's key (64 = none)
      const int q0 = st_q0[slot], hq = st_hq[slot];
      int lo;
      if (!key_ok) {
        lo = kQRows;
      } else if (kt.kind == 1) {
        lo = kt.row0 + r - q0;                      // causal: query position >= key position
      } else if (p.L >= kQRows) {                   // compact row, tile spans at most two chunks
        const int cr = kt.row0 + r;
        lo = cr < st_meta[slot][0] ? 0 : (cr < st_meta[slot][2] ? st_meta[slot][1] : kQRows);
      } else {
        const int cr = kt.row0 + r;                 // compact row: needs cr < S + n_hist(chunk)*K
        lo = kQRows;
        int col = 0;
        while (col < kQRows) {
          const int cch = (q0 + col - p.S) / p.L;
          if (cr < p.S + n_hist_windows(cch, p.ndp, p.Wsel) * p.K) { lo = col; break; }
          col = p.S + (cch + 1) * p.L - q0;         // first column of the next chunk
        }
      }
      lo -= wg * 32;
      if (lo > 0) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (i < lo) s[i] = 0xff800000u;
      }
      const float4* nl2v = reinterpret_cast<const float4*>(st_nl2[slot] + wg * 32);
      const float4* Dv = reinterpret_cast<const float4*>(st_D[slot] + wg * 32);
      uint32_t pp[16], ds[16];
      float x[32];   // P * dP, whose sum over the keys is the accurate D of the query column
      {
        // packed fp32 pairs: one issue slot for two elements of every multiply-add below
        const uint64_t c2 = f2_pack(c, c);
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          const float4 nl = nl2v[v], dd = Dv[v];
          float a0, a1, a2, a3, d0, d1, d2, d3;
          f2_unpack(f2_fma(f2_pack(__uint_as_float(s[4 * v + 0]), __uint_as_float(s[4 * v + 1])), c2, f2_pack(nl.x, nl.y)), a0, a1);
          f2_unpack(f2_fma(f2_pack(__uint_as_float(s[4 * v + 2]), __uint_as_float(s[4 * v + 3])), c2, f2_pack(nl.z, nl.w)), a2, a3);
          const float p0 = ex2(a0), p1 = ex2(a1), p2 = ex2(a2), p3 = ex2(a3);
          pp[2 * v] = pack_bf16(p0, p1);
          pp[2 * v + 1] = pack_bf16(p2, p3);
          const uint64_t p01 = f2_pack(p0, p1), p23 = f2_pack(p2, p3);
          const uint64_t x01 = f2_mul(p01, f2_pack(__uint_as_float(dp[4 * v + 0]), __uint_as_float(dp[4 * v + 1])));
          const uint64_t x23 = f2_mul(p23, f2_pack(__uint_as_float(dp[4 * v + 2]), __uint_as_float(dp[4 * v + 3])));
          f2_unpack(x01, x[4 * v + 0], x[4 * v + 1]);
          f2_unpack(x23, x[4 * v + 2], x[4 * v + 3]);
          f2_unpack(f2_fma(p01, f2_pack(-dd.x, -dd.y), x01), d0, d1);   // dS = P dP - P D
          f2_unpack(f2_fma(p23, f2_pack(-dd.z, -dd.w), x23), d2, d3);
          ds[2 * v] = pack_bf16(d0, d1);
          ds[2 * v + 1] = pack_bf16(d2, d3);
        }
      }
      tmem_st16(S_addr, pp);   // over the first half of this warpgroup's own columns
      tmem_st16(P_addr, ds);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bars.p_full[b]));
      // Off the tensor core's critical path: sum x over the warp's 32 keys.  The values go through the
      // upper halves of this warpgroup's own S^T and dP^T columns (free once P^T and dS^T are packed into
      // the lower halves; the issuers wait for red_done before the buffer is written again) and come back
      // with the 16-lane x 256-bit load shape, which hands every thread four key rows of eight query
      // columns; the remaining three levels are register exchanges.  (A full five-level exchange in
      // registers costs twice the instructions, and shuffles share the shared-memory pipe with the
      // tensor core's operand reads.)
      {
        uint32_t xa[16], xb[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) { xa[i] = __float_as_uint(x[i]); xb[i] = __float_as_uint(x[16 + i]); }
        tmem_st16(S_addr + 16, xa);
        tmem_st16(P_addr + 16, xb);
        tmem_wait_st();
        uint32_t ra0[8], ra1[8], rb0[8], rb1[8];
        tmem_ld_16x256b_x2(S_addr + 16, ra0);
        tmem_ld_16x256b_x2(S_addr + 16 + (16u << 16), ra1);
        tmem_ld_16x256b_x2(P_addr + 16, rb0);
        tmem_ld_16x256b_x2(P_addr + 16 + (16u << 16), rb1);
        tmem_wait_ld();
        tc_fence_before_sync();
        mbar_arrive(smem_u32(&bars.red_done[b]));
        float c8[8];   // index 4B + 2j + e: column 16B + 8j + 2(lane%4) + e of the warpgroup's 32
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            c8[2 * j + e] = (__uint_as_float(ra0[4 * j + e]) + __uint_as_float(ra0[4 * j + 2 + e])) +
                            (__uint_as_float(ra1[4 * j + e]) + __uint_as_float(ra1[4 * j + 2 + e]));
            c8[4 + 2 * j + e] = (__uint_as_float(rb0[4 * j + e]) + __uint_as_float(rb0[4 * j + 2 + e])) +
                                (__uint_as_float(rb1[4 * j + e]) + __uint_as_float(rb1[4 * j + 2 + e]));
          }
#pragma unroll
        for (int m = 4, bit = 16; m >= 1; m >>= 1, bit >>= 1) {
          const bool up = (lane & bit) != 0;
#pragma unroll
          for (int i = 0; i < m; ++i) {
            const float send = up ? c8[i] : c8[i + m];
            const float keep = up ? c8[i + m] : c8[i];
            c8[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
          }
        }
        const int col = 16 * ((lane >> 4) & 1) + 8 * ((lane >> 3) & 1) + 2 * (lane & 3) + ((lane >> 2) & 1);
        const int q = q0 + wg * 32 + col;
        if (q < kt.qend) atomicAdd(a.Dacc + (size_t)hq * a.Nrow + q, c8[0]);
      }
    }
    if (ok) ok = mbar_wait(smem_u32(&bars.acc_done), 0, abort);
    if (ok) {
      tc_fence_after_sync();
      // warpgroup 0 adds dK (scaled), warpgroup 1 adds dV
      const uint32_t acc = tmem + lane_addr + (wg == 0 ? Cfg::kColK : Cfg::kColV);
      const float mul = wg == 0 ? a.scale : 1.0f;
      // a row of a compact tile lands on the position it was gathered from
      const int out_row = kt.kind == 0
                              ? compact_row_pos(a.idx + (size_t)bh_kv * a.kept_stride, p.S, p.Rc, kt.row0 + r, a.tok0)
                              : kt.row0 + r;
      float* dst = (wg == 0 ? a.dKf : a.dVf) + ((size_t)bh_kv * a.Nrow + out_row) * D;
#pragma unroll
      for (int q = 0; q < D / 32; ++q) {
        uint32_t o[32];
        tmem_ld32(acc + q * 32, o);
        tmem_wait_ld();
        if (key_ok) {
#pragma unroll
          for (int v = 0; v < 8; ++v)
            red_add_v4(dst + q * 32 + v * 4, __uint_as_float(o[4 * v]) * mul, __uint_as_float(o[4 * v + 1]) * mul,
                       __uint_as_float(o[4 * v + 2]) * mul, __uint_as_float(o[4 * v + 3]) * mul);
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
  if (tid == 0 && abort_s) atomicExch(a.status, (int)LRSA_ERR_TIMEOUT);
}

// bf16 outputs from the fp32 accumulators [BHkv][N][d]; n4 = number of float4 groups
__global__ void convert_dkv_kernel(const float* __restrict__ dKf, const float* __restrict__ dVf,
                                   __nv_bfloat16* __restrict__ dK, __nv_bfloat16* __restrict__ dV, long long n4) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const long long e = i * 4;
  const float4 k = *reinterpret_cast<const float4*>(dKf + e);
  const float4 v = *reinterpret_cast<const float4*>(dVf + e);
  uint2 ko, vo;
  ko.x = pack_bf16(k.x, k.y); ko.y = pack_bf16(k.z, k.w);
  vo.x = pack_bf16(v.x, v.y); vo.y = pack_bf16(v.z, v.w);
  *reinterpret_cast<uint2*>(dK + e) = ko;
  *reinterpret_cast<uint2*>(dV + e) = vo;
}

}  // namespace

static int dkv_total_segs(const DkvPlan& p) {
  int total = 0;
  for (int i = 0; i < p.n_tiles; ++i) total += tile_segments(p, describe_tile(p, i));
  return total;
}

// Layout: [segment counts: n_tiles + 1 ints][launch order: total_segs int2][dK fp32][dV fp32]
size_t dkv_ws_bytes(const Geom& g, size_t* prefix_bytes) {
  const DkvPlan p = make_dkv_plan(g);
  const size_t cnt = align_up((size_t)(p.n_tiles + 1) * sizeof(int), 1024);
  const size_t pre = cnt + align_up((size_t)(dkv_total_segs(p) + 1) * sizeof(int2), 1024);
  if (prefix_bytes) *prefix_bytes = pre;
  const size_t acc = align_up((size_t)g.B * g.Hkv * g.Nrow * g.d * sizeof(float), 1024);
  return pre + 2 * acc;
}

template <int D>
static int launch_dkv_t(const Geom& g, const DkvArgs& a, const CUtensorMap* m, cudaStream_t st) {
  using Cfg = DkvCfg<D>;
  auto kern = lrsa_bwd_dkv_kernel<D>;
  LRSA_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem));
  const long long grid = (long long)a.total_segs * a.BHkv;
  if (grid > 0x7fffffffLL) return LRSA_ERR_UNSUPPORTED;
  if (grid == 0) return LRSA_OK;
  kern<<<(unsigned)grid, Cfg::kThreads, Cfg::kSmem, st>>>(m[0], m[1], m[2], m[3], m[4], m[5], a);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

// ws_dkv: region of dkv_ws_bytes(whole row) bytes.  Three steps: dkv_zero clears the fp32 accumulators of
// the whole row, launch_bwd_dkv_sm100 runs the tile kernel of one sequence (its launch-order table is
// rebuilt in the region's prefix, in stream order), dkv_convert writes bf16 dK, dV.
static void dkv_regions(const Geom& whole, void* ws_dkv, int** seg_cnt, int2** seg_map, float** dKf, float** dVf,
                        size_t* acc_bytes) {
  size_t pre = 0;
  const size_t total = dkv_ws_bytes(whole, &pre);
  unsigned char* base = static_cast<unsigned char*>(ws_dkv);
  const DkvPlan p = make_dkv_plan(whole);
  *acc_bytes = (total - pre) / 2;
  *seg_cnt = reinterpret_cast<int*>(base);
  *seg_map = reinterpret_cast<int2*>(base + align_up((size_t)(p.n_tiles + 1) * sizeof(int), 1024));
  *dKf = reinterpret_cast<float*>(base + pre);
  *dVf = reinterpret_cast<float*>(base + pre + *acc_bytes);
}

int dkv_zero(const Geom& whole, void* ws_dkv, cudaStream_t st) {
  int* seg_cnt; int2* seg_map; float *dKf, *dVf; size_t acc;
  dkv_regions(whole, ws_dkv, &seg_cnt, &seg_map, &dKf, &dVf, &acc);
  LRSA_CUDA_CHECK(cudaMemsetAsync(dKf, 0, 2 * acc, st));
  launch_counter().n++;
  return LRSA_OK;
}

int dkv_convert(const Geom& whole, void* ws_dkv, __nv_bfloat16* dK, __nv_bfloat16* dV, cudaStream_t st) {
  int* seg_cnt; int2* seg_map; float *dKf, *dVf; size_t acc;
  dkv_regions(whole, ws_dkv, &seg_cnt, &seg_map, &dKf, &dVf, &acc);
  const long long n4 = (long long)whole.B * whole.Hkv * whole.Nrow * whole.d / 4;
  convert_dkv_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(dKf, dVf, dK, dV, n4);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  return LRSA_OK;
}

// `whole`: the geometry of the whole row (workspace layout); `g`: the sequence to process.
int launch_bwd_dkv_sm100(const Geom& whole, const Geom& g, const __nv_bfloat16* Q, const __nv_bfloat16* dO,
                         const __nv_bfloat16* K, const __nv_bfloat16* V, const float2* stats, float* Dacc,
                         const int32_t* idx, void* ws_dkv, int* status, cudaStream_t st) {
  const DkvPlan p = make_dkv_plan(g);
  int* seg_cnt; int2* seg_map; float *dKf, *dVf; size_t acc;
  dkv_regions(whole, ws_dkv, &seg_cnt, &seg_map, &dKf, &dVf, &acc);
  // a part of a row never needs more than the whole row; checked all the same
  if (p.n_tiles > make_dkv_plan(whole).n_tiles || dkv_total_segs(p) > dkv_total_segs(make_dkv_plan(whole)))
    return LRSA_ERR_WORKSPACE_TOO_SMALL;
  dkv_setup_kernel<<<1, 256, 0, st>>>(p, seg_cnt, seg_map);
  LRSA_CUDA_CHECK(cudaGetLastError());
  launch_counter().n++;
  const int total_segs = dkv_total_segs(p);

  CUtensorMap m[6];
  const size_t sh = (size_t)g.tok0 * g.d;
  int r = make_tmap_bf16(&m[0], Q + sh, g.d, g.N, (long long)g.B * g.Hq, kQRows, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&m[1], dO + sh, g.d, g.N, (long long)g.B * g.Hq, kQRows, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&m[2], K + sh, g.d, g.N, (long long)g.B * g.Hkv, kTile, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16(&m[3], V + sh, g.d, g.N, (long long)g.B * g.Hkv, kTile, g.Nrow);
  if (r == LRSA_OK) r = make_tmap_bf16_rows(&m[4], K + sh, g.d, (long long)g.B * g.Hkv * g.Nrow - g.tok0);
  if (r == LRSA_OK) r = make_tmap_bf16_rows(&m[5], V + sh, g.d, (long long)g.B * g.Hkv * g.Nrow - g.tok0);
  if (r != LRSA_OK) return r;
  DkvArgs a;
  a.plan = p; a.BHkv = g.B * g.Hkv; a.Hq = g.Hq; a.Hkv = g.Hkv; a.total_segs = total_segs;
  a.idx = idx + (size_t)g.woff * g.K; a.kept_stride = g.Wtot * g.K; a.Nrow = g.Nrow; a.tok0 = g.tok0;
  a.stats = stats + g.tok0; a.Dacc = Dacc + g.tok0; a.seg_map = seg_map; a.dKf = dKf + sh; a.dVf = dVf + sh;
  a.scale = g.scale; a.scale_log2 = g.scale * 1.4426950408889634f; a.status = status;
  return g.d == 128 ? launch_dkv_t<128>(g, a, m, st) : launch_dkv_t<64>(g, a, m, st);
}

}  // namespace lrsa
