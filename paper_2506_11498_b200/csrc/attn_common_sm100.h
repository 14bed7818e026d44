// Pieces shared by the tensor-core attention kernels: bounded mbarrier waits, the row-block
// decomposition of the chunked mask (Section 3.2, Attn-Fill 1/2), TMA descriptor creation.
#pragma once

#include "lrsa_internal.h"
#include "sm100_ptx.h"

namespace lrsa {

constexpr int kTile = 128;                 // rows of a query tile, keys of a key tile
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s at 2 GHz: no wait in a correct run gets close

// Waits for the phase with the given parity; gives up (returns false, raises *abort) when another
// thread of the CTA has given up or after kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort) return false;
      if (clock64() - t0 > kWaitCycles) { *abort = 1; return false; }
    }
  }
}

// The same wait executed by all 32 lanes of a converged warp, with one verdict for the warp.  The
// warps that issue tcgen05.mma run in warp-uniform control flow with descriptors computed once
// outside the loops (building a descriptor per instruction in a single-lane branch costs ~100
// cycles per MMA, more than the MMA itself) and elect one lane per instruction.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort) {
  const bool ok = mbar_wait(bar, parity, abort);
  return __all_sync(0xffffffffu, ok);
}

// A block of query rows that share one key list: rows [q0, q_end) (at most `rows_per_block`), all in
// one query chunk (or the sink region).  Their keys are the first n_front rows of the compact
// (sinks + kept) buffer followed by original positions [dense_start, own position].
struct RowBlock {
  int q0, q_end;      // query rows of this block
  int n_front;        // compact rows visible: S + n_c*K (0 for sink queries)
  int dense_start;    // first position of the contiguous key range
};

struct BlockPlan {
  int S, L, K, N, W, T, Wsel, ndp;
  int rows;           // rows per block (128 or 256)
  int per_chunk;      // blocks per full chunk
  int per_tail;       // blocks of the tail chunk
  int per_sink;       // blocks of the sink region
  int total;          // per (batch, head)
};

inline BlockPlan make_plan(const Geom& g, int rows) {
  BlockPlan p;
  p.S = g.S; p.L = g.L; p.K = g.K; p.N = g.N; p.W = g.W; p.T = g.T; p.Wsel = g.Wsel; p.ndp = g.ndp;
  p.rows = rows;
  p.per_chunk = (g.L + rows - 1) / rows;
  p.per_tail = (g.T + rows - 1) / rows;
  p.per_sink = (g.S + rows - 1) / rows;
  p.total = g.W * p.per_chunk + p.per_tail + p.per_sink;
  return p;
}

// Blocks are numbered heaviest first: tail chunk, then full chunks from the last to the first (inside
// a chunk from the last rows to the first), then the sink region.
__device__ __forceinline__ RowBlock decode_block(const BlockPlan& p, int blk) {
  RowBlock r;
  int c, i;
  if (blk < p.per_tail) {
    c = p.W; i = p.per_tail - 1 - blk;
  } else if (blk < p.per_tail + p.W * p.per_chunk) {
    blk -= p.per_tail;
    c = p.W - 1 - blk / p.per_chunk;
    i = p.per_chunk - 1 - blk % p.per_chunk;
  } else {
    i = blk - p.per_tail - p.W * p.per_chunk;
    r.q0 = i * p.rows;
    r.q_end = min(p.S, r.q0 + p.rows);
    r.n_front = 0;
    r.dense_start = 0;
    return r;
  }
  const int c0 = p.S + c * p.L;
  const int c1 = min(p.N, c0 + p.L);
  r.q0 = c0 + i * p.rows;
  r.q_end = min(c1, r.q0 + p.rows);
  const int nh = n_hist_windows(c, p.ndp, p.Wsel);
  r.n_front = p.S + nh * p.K;
  r.dense_start = p.S + nh * p.L;
  return r;
}

// 3-D bf16 tensor map over [outer][rows][d] with a (64 x box_rows x 1) box and 128-byte swizzle.
// `row_stride`: rows between consecutive `outer` slices in memory (0: rows); larger when the map covers
// one sequence of a packed row.
int make_tmap_bf16(CUtensorMap* map, const void* base, int d, long long rows, long long outer, int box_rows,
                   long long row_stride = 0);

// Gathers the sink rows and the kept rows of K and V into the compact buffers
// Kc, Vc [B*Hkv][Rc][d] (the condensed KV cache of Section 3.2) for the query-outer kernels, which
// stream the list once per query tile: a TMA row gather in their main loops was measured at about
// 6 bytes per clock and SM, a fifth of what they consume.
int launch_compact_kv(const Geom& g, const __nv_bfloat16* K, const __nv_bfloat16* V, const int32_t* idx,
                      __nv_bfloat16* Kc, __nv_bfloat16* Vc, cudaStream_t st);

// 2-D bf16 tensor map over [rows][d] with a (64 x 1) box and 128-byte swizzle, for row gathers
// (tile::gather4).  The key-outer dK/dV kernel loads its one list tile per CTA this way, four rows per
// copy, straight from K and V into the swizzled operand tile.
int make_tmap_bf16_rows(CUtensorMap* map, const void* base, int d, long long rows);

// Original position of row r of the compact (sinks + kept) key list of one (batch, KV head); `kept`
// points at that head's idx entries.  Rows at or beyond n_rows are never used by a product (their scores
// are masked); they map to position 0 so that the row fetched for them is valid, finite data.
// Positions are local to the sequence (kept entries are positions in the whole row, tok0 + local).
__device__ __forceinline__ int compact_row_pos(const int32_t* __restrict__ kept, int S, int n_rows, int r, int tok0) {
  if (r >= n_rows) return 0;
  return r < S ? r : __ldg(kept + (r - S)) - tok0;
}

}  // namespace lrsa
