// Shared declarations of the PoD library's translation units (host API, write kernel,
// decode kernels).  Private to the library; the public surface is include/pod.h.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pod {

constexpr int SMALL_BATCH = 8;        // batches up to this size pass per-sequence scalars by value
constexpr int SMALL_HEADS = 16;       // up to this many KV heads pass the layer's rows of the block tables by value
constexpr int MAX_SPLITS_CAP = 128;   // upper bound of splits per sequence (partial buffers, combine)

// Shape of the split-K decode kernel (compile-time; -D overrides are for tuning builds).
#ifndef POD_DECODE_WARPS
#define POD_DECODE_WARPS 4
#endif
#ifndef POD_DECODE_STAGES
#define POD_DECODE_STAGES 3
#endif
#ifndef POD_DECODE_CTAS_PER_SM
#define POD_DECODE_CTAS_PER_SM 2
#endif
constexpr int DECODE_WARPS = POD_DECODE_WARPS;              // warps per CTA, each an independent stream
constexpr int DECODE_STAGES = POD_DECODE_STAGES;            // tiles in flight per warp
constexpr int DECODE_CTAS_PER_SM = POD_DECODE_CTAS_PER_SM;  // register budget of the kernel

// Scheduling words of one (sequence, KV head): 128 bytes apart so that heads do not share a line.
constexpr int SCHED_STRIDE = 32;      // int32 per (sequence, KV head)
constexpr int SCHED_TICKET = 16;      // [0] = chunk counter, [SCHED_TICKET] = finished-CTA tickets
constexpr int SCHED_NEED = 2;         // [SCHED_NEED] = query heads of this KV head that still need their distant tokens (gate)
constexpr int SCHED_CTR1 = 4;         // [(seq & 1) * SCHED_CTR1] = chunk counter: launches alternate between two, because a launch
                                      //   may draw chunks while the previous launch of the cache is still finishing
constexpr int SCHED_DONE = 24;        // CTAs of this head, over all launches that store logits, whose warps have finished streaming
                                      //   with valid inputs (a head that had to be recomputed counts them afterwards); own 32-byte sector

// Physical layout of the arena.  All offsets are in rows; one row is one head's d bf16
// values (128 B at d = 64, 256 B at d = 128), so every region base is 128-byte aligned.
//
// Sequence b owns a contiguous block starting at row seq_row_base[b]:
//   prox  [L][2 (K, V)][H_kv][n_s + n_r]     rows [0, n_s) = sink, row n_s + slot = ring slot
//   distV [L][H_kv][cap_d[b]]                 index p - n_s
//   distK [n_slots][cap_d[b]]                 index p - n_s, key of a block's lowest layer; one slot per
//                                             (head, block of that head), a head's slots adjacent
//   guard [32]                                only when layers share: rows that stay zero
//   score [H_kv][2][score_rows_per_head]      only when layers share: the distant logits of the block being
//                                             decoded (fp32, log2 units), one group of 16 tokens x r
//                                             query heads = r * 64 bytes in mma fragment order; two stores
//                                             per head, used in turn by the head's consecutive blocks, so
//                                             that a launch which stores the logits of the next block never
//                                             writes where the launch before it (possibly still running) reads
// with cap_d[b] = max(0, capacity[b] - n_s - n_r).  Sink and ring of one (layer, head) are
// adjacent so that the proximal tokens of a head are one contiguous stream (the softmax does
// not care about token order, so ring slots are read in slot order).
//
// Blocks are per KV head (Section 2.1, Algorithm 1): low[l][h] is the lowest layer of the block
// that holds layer l for head h, slot[l][h] the index of that block's key store.  Null tables mean
// that every layer is its own block (slot = l * H_kv + h).
struct Layout {
  int32_t L, H_kv, H_q, D, S, W, B;
  int32_t n_slots;              // key stores = (layer, head) pairs that are lowest in their block
  int32_t shared;               // 1 if some block has more than one layer
  const int64_t* seq_row_base;  // device [B]
  const int32_t* seq_cap_d;     // device [B]
  const int32_t* low;           // device [L][H_kv] or nullptr
  const int32_t* slot;          // device [L][H_kv] or nullptr
};
__device__ inline int lowest_of(const Layout& y, int layer, int head) {
  return y.low ? y.low[layer * y.H_kv + head] : layer;
}
__device__ inline int slot_of(const Layout& y, int layer, int head) {
  return y.slot ? y.slot[layer * y.H_kv + head] : layer * y.H_kv + head;
}

__host__ __device__ inline int64_t prox_row(const Layout& y, int layer, int kv /*0=K,1=V*/, int head) {
  return (((int64_t)layer * 2 + kv) * y.H_kv + head) * (int64_t)(y.S + y.W);
}
__host__ __device__ inline int64_t dist_base_row(const Layout& y) {
  return (int64_t)y.L * 2 * y.H_kv * (int64_t)(y.S + y.W);
}
__host__ __device__ inline int64_t distv_row(const Layout& y, int layer, int head, int64_t cap_d) {
  return dist_base_row(y) + ((int64_t)layer * y.H_kv + head) * cap_d;
}
__host__ __device__ inline int64_t distk_row(const Layout& y, int slot, int64_t cap_d) {
  return dist_base_row(y) + ((int64_t)y.L * y.H_kv + slot) * cap_d;
}

// Bytes of one 16-token group of shared distant logits (r query heads), and rows one head's
// groups take (a row is D bf16).
__host__ __device__ inline int score_group_bytes(const Layout& y) { return (y.H_q / y.H_kv) * 64; }
__host__ __device__ inline int64_t score_rows_per_head(const Layout& y, int64_t cap_d) {
  if (!y.shared) return 0;
  const int64_t bytes = 2 * ((cap_d + 31) / 32) * score_group_bytes(y);   // read two groups at a time
  return (bytes + y.D * 2 - 1) / (y.D * 2);
}
// Tiles of the decode kernel may extend up to 31 rows past a head's rows; everything they can
// reach must be finite bf16.  The logits are fp32 (and may be -inf), so a guard of zero rows
// separates them from the key and value rows before them.
constexpr int SCORE_GUARD_ROWS = 32;
__host__ __device__ inline int64_t score_rows_per_seq(const Layout& y, int64_t cap_d) {
  return !y.shared ? 0 : SCORE_GUARD_ROWS + 2 * y.H_kv * score_rows_per_head(y, cap_d);
}
// `kslot` is the key store of the head's block: a head's blocks have consecutive key stores, so its parity
// alternates from one block of the head to the next.
__host__ __device__ inline int64_t score_row(const Layout& y, int head, int64_t cap_d, int kslot) {
  return dist_base_row(y) + ((int64_t)y.L * y.H_kv + y.n_slots) * cap_d + SCORE_GUARD_ROWS +
         (2 * head + (kslot & 1)) * score_rows_per_head(y, cap_d);
}

// What one (sequence, KV head) of a decode launch needs to know before it can request its first tile.
// The same function fills it on the host (small launches: it then travels by value with the launch, so
// that a CTA's first requests are a handful of instructions away from its start) and on the device.
struct HeadPlan {
  int32_t n, n_p, n_d;                     // tokens held, proximal, distant
  int32_t ntp, ntd;                        // tiles of the proximal / distant tokens this launch streams
  int32_t nsplit, k_static;                // CTAs of the head; chunks per warp taken without a draw
  int32_t rowKp, rowVp, rowKd, rowVd;      // arena rows: proximal keys / values, the block's distant keys, distant values
  int32_t score_row;                       // arena row where the head's stored logits start
  int32_t kslot;                           // key store (and query stash) of the head's block
  int32_t flags;                           // HP_*
  int32_t rA, rB;                          // a launch that appends: proximal row of the new token, distant row of the
                                           // token it pushes out of the window (-1 = none)
  int32_t wait_done;                       // a head that reads stored logits: what its DONE word reads once the launch
                                           // that stored them is through with the head
};
constexpr int HP_LOW = 1;                  // this layer is the lowest of the head's block
constexpr int HP_STORE = 2;                // ... and the block goes on: the head stores its distant logits
constexpr int HP_READ = 4;                 // the head reads its block's stored logits instead of the keys
constexpr int SMALL_PLANS = 16;            // launches with up to this many (sequence, KV head) pairs carry their plans

struct PlanInputs {                        // per launch
  int32_t layer, segment, fused, max_splits, split_rows, tiles_per_chunk, static_eighths, tile_tokens, warps;
};
__host__ __device__ inline HeadPlan make_head_plan(const Layout& y, const PlanInputs& in, int kvh, int n, int64_t cap_d,
                                                   int64_t seq_row, int low_layer, int kslot, bool store, bool read) {
  HeadPlan hp;
  const int TOKS = in.tile_tokens;
  hp.n = n;
  hp.n_p = n < y.S + y.W ? n : y.S + y.W;
  hp.n_d = n - hp.n_p;
  // a gated decode streams the proximal tokens (segment 1) and the distant tokens (segment 2) in two launches
  const int n_p_s = in.segment == 2 ? 0 : hp.n_p, n_d_s = in.segment == 1 ? 0 : hp.n_d;
  const bool is_low = low_layer == in.layer;
  hp.flags = (is_low ? HP_LOW : 0) | (store ? HP_STORE : 0) | (read ? HP_READ : 0);
  hp.kslot = kslot;
  // CTAs of this head: in proportion to the rows it streams (keys and values, or values and the
  // proximal keys only), so that heads with different roles in one launch finish together.
  // (a head's rows are a fraction of the arena's, which number less than 2^31: 32-bit arithmetic)
  const uint32_t work_rows = read ? (uint32_t)n_p_s * 2u + (uint32_t)n_d_s : 2u * ((uint32_t)n_p_s + (uint32_t)n_d_s);
  const uint32_t ns = (work_rows + (uint32_t)in.split_rows - 1u) / (uint32_t)in.split_rows;
  hp.nsplit = (int32_t)(ns < (uint32_t)in.max_splits ? ns : (uint32_t)in.max_splits);
  // A head that reads stored logits needs no key rows: its distant tiles hold twice the value rows
  const int DT = read ? 2 * TOKS : TOKS;
  hp.ntp = (n_p_s + TOKS - 1) / TOKS;
  hp.ntd = (n_d_s + DT - 1) / DT;
  const uint32_t nchunks = (uint32_t)(hp.ntp + hp.ntd + in.tiles_per_chunk - 1) / (uint32_t)in.tiles_per_chunk;
  const uint32_t nwh = (uint32_t)(hp.nsplit > 0 ? hp.nsplit : 1) * (uint32_t)in.warps;
  hp.k_static = (int32_t)(nchunks / nwh) * in.static_eighths / 8;
  hp.rowKp = (int32_t)(seq_row + prox_row(y, in.layer, 0, kvh));
  hp.rowVp = (int32_t)(seq_row + prox_row(y, in.layer, 1, kvh));
  hp.rowKd = (int32_t)(seq_row + distk_row(y, kslot, cap_d));
  hp.rowVd = (int32_t)(seq_row + distv_row(y, in.layer, kvh, cap_d));
  hp.score_row = (int32_t)(seq_row + score_row(y, kvh, cap_d, kslot));
  hp.wait_done = 0;
  hp.rA = -1; hp.rB = -1;
  if (in.fused) {
    const int pos = n - 1;
    if (pos < y.S) {
      hp.rA = pos;
    } else {
      hp.rA = y.S + (pos - y.S) % y.W;
      if (pos - y.W >= y.S) hp.rB = pos - y.W - y.S;
    }
  }
  return hp;
}

struct WriteParams {
  Layout y;
  uint16_t* arena;       // bf16 bit patterns
  const uint16_t* k;     // [T][H_kv][D] (seq >= 0) or [B][H_kv][D] (seq == -1)
  const uint16_t* v;
  int32_t* len;          // device lengths of this layer, [B]
  int32_t layer, seq, n0, T;
  int32_t bulk_blocks;   // leading blocks of the grid that copy tokens going straight to the distant stores
};

struct DecodeParams {
  Layout y;
  const uint16_t* arena;
  const int32_t* len;      // device lengths of this layer, [B]
  // Append fused into the launch: one new token per sequence, k/v [B][H_kv][D]; nullptr = the
  // cache already holds the token.  len then holds the lengths before the append and the kernel
  // writes the new ones to len_out (a different array: CTAs read len at different times).
  const uint16_t* new_k;
  const uint16_t* new_v;
  int32_t* len_out;
  const uint16_t* q;       // [B][H_q][D] queries of this layer
  uint16_t* stash;         // [n_slots][B][r][D]: a head's lowest layer saves its queries for the block here
  float* part_acc;         // [B][H_q][max_splits][D]
  float* part_ml;          // [B][H_q][max_splits][4]  (running max in log2 units, sum, distant part of the sum, -)
  uint16_t* out;           // [B][H_q][D]
  int32_t* err_flag;
  unsigned long long* trace;   // nullptr, or this launch's (first CTA start, last CTA end) pair of GPU-timer nanoseconds
  int32_t* sched;          // [B][H_kv][SCHED_STRIDE] zeroed chunk counters and tickets (the kernel re-zeroes them)
  // Gate threshold (paper appendix "Computation Optimization for Distant Tokens"): a gated decode of a
  // layer is two launches.  segment 1 streams the proximal tokens only and evaluates the gate of
  // Eq. 2 per query head against the distant log-sum-exp its block's lowest layer left in dlse: heads
  // that skip (g >= gate_tau), or have no distant tokens, get their final output; the others leave
  // their proximal state (acc, max, sum) and a bit in the SCHED_NEED word.  segment 2 streams the
  // distant tokens of KV heads with a bit set and merges with that state.  segment 0 = one launch over
  // the whole context, no gate.
  int32_t segment;
  float gate_tau;
  float* dlse;             // [B][H_q] log2 of the sum of 2^logit over the distant tokens, written by a head's lowest layer
  float* state_acc;        // [B][H_q][D]
  float* state_ml;         // [B][H_q][2]
  int32_t layer, max_splits;
  int32_t split_rows;      // K or V rows a CTA should stream: a head that reads keys and values has 2 n rows of
                           // work, a head that reads stored logits n + n_p; its CTAs = ceil(work / split_rows)
  int32_t tiles_per_chunk; // tiles a warp takes per draw from the head's chunk counter
  int32_t static_eighths;  // eighths of a warp's fair share of chunks that are assigned without a draw
  float scale_log2;        // sm_scale * log2(e)
  // Small batches carry the per-sequence lengths and row offsets by value (the host mirrors the
  // device lengths exactly), which takes two dependent global loads off every CTA's start-up.
  // Shared distant logits (Section 2.2: a block shares the attention scores of its lowest layer).
  // A head for which this layer is the lowest of a block with more layers stores them; a head for
  // which it is not reads them instead of the block's keys when its bit is set here (the host sets
  // it when the stored logits are those of the head's block at these lengths), else it scores the
  // block's keys itself.  Bit h & 31 of word h >> 5; heads >= 256 never read stored logits.
  uint32_t score_read_mask[8];
  // Optimistic start.  Launches of one cache follow each other in a stream with programmatic
  // dependencies, and the tail of a launch (partials, tickets, the combine of the last CTA of a head)
  // keeps memory idle.  With optimistic = 1 (implies early_ok) a CTA does not wait for the previous
  // kernel before it streams: it reads q at once, and only before it publishes anything does it wait
  // (griddepcontrol.wait), read q again and compare.  q is the one input that the previous kernel of
  // the stream may still be writing (a projection of the caller's); a warp whose early copy turns out
  // stale marks its head, and the head's last CTA recomputes it with a plain loop (slow, exact, in
  // practice never taken).  What this launch needs from an earlier launch of the cache -- the block's
  // stored logits and stashed queries -- is awaited per head through the head's DONE word instead.
  int32_t optimistic;
  int32_t closer;          // 1: every CTA of the grid is resident at once; a head's first CTA combines and waits for the others
  int32_t seq;             // sequence number of this launch on its cache (chunk-counter parity)
  int32_t force_redo;      // test hook set from the host: every warp behaves as if its early copy of q were stale
  int32_t keep_logits;     // 1: the cache's logit stores are a small part of the L2: write and read them with evict_last
  int32_t early_ok;        // 1: no unfinished launch writes cache rows this launch streams (the two rows a
                           //    fused launch changes itself aside): tiles may be requested before the
                           //    wait for the previous kernel of the stream
  int32_t by_value;        // 1: use the arrays below instead of len / seq_row_base / seq_cap_d
  int32_t v_len[SMALL_BATCH];
  int32_t v_cap_d[SMALL_BATCH];
  int64_t v_row_base[SMALL_BATCH];
  // Few KV heads: this layer's rows of the block tables by value (low[layer][h], slot[layer][h]) and the
  // heads that store their distant logits in this launch (lowest layer of a block that goes on).
  int32_t heads_by_value;
  int32_t v_low[SMALL_HEADS];
  int32_t v_slot[SMALL_HEADS];
  uint32_t v_store_mask;
  int32_t plans_by_value;                  // 1: v_plan[b * H_kv + h] holds the plan of every (sequence, KV head)
  HeadPlan v_plan[SMALL_PLANS];
};

struct DecodePlan {
  int32_t split_rows;     // rows of work per split
  int32_t grid_splits;    // grid.x
  int32_t n_ctas;         // CTAs that do work
};

// launchers (defined in the .cu files); return a cudaError_t as int
int launch_write(const WriteParams& p, cudaStream_t s);
int launch_decode(const CUtensorMap& tmap, const DecodeParams& p, int grid_splits, cudaStream_t s);
int launch_zero_empty(const DecodeParams& p, cudaStream_t s);   // zero outputs of empty sequences
int decode_resident_ctas_per_sm(int D);   // occupancy of the split-K kernel, 0 on error
int decode_tile_tokens();                 // rows of the TMA box the split-K kernel loads
int decode_warps_per_cta();

}  // namespace pod
