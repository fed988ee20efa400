// Cache-write kernel: scatters new K/V rows of one layer into the PoD layout and demotes the
// rows that leave the recent window (values always, keys once per block).
//
// One work item = (token t, KV head h, K or V), handled by D/8 lanes moving 16 bytes each.
// The lanes that write a ring slot first move the slot's previous occupant to the distant
// store, so eviction and insertion of one slot never race: every slot is touched by exactly
// one item per call (two new positions of one call never share a slot because only the last
// n_r new positions go to the ring).
//
// A long prefill is mostly tokens that are already outside the window when the call ends: they
// go straight to the distant stores, consecutive positions to consecutive rows.  Those are
// copied by the leading blocks of the grid, each a run of 128 tokens of one (head, K or V):
// no per-row index arithmetic, eight 16-byte loads in flight per thread.  The remaining blocks
// handle the sink and ring rows (and the rows they displace) item by item.
#include "pod_common.h"

namespace pod {

template <int D>
__global__ void __launch_bounds__(256, 4) pod_write_kernel(const WriteParams p) {
  constexpr int LPR = D / 8;                 // lanes per row (16 bytes per lane)
  constexpr int ITEMS_PER_BLOCK = 256 / LPR;
  const Layout& y = p.y;
  const int S = y.S, W = y.W, H = y.H_kv;

  // Launched with programmatic stream serialization: wait for the previous kernel of the
  // stream (it may still read rows this kernel overwrites) before touching global memory.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const bool batched = (p.seq < 0);
  const int b = batched ? (int)blockIdx.y : p.seq;
  const int n0 = batched ? p.len[b] : p.n0;
  const int T = p.T;
  const int n1 = n0 + T;
  if (batched) __syncthreads();              // every thread has read len[b] before it changes

  const int sub = threadIdx.x % LPR;
  const int64_t cap_d = y.seq_cap_d[b];
  uint16_t* seq_base = p.arena + y.seq_row_base[b] * D;
  const int ring_first = max(S, n1 - W);     // first position that is in the ring after the call
  // new positions [mid0, ring_first) go straight to the distant stores (empty for short calls)
  const int mid0 = max(n0, S);
  const int n_mid = max(0, ring_first - mid0);

  if ((int)blockIdx.x < p.bulk_blocks) {     // ---- straight-to-distant run of BULK_TOK tokens ----
    constexpr int BULK_TOK = 128, ROWS = 256 / LPR;
    const int hk = blockIdx.x % (2 * H), chunk = blockIdx.x / (2 * H);
    const int kv = hk & 1, h = hk >> 1;
    uint16_t* dist = nullptr;
    if (kv) dist = seq_base + distv_row(y, p.layer, h, cap_d) * D;
    else if (lowest_of(y, p.layer, h) == p.layer) dist = seq_base + distk_row(y, slot_of(y, p.layer, h), cap_d) * D;
    if (dist == nullptr) return;             // distant keys of a layer that is not the head's lowest are dropped
    const int p0 = mid0 + chunk * BULK_TOK, p1 = min(p0 + BULK_TOK, ring_first);
    const uint16_t* src = (kv ? p.v : p.k) + ((int64_t)(p0 - n0) * H + h) * D + sub * 8;
    uint16_t* dst = dist + (int64_t)(p0 - S) * D + sub * 8;
    const int row0 = threadIdx.x / LPR;
    constexpr int IT = BULK_TOK / ROWS;      // rows of a run per thread
    uint4 val[IT];
#pragma unroll
    for (int i = 0; i < IT; ++i) {
      const int rr = row0 + i * ROWS;
      if (p0 + rr < p1) val[i] = *reinterpret_cast<const uint4*>(src + (int64_t)rr * H * D);
    }
#pragma unroll
    for (int i = 0; i < IT; ++i) {
      const int rr = row0 + i * ROWS;
      if (p0 + rr < p1) *reinterpret_cast<uint4*>(dst + (int64_t)rr * D) = val[i];
    }
    return;
  }

  // ---- sink and ring rows: the new tokens outside [mid0, ring_first) ----------------------------
  const int n_head_tok = batched ? 0 : max(0, mid0 - n0);    // new tokens before the run (sink rows)
  const int T_gen = T - n_mid;
  const int gblock = blockIdx.x - p.bulk_blocks, gblocks = gridDim.x - p.bulk_blocks;
  const int item0 = gblock * ITEMS_PER_BLOCK + threadIdx.x / LPR;
  const int item_stride = gblocks * ITEMS_PER_BLOCK;
  const int n_items = T_gen * H * 2;

  // Two items per trip: where each goes is worked out first, then all loads are issued, then the
  // stores, so that a thread keeps several 16-byte requests in flight.  A key row that is neither
  // proximal nor kept (distant, and this layer is not the lowest of the head's block) is not read.
  constexpr int UNROLL = 2;
  for (int base = item0; base < n_items; base += UNROLL * item_stride) {
    const uint4* src[UNROLL];
    uint4* dst[UNROLL];
    uint4* ev_dst[UNROLL];                   // where the row that `dst` displaces goes, if anywhere
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int item = base + u * item_stride;
      src[u] = nullptr; dst[u] = nullptr; ev_dst[u] = nullptr;
      if (item >= n_items) continue;
      const int kv = item & 1;
      const int h = (item >> 1) % H;
      const int tg = (item >> 1) / H;
      const int t = tg < n_head_tok ? tg : tg + n_mid;       // skip the straight-to-distant run
      const int pos = n0 + t;
      const int64_t src_tok = batched ? b : t;
      uint16_t* prox = seq_base + prox_row(y, p.layer, kv, h) * D;
      uint16_t* dist = nullptr;              // distant store of this item's kind, if it is kept
      if (kv) dist = seq_base + distv_row(y, p.layer, h, cap_d) * D;
      else if (lowest_of(y, p.layer, h) == p.layer)        // keys survive once per block of this head
        dist = seq_base + distk_row(y, slot_of(y, p.layer, h), cap_d) * D;
      if (pos < S) {
        dst[u] = reinterpret_cast<uint4*>(prox + (int64_t)pos * D + sub * 8);
      } else if (pos >= ring_first) {
        const int slot = (pos - S) % W;
        dst[u] = reinterpret_cast<uint4*>(prox + (int64_t)(S + slot) * D + sub * 8);
        // previous occupant: the largest position below n0 in the same slot
        const int old = pos - ((pos - n0) / W + 1) * W;
        if (old >= S && dist != nullptr) ev_dst[u] = reinterpret_cast<uint4*>(dist + (int64_t)(old - S) * D + sub * 8);
      }
      if (dst[u] != nullptr)
        src[u] = reinterpret_cast<const uint4*>((kv ? p.v : p.k) + (src_tok * H + h) * D + sub * 8);
    }
    uint4 val[UNROLL], ev[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (src[u] != nullptr) val[u] = *src[u];
      if (ev_dst[u] != nullptr) ev[u] = *dst[u];
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (ev_dst[u] != nullptr) *ev_dst[u] = ev[u];
      if (dst[u] != nullptr) *dst[u] = val[u];
    }
  }

  if (threadIdx.x == 0 && gblock == 0) p.len[b] = n1;
}

int launch_write(const WriteParams& p_in, cudaStream_t s) {
  WriteParams p = p_in;
  p.bulk_blocks = 0;
  const int D = p.y.D;
  const int lpr = D / 8;
  const int items_per_block = 256 / lpr;
  dim3 grid(1, 1, 1);
  if (p.seq < 0) {
    grid.y = p.y.B;                          // one block per sequence: it alone touches len[b]
  } else {
    // tokens that are outside the window when the call ends: runs of 128 per (head, K or V)
    const int n1 = p.n0 + p.T;
    const int ring_first = n1 - p.y.W > p.y.S ? n1 - p.y.W : p.y.S;
    const int mid0 = p.n0 > p.y.S ? p.n0 : p.y.S;
    const int n_mid = ring_first > mid0 ? ring_first - mid0 : 0;
    const int64_t bulk = (int64_t)((n_mid + 127) / 128) * 2 * p.y.H_kv;
    const int64_t n_items = (int64_t)(p.T - n_mid) * p.y.H_kv * 2;
    int64_t blocks = (n_items + items_per_block - 1) / items_per_block;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;              // block 0 of this part also publishes the new length
    if (bulk + blocks > 0x7fffffff) return (int)cudaErrorInvalidValue;
    grid.x = (unsigned)(bulk + blocks);
    p.bulk_blocks = (int32_t)bulk;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (D == 128) return (int)cudaLaunchKernelEx(&cfg, pod_write_kernel<128>, p);
  return (int)cudaLaunchKernelEx(&cfg, pod_write_kernel<64>, p);
}

}  // namespace pod
