// Cache-write kernel: scatters new K/V rows of one layer into the PoD layout and demotes the
// rows that leave the recent window (values always, keys once per block).
//
// One work item = (token t, KV head h, K or V), handled by D/8 lanes moving 16 bytes each.
// The lanes that write a ring slot first move the slot's previous occupant to the distant
// store, so eviction and insertion of one slot never race: every slot is touched by exactly
// one item per call (two new positions of one call never share a slot because only the last
// n_r new positions go to the ring).
#include "pod_common.h"

namespace pod {

template <int D>
__global__ void __launch_bounds__(256) pod_write_kernel(const WriteParams p) {
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
  const int item0 = blockIdx.x * ITEMS_PER_BLOCK + threadIdx.x / LPR;
  const int item_stride = gridDim.x * ITEMS_PER_BLOCK;
  const int n_items = T * H * 2;

  const int64_t cap_d = y.seq_cap_d[b];
  uint16_t* seq_base = p.arena + y.seq_row_base[b] * D;
  const int ring_first = max(S, n1 - W);     // first position that is in the ring after the call

  for (int item = item0; item < n_items; item += item_stride) {
    const int kv = item & 1;
    const int h = (item >> 1) % H;
    const int t = (item >> 1) / H;
    const int pos = n0 + t;
    const uint16_t* src_all = kv ? p.v : p.k;
    const int64_t src_tok = batched ? b : t;
    const uint4 val = *reinterpret_cast<const uint4*>(src_all + (src_tok * H + h) * D + sub * 8);

    uint16_t* prox = seq_base + prox_row(y, p.layer, kv, h) * D;
    uint16_t* dist = nullptr;                // distant store of this item's kind, if it is kept
    if (kv) dist = seq_base + distv_row(y, p.layer, h, cap_d) * D;
    else if (lowest_of(y, p.layer, h) == p.layer)          // keys survive once per block of this head
      dist = seq_base + distk_row(y, slot_of(y, p.layer, h), cap_d) * D;

    if (pos < S) {
      *reinterpret_cast<uint4*>(prox + (int64_t)pos * D + sub * 8) = val;
    } else if (pos >= ring_first) {
      const int slot = (pos - S) % W;
      uint16_t* slot_ptr = prox + (int64_t)(S + slot) * D + sub * 8;
      // previous occupant: the largest position below n0 in the same slot
      const int old = pos - ((pos - n0) / W + 1) * W;
      if (old >= S && dist != nullptr) {
        const uint4 ev = *reinterpret_cast<const uint4*>(slot_ptr);
        *reinterpret_cast<uint4*>(dist + (int64_t)(old - S) * D + sub * 8) = ev;
      }
      *reinterpret_cast<uint4*>(slot_ptr) = val;
    } else if (dist != nullptr) {            // new token that is already outside the window
      *reinterpret_cast<uint4*>(dist + (int64_t)(pos - S) * D + sub * 8) = val;
    }
  }

  if (threadIdx.x == 0 && blockIdx.x == 0) p.len[b] = n1;
}

int launch_write(const WriteParams& p, cudaStream_t s) {
  const int D = p.y.D;
  const int lpr = D / 8;
  const int items_per_block = 256 / lpr;
  dim3 grid(1, 1, 1);
  if (p.seq < 0) {
    grid.y = p.y.B;                          // one block per sequence: it alone touches len[b]
  } else {
    const int64_t n_items = (int64_t)p.T * p.y.H_kv * 2;
    int64_t blocks = (n_items + items_per_block - 1) / items_per_block;
    if (blocks > 148 * 16) blocks = 148 * 16;
    grid.x = (unsigned)(blocks < 1 ? 1 : blocks);
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
