// Split-K decode attention over the PoD layout with the log-sum-exp combine in the same launch.
//
// Grid (KV head, split, sequence): consecutive CTAs belong to different heads, so every head's
// CTAs are spread over all SMs.  The CTAs of one (sequence, KV head) share that head's tokens.
// The tokens are cut into tiles of 16 in "virtual" order -- proximal rows first (sink, then
// ring slots), distant rows after -- and tiles into chunks of a few tiles.  Each warp is an
// independent flash-decoding stream over chunks:
//   * the first chunks of a warp are fixed (round-robin over the head's warps); the rest are
//     drawn from a per-head counter with atomicAdd, so warps on SMs that get less memory
//     bandwidth simply take fewer chunks and all warps of a head finish together.  The draw for
//     the next chunk is issued one chunk ahead and its result is only read when that chunk is
//     entered, so the round trip hides behind the loads already in flight;
//   * lane 0 stages a tile (16 K rows + 16 V rows) into the warp's private shared-memory ring
//     with tiled TMA loads (one tensor map views the whole arena as [rows][d]; 128-byte
//     swizzle, no multicast) that complete on an mbarrier;
//   * when a tile lands the warp pulls all of its K and V fragments into registers with
//     ldmatrix and refills the stage at once, so the memory pipeline never waits for the
//     arithmetic;
//   * logits: S[16 x 16] = Q[16 x d] K^T with mma.sync m16n8k16 (bf16 in, fp32 out); the rows of Q
//     are the r <= 8 query heads of the KV head, zero-padded to 16.  One online softmax in base
//     2 runs over proximal and distant tiles alike: proximal tiles use the layer's own query,
//     distant tiles the stashed query of the block's lowest layer (Eq. 1 rows 1 and 3);
//   * values: O^T[d x 8] += V^T[d x 16] P^T[16 x 8]: the channels are the M dimension, so no
//     accumulator row is padding; the exponentials in the accumulator layout of S are exactly
//     the B fragments, V^T fragments come from ldmatrix.trans.
//   * shared distant scores (Section 2.2: the layers of a block share the attention scores of the
//     lowest layer): a lowest layer of a block with several layers stores its distant logits as it
//     computes them; the other layers read them (r * 64 bytes per 16 tokens) in place of the key
//     rows and skip Q K^T.  Their distant tiles hold 32 value rows, so a stage carries the same
//     bytes either way.
// A launch may also do the append of the step's token (pod_append_decode_attn): warp 0 of a head's
// first CTA copies the new rows in, moves the displaced rows to the distant stores and adds the
// terms of those two tokens from registers, while every streaming warp masks those two rows.
// Warps merge through shared memory; the CTA writes one fp32 partial (acc, max, sum) per query
// head, takes a ticket of its (sequence, KV head), and the CTA that draws the last ticket merges
// all partials (the gate of Eq. 2 generalised from two parts to n_splits parts): each of its warps
// pulls one query head's partials into shared memory with bulk async copies, so the merge costs
// one memory round trip instead of one per split.  Nobody waits for anybody, so nothing can hang;
// every mbarrier wait is bounded and a wait that gives up raises the cache's error flag.
// The kernels are launched with programmatic stream serialization: everything above
// griddepcontrol.wait overlaps the tail of the previous kernel in the stream -- barrier setup
// always, and the requests for the first tiles when the host knows that no unfinished launch
// writes the rows they read.
#include <cuda_bf16.h>

#include "pod_common.h"

namespace pod {

namespace {

constexpr int TOK = 16;          // tokens per tile (one mma k-step of P V)
constexpr uint32_t WAIT_LIMIT = 1u << 20;
constexpr int REDO_SHIFT = 20;
constexpr int REDO_MARK = 1 << REDO_SHIFT;     // added to a head's ticket word by a warp whose early copy of q, k or v was stale
constexpr int DONE_POLLS = 1 << 13;   // polls (about 0.3 us apart) of a head's DONE word before falling back to the grid wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
// Tiled TMA load of a [TOK rows][64 bf16] box at (x, y) = (channel, arena row).  x is 0 or
// 64 elements, i.e. a multiple of 16 bytes as TMA requires.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}
// L2 eviction policy: cache rows are read once per decode step and stream through with evict_first.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// The stored logits are written by one launch and read by the next: when all of a cache's logit stores are a
// small part of the L2 (the host decides), they are kept there with evict_last.
__device__ __forceinline__ uint64_t policy_logits(bool keep) {
  uint64_t p;
  if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_f32x4_hint(float* a, float4 v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1,%2,%3,%4}, %5;"
               ::"l"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(policy) : "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
// Untiled bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void bulk_load_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
               : "memory");
}
// Launch trace (pod_cache_set_trace): the first CTA to start and the last to finish leave the
// GPU's nanosecond timer, so that a benchmark can see when consecutive launches of a stream, which
// overlap, really begin and end.  Two fire-and-forget atomics per CTA, none when the trace is off.
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void trace_begin(const DecodeParams& p) {
  if (p.trace != nullptr && threadIdx.x == 0) atomicMin(p.trace, global_timer_ns());
}
__device__ __forceinline__ void trace_end(const DecodeParams& p) {
  if (p.trace != nullptr && threadIdx.x == 0) atomicMax(p.trace + 1, global_timer_ns());
}
__device__ __forceinline__ int ld_acquire_gpu(const int* a) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(a) : "memory");
  return v;
}
// A load that may race with a store of the previous kernel (the early copies of q, k, v, checked later),
// or that must see that kernel's stores after the grid wait: served by the L2, never by an L1 line of this
// SM (which an earlier load of this kernel may have filled with older data).
__device__ __forceinline__ uint4 ld_relaxed_u32x4(const void* a) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(a) : "memory");
  return v;
}
// 16 bytes global -> shared, asynchronously, through the L2 only (cp.async.cg)
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ bool differ(const uint4& a, const uint4& b) {
  return a.x != b.x || a.y != b.y || a.z != b.z || a.w != b.w;
}
__device__ __forceinline__ float lds_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ float2 lds_f32x2(uint32_t a) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts_f32(uint32_t a, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D = A (16x16, bf16, row) * B (16x8, bf16, col) + D, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}


template <int D>
struct Cfg {
  static constexpr int NW = DECODE_WARPS;
  static constexpr int NSTAGE = DECODE_STAGES;
  static constexpr int NSUB = D / 64;                 // 128-byte wide sub-tiles per row
  static constexpr int SUB_B = TOK * 128;             // bytes of one sub-tile (1024-byte multiple)
  static constexpr int TILE_B = NSUB * SUB_B;         // bytes of one K (or V) tile
  static constexpr int STAGE_B = 2 * TILE_B;
  static constexpr int WARP_B = NSTAGE * STAGE_B;
  static constexpr int RING_B = NW * WARP_B;
  static constexpr int SC_SLOT_B = 1024;              // per stage: logits of 32 tokens x up to 8 heads, fp32
  static constexpr int SC_B = NW * NSTAGE * SC_SLOT_B;
  static constexpr int N_BARS = NW * NSTAGE + NW;     // one per stage, one per warp for the combine
  static constexpr int SMEM = RING_B + SC_B + N_BARS * 8 + 1024;   // + slack to align to 1024
  // the combine reuses each warp's ring: (max, sum) pairs, split weights, then partial rows
  static constexpr int CML_OFF = 0, CW_OFF = MAX_SPLITS_CAP * 16, CROW_OFF = CW_OFF + MAX_SPLITS_CAP * 4;
  static constexpr int CROWS = (WARP_B - CROW_OFF) / (D * 4);   // partial rows per round
  static_assert(CROWS >= 8, "a warp's ring must hold a few partial rows for the combine");
  static_assert(WARP_B >= (8 * D + 24) * 4, "merge scratch must fit the warp's ring");
};

// Everything a warp needs to request a tile; filled once per warp.
struct TileSource {
  const CUtensorMap* tmap;
  uint64_t policy;                  // of the cache rows
  uint64_t sc_policy;               // of the stored logits
  unsigned char* sc_base;           // the head's stored logits
  uint32_t bar0, ring, sc0;         // shared-memory addresses: first stage barrier, first stage, first logit slot
  int32_t ntp, rowKp, rowVp, rowKd, rowVd, sc_group_b;
  int32_t dt_shift;                 // log2 of the tokens of a distant tile
  int32_t from_scores;              // the head reads stored logits instead of distant keys
};
// Requests virtual tile vt into a stage (lane 0 only).  Rows past the segment are other (finite) cache rows,
// or zero fill past the arena; their logits are masked.  `dep` is zero; it carries a register dependency.
// part 0: the whole tile; 1: all but the stored logits (before the head's logits are known to be complete);
// 2: the logits alone.  Not inlined: it is called from a dozen places, none of them hot.
template <int D>
__device__ __noinline__ void issue_tile(const TileSource t, int vt, int stage, int dep, int part) {
  using C = Cfg<D>;
  const bool dist = vt >= t.ntp;
  const uint32_t bar = t.bar0 + stage * 8;
  const uint32_t dst = t.ring + stage * C::STAGE_B;
  if (dist && t.from_scores) {        // 32 value rows + their logits; no key rows
    const int yv0 = t.rowVd + ((vt - t.ntp) << t.dt_shift) + dep;
    if (part != 2) mbar_expect_tx(bar, C::STAGE_B + 2 * t.sc_group_b);
    if (part != 1)
      bulk_load_hint(t.sc0 + stage * C::SC_SLOT_B, t.sc_base + (int64_t)(vt - t.ntp) * 2 * t.sc_group_b, 2 * t.sc_group_b, bar,
                     t.sc_policy);
    if (part == 2) return;
#pragma unroll
    for (int s = 0; s < C::NSUB; ++s) {
      tma_load_2d(dst + s * C::SUB_B, t.tmap, s * 64, yv0, bar, t.policy);
      tma_load_2d(dst + C::TILE_B + s * C::SUB_B, t.tmap, s * 64, yv0 + TOK, bar, t.policy);
    }
    return;
  }
  if (part == 2) return;
  const int yk = (dist ? t.rowKd + (vt - t.ntp) * TOK : t.rowKp + vt * TOK) + dep;
  const int yv = dist ? t.rowVd + (vt - t.ntp) * TOK : t.rowVp + vt * TOK;
  mbar_expect_tx(bar, C::STAGE_B);
#pragma unroll
  for (int s = 0; s < C::NSUB; ++s) {
    tma_load_2d(dst + s * C::SUB_B, t.tmap, s * 64, yk, bar, t.policy);
    tma_load_2d(dst + C::TILE_B + s * C::SUB_B, t.tmap, s * 64, yv, bar, t.policy);
  }
}

// Recomputation of one (sequence, KV head) by a single CTA with a plain loop over its tokens: the way out
// for a head in which some warp streamed with a copy of q that the previous kernel of the stream had not
// finished writing (optimistic start).  Exact and slow (a warp per query head, a token per trip); it reads
// the final rows of the cache -- every CTA of the head has taken its ticket -- and the final q, and writes
// what the fast path writes: the output, and for a block's lowest layer the distant logits and their
// log-sum-exp.
template <int D>
__device__ __noinline__ void redo_head(const uint16_t* arena, const uint16_t* q_all, const uint16_t* stash, uint16_t* out,
                                       float* dlse, float scale_log2, int64_t hq0, int r, int n_p, int n_d, int64_t rowKp,
                                       int64_t rowVp, int64_t rowKd, int64_t rowVd, unsigned char* sc_base, int sc_group_b,
                                       bool is_low, bool sc_write, int64_t q_own, int64_t q_st) {
  // (plain arguments: a reference to the kernel's parameter block would force a copy of it onto the stack)
  constexpr int CPL = D / 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const __nv_bfloat16* rows = reinterpret_cast<const __nv_bfloat16*>(arena);
  const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(q_all);
  const __nv_bfloat16* st = reinterpret_cast<const __nv_bfloat16*>(stash);
  for (int h = warp; h < r; h += DECODE_WARPS) {
    float qo[CPL], ql[CPL], acc[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
      qo[j] = __bfloat162float(q[q_own + h * D + lane * CPL + j]);
      ql[j] = is_low ? qo[j] : __bfloat162float(st[q_st + h * D + lane * CPL + j]);
      acc[j] = 0.f;
    }
    float m = -INFINITY, l = 0.f, ld = 0.f;
    for (int t = 0; t < n_p + n_d; ++t) {
      const bool dist = t >= n_p;
      const int64_t kr = dist ? rowKd + (t - n_p) : rowKp + t, vr = dist ? rowVd + (t - n_p) : rowVp + t;
      float dot = 0.f;
#pragma unroll
      for (int j = 0; j < CPL; ++j) dot += (dist ? ql[j] : qo[j]) * __bfloat162float(rows[kr * D + lane * CPL + j]);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      const float a = dot * scale_log2;
      if (dist && sc_write && lane == 0) {          // same place as the streaming path: groups of 16 tokens, fragment order
        const int td = t - n_p, c = td & 15;
        float* slot = reinterpret_cast<float*>(sc_base + (int64_t)(td >> 4) * sc_group_b + (h * 4 + ((c & 7) >> 1)) * 16) +
                      ((c >> 3) * 2 + (c & 1));
        *slot = a;
      }
      const float m_new = fmaxf(m, a), alpha = ex2(m - m_new), pr = ex2(a - m_new);
      m = m_new;
      l = l * alpha + pr;
      ld = ld * alpha + (dist ? pr : 0.f);
#pragma unroll
      for (int j = 0; j < CPL; ++j) acc[j] = acc[j] * alpha + pr * __bfloat162float(rows[vr * D + lane * CPL + j]);
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int64_t hq = hq0 + h;
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + hq * D + lane * CPL;
#pragma unroll
    for (int j = 0; j < CPL; j += 2)
      *reinterpret_cast<__nv_bfloat162*>(dst + j) = __floats2bfloat162_rn(acc[j] * inv, acc[j + 1] * inv);
    if (sc_write && lane == 0) dlse[hq] = ld > 0.f ? m + __log2f(ld) : -INFINITY;
  }
}

template <int D>
__global__ void __launch_bounds__(DECODE_WARPS * 32, DECODE_CTAS_PER_SM)
pod_decode_splitk_kernel(const __grid_constant__ CUtensorMap tmap, const DecodeParams p) {
  using C = Cfg<D>;
  constexpr int NW = C::NW, NSTAGE = C::NSTAGE;
  const Layout& y = p.y;
  const int r = y.H_q / y.H_kv;   // query heads per KV head (<= 8): rows of the Q operand

  const int b = blockIdx.z, kvh = blockIdx.x, split = blockIdx.y;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);   // swizzle atoms are 1024 B
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  trace_begin(p);
  unsigned char* wbuf = smem + warp * C::WARP_B;
  const uint32_t wbuf_s = smem_u32(wbuf);
  const uint32_t sc0 = smem_u32(smem + C::RING_B) + warp * NSTAGE * C::SC_SLOT_B;   // this warp's logit slots
  const uint32_t bar0 = smem_u32(smem + C::RING_B + C::SC_B) + warp * NSTAGE * 8;
  const uint32_t cbar = smem_u32(smem + C::RING_B + C::SC_B) + (NW * NSTAGE + warp) * 8;   // this warp's combine barrier
  if (lane == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + s * 8, 1);
    mbar_init(cbar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
  }
  const int bv = b < SMALL_BATCH ? b : 0;
  int n = p.v_len[bv];
  int64_t cap_d = p.v_cap_d[bv];
  int64_t seq_row = p.v_row_base[bv];
  const uint64_t pol_stream = policy_evict_first();
  const uint64_t pol_logits = policy_logits(p.keep_logits != 0);

  // The wait for the previous kernel of the stream comes before anything that kernel may have
  // written is read: stash, counters, logits, the new token.  The cache rows and this layer's
  // lengths are older when the host says so (early_ok: the previous launch on this cache was a decode
  // launch of another layer); then the first tiles are requested before the wait, so that the
  // memory latency of the start-up overlaps the previous kernel's tail.
  bool waited = false;
  if (!p.early_ok) {
    pdl_wait();
    pdl_launch_dependents();
    waited = true;
  }
  const bool fused = p.new_k != nullptr;      // this launch also appends one token per sequence
  if (!p.by_value) {
    n = p.len[b] + (fused ? 1 : 0);
    cap_d = y.seq_cap_d[b];
    seq_row = y.seq_row_base[b];
  }

  // ---- tiles and chunks of this (sequence, KV head) -----------------------------------------
  // The plan comes with the launch when the launch is small (no arithmetic and no load between a CTA's
  // start and its first tile requests); otherwise it is worked out here, by the same function.
  HeadPlan hp;
  if (p.plans_by_value) {
    hp = p.v_plan[b * y.H_kv + kvh];
  } else {
    int low_layer, kslot_;
    bool store;
    if (p.heads_by_value) {
      low_layer = p.v_low[kvh];
      kslot_ = p.v_slot[kvh];
      store = (p.v_store_mask >> kvh) & 1u;
    } else {
      low_layer = lowest_of(y, p.layer, kvh);
      kslot_ = slot_of(y, p.layer, kvh);
      store = y.shared && low_layer == p.layer && p.layer + 1 < y.L && lowest_of(y, p.layer + 1, kvh) == p.layer;
    }
    const bool read = low_layer != p.layer && kvh < 256 && ((p.score_read_mask[kvh >> 5] >> (kvh & 31)) & 1u);
    PlanInputs in;
    in.layer = p.layer; in.segment = p.segment; in.fused = fused ? 1 : 0; in.max_splits = p.max_splits;
    in.split_rows = p.split_rows; in.tiles_per_chunk = p.tiles_per_chunk; in.static_eighths = p.static_eighths;
    in.tile_tokens = TOK; in.warps = NW;
    hp = make_head_plan(y, in, kvh, n, cap_d, seq_row, low_layer, kslot_, store, read);
  }
  const int n_p = hp.n_p, n_d = hp.n_d;
  const int kslot = hp.kslot;
  const bool is_low = hp.flags & HP_LOW, sc_write = hp.flags & HP_STORE, sc_read = hp.flags & HP_READ;
  const int nsplit = hp.nsplit;
  if (split >= nsplit) return;
  const int DT_SH = sc_read ? 5 : 4;              // log2 of the tokens per distant tile
  const int DT = 1 << DT_SH;
  const int ntp = hp.ntp, ntd = hp.ntd;
  const int ntiles = ntp + ntd;
  const int tch = p.tiles_per_chunk;
  const int nwh = nsplit * NW;                    // warps working on this head
  const int gw = split * NW + warp;               // this warp's index among them
  const int k_static = hp.k_static;               // chunks per warp taken without a draw
  const int dyn_base = k_static * nwh;            // first chunk id that is drawn
  int* sched = p.sched + ((int64_t)b * y.H_kv + kvh) * SCHED_STRIDE;
  int* ctr = sched + (p.seq & 1) * SCHED_CTR1;    // this launch's chunk counter
  // Optimistic start (see DecodeParams): no wait for the previous kernel before streaming.  Heads that
  // must score the block's keys with the stashed queries themselves (their stored logits were
  // overwritten) are rare and wait as usual.
  const bool opt = p.optimistic && !waited && (is_low || sc_read);
  bool late_pending = opt;                        // the grid wait is still to come
  const int64_t q_own = ((int64_t)b * y.H_q + kvh * r) * D;         // this head's r query rows in q
  const int64_t q_st = ((int64_t)kslot * y.B + b) * r * D;          // and in the stash of its block
  constexpr int QS = D + 8;                       // row stride in elements: the fragment reads hit 32 banks
  __shared__ __align__(16) uint16_t s_q[8 * QS];
  // Warp 0 brings the CTA's copy of q into shared memory in two steps: the loads go out into registers,
  // and the stores to shared memory follow where the values are first needed, so that the warp does not sit
  // out a memory round trip between the two.
  constexpr int QL = D / 32;                      // 16-byte pieces per lane: up to 8 heads x D / 8 pieces
  uint4 q_reg[QL];
  auto request_q = [&]() {
    if (warp == 0) {
#pragma unroll
      for (int k = 0; k < QL; ++k) {
        const int i = lane + 32 * k;
        if (i < r * (D / 8)) q_reg[k] = ld_relaxed_u32x4(p.q + q_own + (int64_t)i * 8);
      }
    }
  };
  auto keep_q = [&]() {
    if (warp == 0) {
#pragma unroll
      for (int k = 0; k < QL; ++k) {
        const int i = lane + 32 * k;
        if (i < r * (D / 8)) *reinterpret_cast<uint4*>(&s_q[(i / (D / 8)) * QS + (i % (D / 8)) * 8]) = q_reg[k];
      }
    }
  };
  // q is requested before the tiles when it may be read already (the tile requests of a whole SM would
  // be served first otherwise): the launch has waited, or starts optimistically
  const bool q_loaded = waited || opt;
  if (q_loaded) request_q();

  // arena rows of this (sequence, layer, head): tile coordinates of the tensor map
  const int rowKp = hp.rowKp, rowVp = hp.rowVp, rowKd = hp.rowKd, rowVd = hp.rowVd;
  // shared distant logits of this head: groups of 16 tokens x r heads, fp32, fragment order
  const int sc_group_b = score_group_bytes(y);
  unsigned char* sc_base = reinterpret_cast<unsigned char*>(const_cast<uint16_t*>(p.arena)) + (int64_t)hp.score_row * (D * 2);

  if (p.segment == 2 && sched[SCHED_NEED] == 0) {          // every query head of this KV head skipped: no distant work
    if (sc_write && threadIdx.x == 0) atomicAdd(sched + SCHED_DONE, 1);   // (the host counts every CTA of a storing head)
    return;
  }

  // ---- the warp's walk over its chunks (all values uniform across the warp) -----------------
  if (!waited && !opt && k_static * tch < NSTAGE) {   // the first tiles need draws: no early start
    pdl_wait();
    pdl_launch_dependents();
    waited = true;
  }
  // A warp's first draw is issued when it enters the last of its fixed chunks (not at the start, where
  // the draws of all warps of a head would queue up on one counter).  Consecutive launches use different
  // counters, and a launch starts only after the launch before the previous one has ended (every launch
  // lets its dependents go only after its own grid wait), so a counter is zero and unused when its launch
  // starts; without the optimistic start nothing is drawn before the wait all the same.
  unsigned drawn = 0;                             // lane 0: result of the draw issued one chunk ahead
  bool drew = false;
  int c_id, c_t = 0, c_j = 0;
  bool walk_done = false;
  auto first_draw = [&]() {
    if (!drew && (waited || opt) && c_j >= k_static - 1) {
      if (lane == 0) drawn = (unsigned)atomicAdd(ctr, 1);
      drew = true;
    }
  };
  if (k_static > 0) {
    c_id = gw;
    first_draw();
  } else {                                        // (the wait above has happened)
    if (lane == 0) drawn = (unsigned)atomicAdd(ctr, 1);
    c_id = dyn_base + (int)__shfl_sync(0xffffffffu, drawn, 0);
    if (lane == 0) drawn = (unsigned)atomicAdd(ctr, 1);
    drew = true;
  }
  auto next_tile = [&]() -> int {                 // virtual tile index, or -1 when the head is used up
    if (walk_done) return -1;
    if (c_t == tch) {
      c_t = 0;
      ++c_j;
      if (c_j < k_static) {
        c_id = gw + c_j * nwh;
        first_draw();
      } else {
        c_id = dyn_base + (int)__shfl_sync(0xffffffffu, drawn, 0);
        if (lane == 0) drawn = (unsigned)atomicAdd(ctr, 1);
      }
    }
    const int64_t vt = (int64_t)c_id * tch + c_t;
    ++c_t;
    if (vt >= ntiles) { walk_done = true; return -1; }
    return (int)vt;
  };
  TileSource src;
  src.tmap = &tmap; src.policy = pol_stream; src.sc_policy = pol_logits; src.sc_base = sc_base; src.bar0 = bar0; src.ring = wbuf_s; src.sc0 = sc0;
  src.ntp = ntp; src.rowKp = rowKp; src.rowVp = rowVp; src.rowKd = rowKd; src.rowVd = rowVd; src.sc_group_b = sc_group_b;
  src.dt_shift = DT_SH; src.from_scores = sc_read ? 1 : 0;
  auto issue = [&](int vt, int stage, int dep, int part) { issue_tile<D>(src, vt, stage, dep, part); };

  // Rows that change in a fused launch are masked in the streamed tiles and added by one warp
  // from registers: the new token's proximal row, and the distant row of the token it pushes
  // out of the recent window.
  int tA = -1, cA = 0, tB = -1, cB = 0;
  const int rA = hp.rA, rB = hp.rB;
  if (fused) {
    tA = rA / TOK; cA = rA % TOK;
    if (rB >= 0) { tB = ntp + (rB >> DT_SH); cB = rB & (DT - 1); }
  }

  // The block's logits (and stashed queries) come from an earlier launch of this cache, possibly the one
  // still running.  Every CTA of that launch adds one to the head's DONE word when its warps have finished
  // streaming (all logits of theirs are stored); the host knows what the word reads once the head is
  // complete.  A CTA that found its copy of q stale does not add its one: the CTA that recomputes the head
  // adds the missing ones when the logits have been rewritten, so the word is complete only then.
  auto scores_complete = [&]() -> bool {          // lane 0's view, passed to the warp
    int ok = 0;
    if (lane == 0) ok = (int)(ld_acquire_gpu(sched + SCHED_DONE) - hp.wait_done) >= 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
  };
  // An optimistic launch that reads stored logits looks before its tile requests go out (behind them an
  // answer takes microseconds).  CTAs that start after the head is complete then request whole tiles at
  // once and never poll; the others request one stage (values only) and poll.
  const bool scores_done = opt && sc_read && scores_complete();
  if (scores_done && lane == 0) fence_async_global();       // the logits are read through the async proxy
  const int n_prime = (opt && sc_read && !scores_done) ? 1 : NSTAGE;
  int vt_q[NSTAGE];                               // tile held by each stage, -1 = none
#pragma unroll
  for (int s = 0; s < NSTAGE; ++s) {
    vt_q[s] = -1;
    if (s < n_prime) {
      vt_q[s] = next_tile();
      if (lane == 0 && vt_q[s] >= 0) issue(vt_q[s], s, 0, (waited || scores_done) ? 0 : 1);
    }
  }
  if (!waited) {
    if (!opt) {
      pdl_wait();
      pdl_launch_dependents();
    } else if (sc_read && warp == 0 && !scores_done) {
      // One warp of the CTA polls (the barrier below passes the news on).  Bounded; after the limit the
      // grid wait settles it.
      bool ready = false;
      for (int it = 0; it < DONE_POLLS && !ready; ++it) {
        ready = scores_complete();
        if (!ready) __nanosleep(128);
      }
      if (!ready) {                     // (the grid wait again later, in late_wait, returns at once)
        pdl_wait();
        pdl_launch_dependents();
      }
    }
  }
  if (!q_loaded) request_q();           // (a launch that had to wait first reads q only now)
  keep_q();
  __syncthreads();                      // q in shared memory; the head's logits known to be complete
  if (!waited) {
    if (lane == 0 && !scores_done) {
      if (opt && sc_read) fence_async_global();     // the logits are read through the async proxy
#pragma unroll
      for (int s = 0; s < NSTAGE; ++s)
        if (s < n_prime && vt_q[s] >= 0) issue(vt_q[s], s, 0, 2);
    }
    waited = true;
    first_draw();
#pragma unroll
    for (int s = 0; s < NSTAGE; ++s)
      if (s >= n_prime) {
        vt_q[s] = next_tile();
        if (lane == 0 && vt_q[s] >= 0) issue(vt_q[s], s, 0, 0);
      }
  }

  // a head's lowest layer saves its queries for the other layers of the block
  auto stash_q = [&]() {
    if (sc_write && split == 0 && warp == 0 && lane < D / 8) {
      for (int h = 0; h < r; ++h)
        *reinterpret_cast<uint4*>(p.stash + q_st + h * D + lane * 8) =
            *reinterpret_cast<const uint4*>(p.q + q_own + h * D + lane * 8);
    }
  };
  if (!late_pending) stash_q();          // (an optimistic launch stashes after its wait: q may still change)

  // ---- per-lane state -------------------------------------------------------------------
  const int qrow = lane >> 2;          // query head (row of S) owned by this lane's quad
  const int qcol = (lane & 3) * 2;     // first of the two columns this lane holds in a fragment
  // The CTA's copy of its query rows: read once, by warp 0 and past the L1 (when the launch is optimistic
  // the previous kernel may still be writing q, and the copy is compared with a second reading after the
  // grid wait: neither reading may come out of a stale L1 line), then shared by the warps.
  uint32_t qp[D / 16][2], qd[D / 16][2];   // A fragments of Q (rows 0..7; rows 8..15 are zero):
  {                                        // own query (proximal tiles), lowest layer's (distant)
    const uint16_t* qo = s_q + qrow * QS + qcol;
    const uint16_t* ql = p.stash + q_st + qrow * D + qcol;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      qp[kk][0] = qrow < r ? *reinterpret_cast<const uint32_t*>(qo + kk * 16) : 0u;
      qp[kk][1] = qrow < r ? *reinterpret_cast<const uint32_t*>(qo + kk * 16 + 8) : 0u;
      // (the stash of a block that started lower is complete: it was awaited above)
      qd[kk][0] = is_low ? qp[kk][0] : (qrow < r ? *reinterpret_cast<const uint32_t*>(ql + kk * 16) : 0u);
      qd[kk][1] = is_low ? qp[kk][1] : (qrow < r ? *reinterpret_cast<const uint32_t*>(ql + kk * 16 + 8) : 0u);
    }
  }
  // O^T accumulators: ot[cb][0], [1] = channel cb*16 + qrow of heads qcol, qcol + 1;
  // ot[cb][2], [3] = channel cb*16 + 8 + qrow of the same heads
  float ot[D / 16][4];
#pragma unroll
  for (int cb = 0; cb < D / 16; ++cb) { ot[cb][0] = ot[cb][1] = ot[cb][2] = ot[cb][3] = 0.f; }
  float m_row = -INFINITY, l_row = 0.f;   // running max (log2 units) and sum of head qrow
  float ld_row = 0.f;                     // the distant tokens' part of l_row (same scaling)
  bool failed = false;
  uint32_t round = 0;                     // stage s holds its (round)-th tile: barrier parity round & 1
  int fail_stage = 0;

  uint4 nw_early = make_uint4(0u, 0u, 0u, 0u);     // warp 0 of the head's first CTA: its early copy of the new k / v row
  // ---- fused append: warp 0 of the head's first CTA moves the rows and adds their terms ------
  // (An optimistic launch does this with copies of k and v read before its wait, like q; they are checked
  // with q.  Every streaming warp masks the two rows, and the layer's rows are read by no other launch
  // until the layer's next step, so a stale row harms nobody before the head is redone.)
  if (fused && split == 0 && warp == 0) {
    __shared__ __align__(16) uint16_t s_sp[4][128];     // new K, new V, displaced K, displaced V
    constexpr int LPR = D / 8;                          // lanes per row, 16 bytes each
    uint16_t* arena_w = const_cast<uint16_t*>(p.arena);
    const bool lowest = is_low;
    if (lane < 2 * LPR) {
      const bool isv = lane >= LPR;
      const int sub = lane % LPR;
      const uint4 nw = ld_relaxed_u32x4((isv ? p.new_v : p.new_k) + ((int64_t)b * y.H_kv + kvh) * D + sub * 8);
      nw_early = nw;
      uint4* slot = reinterpret_cast<uint4*>(arena_w + ((int64_t)(isv ? rowVp : rowKp) + rA) * D + sub * 8);
      if (rB >= 0) {
        // The slot's occupant leaves the window: its value row moves to the layer's distant values,
        // its key row to the block's key store only from the lowest layer (other layers drop theirs
        // and score the token with the block's key, written by the lowest layer's launch).
        const uint4 old = *slot;
        uint4* dst = reinterpret_cast<uint4*>(arena_w + ((int64_t)(isv ? rowVd : rowKd) + rB) * D + sub * 8);
        uint4 use = old;
        if (isv || lowest) *dst = old; else use = *dst;
        *reinterpret_cast<uint4*>(&s_sp[isv ? 3 : 2][sub * 8]) = use;
      }
      *slot = nw;
      *reinterpret_cast<uint4*>(&s_sp[isv ? 1 : 0][sub * 8]) = nw;
    }
    if (kvh == 0 && lane == 0) p.len_out[b] = n;
    __syncwarp();
    // one token: logit of head qrow from this lane's Q fragments (quad-reduced), then the same
    // online-softmax update as a tile, in fp32
    auto add_token = [&](const uint16_t* krow, const uint16_t* vrow, const uint32_t (&qf)[D / 16][2], float* logit_dst, bool distant) {
      float dot = 0.f;
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const float2 q0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qf[kk][0]));
        const float2 q1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qf[kk][1]));
        const float2 k0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(krow + kk * 16 + qcol));
        const float2 k1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(krow + kk * 16 + 8 + qcol));
        dot += q0.x * k0.x + q0.y * k0.y + q1.x * k1.x + q1.y * k1.y;
      }
      dot += __shfl_xor_sync(0xffffffffu, dot, 1);
      dot += __shfl_xor_sync(0xffffffffu, dot, 2);
      const float a = dot * p.scale_log2;
      if (logit_dst != nullptr && (lane & 3) == 0 && qrow < r) *logit_dst = a;
      const float m_new = fmaxf(m_row, a);
      const float alpha = ex2(m_row - m_new);
      const float pr = ex2(a - m_new);
      m_row = m_new;
      l_row = l_row * alpha + ((lane & 3) == 0 ? pr : 0.f);   // l_row holds per-lane partial sums
      ld_row = ld_row * alpha + ((distant && (lane & 3) == 0) ? pr : 0.f);
      const float al0 = __shfl_sync(0xffffffffu, alpha, qcol * 4), al1 = __shfl_sync(0xffffffffu, alpha, qcol * 4 + 4);
      const float p0 = __shfl_sync(0xffffffffu, pr, qcol * 4), p1 = __shfl_sync(0xffffffffu, pr, qcol * 4 + 4);
#pragma unroll
      for (int cb = 0; cb < D / 16; ++cb) {
        const float v0 = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vrow + cb * 16 + qrow));
        const float v1 = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vrow + cb * 16 + 8 + qrow));
        ot[cb][0] = ot[cb][0] * al0 + p0 * v0; ot[cb][1] = ot[cb][1] * al1 + p1 * v0;
        ot[cb][2] = ot[cb][2] * al0 + p0 * v1; ot[cb][3] = ot[cb][3] * al1 + p1 * v1;
      }
    };
    add_token(s_sp[0], s_sp[1], qp, nullptr, false);    // the new token is proximal: own query
    if (rB >= 0 && p.segment != 1) {                    // the displaced token is distant: block's query (a
                                                        // proximal-only launch leaves it to the distant launch)
      float* slot = reinterpret_cast<float*>(sc_base + (int64_t)(rB / TOK) * sc_group_b + (qrow * 4 + ((cB & 7) >> 1)) * 16) +
                    ((cB >> 3) * 2 + (cB & 1));
      add_token(s_sp[2], s_sp[3], qd, sc_write ? slot : nullptr, true);
    }
  }

  // ldmatrix lane addressing inside a [TOK][128 B] sub-tile with the 128-byte swizzle:
  // 16-byte chunk c of row t lives at t * 128 + ((c ^ (t & 7)) << 4).
  const int lm = lane >> 3, lr = lane & 7;
  // K (non-transposed): matrices (tokens 0-7, chunk 2kk), (0-7, 2kk+1), (8-15, 2kk), (8-15, 2kk+1)
  const int k_tok = (lm >> 1) * 8 + lr, k_chunk = lm & 1;
  // V (transposed): matrices (tokens 0-7, chunk 2cb), (0-7, 2cb+1), (8-15, 2cb), (8-15, 2cb+1):
  // the A fragments a0..a3 of V^T [16 channels x 16 tokens]
  const int v_tok = (lm >> 1) * 8 + lr, v_chunk = lm & 1;

  // ---- optimistic start: the wait for the previous kernel, and the check of the early copies ----
  // Called when the warp has requested its last tile (the reads below then hide behind the tiles still in
  // flight), at the latest after the loop.  Dependents are let go only now, so that the launch after the
  // next cannot start before the previous one has ended (they would share a chunk counter).
  // The second reading of q (and of the new k, v rows) goes into a stage the warp no longer needs as an
  // asynchronous copy (L2 to shared memory), so that nobody waits for it; it is compared after the loop.
  int check_stage = -1;
  auto late_wait = [&](int free_stage) {   // free_stage: a stage of this warp that no tile will use any more
    pdl_wait();
    pdl_launch_dependents();
    late_pending = false;
    if (warp != 0) return;                 // the CTA's copies were made, and are checked, by warp 0
    check_stage = free_stage;
    const uint32_t dst = wbuf_s + check_stage * C::STAGE_B;
    for (int i = lane; i < r * (D / 8); i += 32) cp_async_16(dst + i * 16, p.q + q_own + (int64_t)i * 8);
    if (fused && split == 0 && lane < D / 4)
      cp_async_16(dst + 8 * D * 2 + lane * 16,
                  (lane >= D / 8 ? p.new_v : p.new_k) + ((int64_t)b * y.H_kv + kvh) * D + (lane % (D / 8)) * 8);
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  auto late_check = [&]() -> bool {        // after the loop: compare; true (in warp 0) if a copy was stale
    if (warp != 0 || check_stage < 0) return false;
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    const unsigned char* got = wbuf + check_stage * C::STAGE_B;
    bool stale = false;
    for (int i = lane; i < r * (D / 8); i += 32) {
      const int h = i / (D / 8), c8 = i % (D / 8);
      stale = stale || differ(*reinterpret_cast<const uint4*>(&s_q[h * QS + c8 * 8]), *reinterpret_cast<const uint4*>(got + i * 16));
    }
    if (fused && split == 0 && lane < D / 4)
      stale = stale || differ(nw_early, *reinterpret_cast<const uint4*>(got + 8 * D * 2 + lane * 16));
    stale = __any_sync(0xffffffffu, stale);
    stash_q();
    return stale;
  };

  // One tile per trip, the stages in turn (the loop is not unrolled over the stages: the code of a trip is
  // large, and three copies of it did not fit the instruction cache with the rest of the kernel).  v0 is the
  // tile in stage s, v1 and v2 the tiles in the two stages after it.
  int v0 = vt_q[0], v1 = NSTAGE > 1 ? vt_q[1] : -1, v2 = NSTAGE > 2 ? vt_q[2] : -1;
  static_assert(NSTAGE <= 3, "the tile rotation below holds three stages");
  int s = 0;
  while (v0 >= 0) {
    {
      const int vt = v0;
      if (!__all_sync(0xffffffffu, mbar_wait(bar0 + s * 8, round & 1))) { failed = true; fail_stage = s; break; }
      const bool dist = vt >= ntp;
      const bool from_scores = dist && sc_read;
      const int rem = dist ? n_d - (vt - ntp) * DT : n_p - vt * TOK;      // valid rows from the tile's start
      const int mtile = vt == tA ? cA : (vt == tB ? cB : -1);             // row handled outside the stream
      const uint32_t ks = wbuf_s + s * C::STAGE_B;
      const uint32_t vs = ks + C::TILE_B;

      // ---- the whole tile into registers, then hand the stage back --------------------------
      // fa: key fragments, or (reading stored logits) value fragments of rows 0-15;
      // fb: value fragments (of rows 16-31 when reading stored logits)
      uint32_t fa[D / 16][4], fb[D / 16][4];
      float4 sca = make_float4(0.f, 0.f, 0.f, 0.f), scb = sca;
      if (from_scores) {
        if (qrow < r) {
          sca = lds_f32x4(sc0 + s * C::SC_SLOT_B + (qrow * 4 + (lane & 3)) * 16);
          scb = lds_f32x4(sc0 + s * C::SC_SLOT_B + sc_group_b + (qrow * 4 + (lane & 3)) * 16);
        }
#pragma unroll
        for (int cb = 0; cb < D / 16; ++cb) {
          const int chunk = 2 * cb + v_chunk;
          ldsm4_t(ks + (chunk >> 3) * C::SUB_B + v_tok * 128 + (((chunk & 7) ^ (v_tok & 7)) << 4), fa[cb]);
        }
      } else {
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const int chunk = 2 * kk + k_chunk;          // 16-byte chunk of the row
          ldsm4(ks + (chunk >> 3) * C::SUB_B + k_tok * 128 + (((chunk & 7) ^ (k_tok & 7)) << 4), fa[kk]);
        }
      }
#pragma unroll
      for (int cb = 0; cb < D / 16; ++cb) {
        const int chunk = 2 * cb + v_chunk;
        ldsm4_t(vs + (chunk >> 3) * C::SUB_B + v_tok * 128 + (((chunk & 7) ^ (v_tok & 7)) << 4), fb[cb]);
      }
      // The refill must not start before the last fragment load has returned (shared-memory
      // loads of a warp return in order): its row coordinate depends on that load's result.
      int dep;
      asm volatile("and.b32 %0, %1, 0;" : "=r"(dep) : "r"(fb[D / 16 - 1][3]));
      __syncwarp();
      const int v_new = next_tile();
      if (lane == 0 && v_new >= 0) issue(v_new, s, dep, 0);

      // one online-softmax step (base 2) over 16 tokens: logits l (log2 units; tokens qcol, +1,
      // +8, +9 of head qrow), `cnt` valid tokens, token `mcol` left out, value fragments vf
      auto softmax_pv = [&](float l00, float l01, float l10, float l11, int cnt, int mcol, const uint32_t (&vf)[D / 16][4],
                            float* store, bool distant) {
        float a00 = (qcol < cnt && qcol != mcol) ? l00 : -INFINITY;
        float a01 = (qcol + 1 < cnt && qcol + 1 != mcol) ? l01 : -INFINITY;
        float a10 = (qcol + 8 < cnt && qcol + 8 != mcol) ? l10 : -INFINITY;
        float a11 = (qcol + 9 < cnt && qcol + 9 != mcol) ? l11 : -INFINITY;
        if (store != nullptr) {                        // the other layers of the block reuse these logits
          if (mcol < 0) {
            st_f32x4_hint(store, make_float4(a00, a01, a10, a11), pol_logits);
          } else {                                     // the displaced token's column is written by warp 0
            if (qcol != mcol) store[0] = a00;
            if (qcol + 1 != mcol) store[1] = a01;
            if (qcol + 8 != mcol) store[2] = a10;
            if (qcol + 9 != mcol) store[3] = a11;
          }
        }
        float mx = fmaxf(fmaxf(a00, a01), fmaxf(a10, a11));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (__any_sync(0xffffffffu, mx > m_row)) {
          const float m_new = fmaxf(m_row, mx);
          const float alpha = ex2(m_row - m_new);     // 0 on the first tile, 1 if unchanged
          m_row = m_new;
          l_row *= alpha;
          ld_row *= alpha;
          // the accumulators of this lane belong to heads qcol and qcol + 1
          const float al0 = __shfl_sync(0xffffffffu, alpha, qcol * 4);
          const float al1 = __shfl_sync(0xffffffffu, alpha, qcol * 4 + 4);
#pragma unroll
          for (int cb = 0; cb < D / 16; ++cb) { ot[cb][0] *= al0; ot[cb][1] *= al1; ot[cb][2] *= al0; ot[cb][3] *= al1; }
        }
        // a tile whose only valid column is handled outside the stream leaves the maximum at -inf
        const float m_use = (m_row == -INFINITY) ? 0.f : m_row;
        a00 = ex2(a00 - m_use); a01 = ex2(a01 - m_use); a10 = ex2(a10 - m_use); a11 = ex2(a11 - m_use);
        l_row += (a00 + a01) + (a10 + a11);
        if (distant) ld_row += (a00 + a01) + (a10 + a11);
        const uint32_t pb0 = pack_bf16(a00, a01), pb1 = pack_bf16(a10, a11);
        // O^T += V^T P^T
#pragma unroll
        for (int cb = 0; cb < D / 16; ++cb) mma16816(ot[cb], vf[cb][0], vf[cb][1], vf[cb][2], vf[cb][3], pb0, pb1);
      };

      if (from_scores) {
        softmax_pv(sca.x, sca.y, sca.z, sca.w, min(TOK, rem), mtile, fa, nullptr, true);
        if (rem > TOK) softmax_pv(scb.x, scb.y, scb.z, scb.w, min(TOK, rem - TOK), mtile - TOK, fb, nullptr, true);
      } else {
        // S = Q K^T, two accumulation chains per token half
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < D / 16; kk += 2) {
          const uint32_t a0 = dist ? qd[kk][0] : qp[kk][0], a2 = dist ? qd[kk][1] : qp[kk][1];
          const uint32_t c0 = dist ? qd[kk + 1][0] : qp[kk + 1][0], c2 = dist ? qd[kk + 1][1] : qp[kk + 1][1];
          mma16816(s0, a0, 0u, a2, 0u, fa[kk][0], fa[kk][1]);
          mma16816(s1, a0, 0u, a2, 0u, fa[kk][2], fa[kk][3]);
          mma16816(t0, c0, 0u, c2, 0u, fa[kk + 1][0], fa[kk + 1][1]);
          mma16816(t1, c0, 0u, c2, 0u, fa[kk + 1][2], fa[kk + 1][3]);
        }
        float* store = nullptr;
        if (dist && sc_write && qrow < r)
          store = reinterpret_cast<float*>(sc_base + (int64_t)(vt - ntp) * sc_group_b + (qrow * 4 + (lane & 3)) * 16);
        softmax_pv((s0[0] + t0[0]) * p.scale_log2, (s0[1] + t0[1]) * p.scale_log2, (s1[0] + t1[0]) * p.scale_log2,
                   (s1[1] + t1[1]) * p.scale_log2, min(TOK, rem), mtile, fb, store, dist);
      }
      // the stage just used holds the new tile, or is free from now on
      if (NSTAGE == 3) { v0 = v1; v1 = v2; v2 = v_new; } else if (NSTAGE == 2) { v0 = v1; v1 = v_new; } else { v0 = v_new; }
      if (late_pending && walk_done) late_wait(s);
      if (++s == NSTAGE) { s = 0; ++round; }
    }
  }
  if (late_pending) late_wait(0);
  // A CTA with a stale copy marks the head: a large number added to the head's ticket word, which the CTA that
  // draws the last ticket sees (this thread's ticket comes later, to the same word).
  const bool cta_stale = late_check() || (p.force_redo && p.segment == 0);    // as seen by warp 0
  if (cta_stale && threadIdx.x == 0) atomicAdd(sched + SCHED_TICKET, REDO_MARK);

  if (failed) {
    if (lane == 0) atomicExch(p.err_flag, 1);
    // Drain the copies this warp still has in flight before its shared memory is reused: v0, v1, v2 sit in
    // the failing stage and the ones after it; stages before the failing one were refilled in this round
    // (next parity), the others still hold this round's tile.
    const int vq[3] = {v0, v1, v2};
    for (int i = 0; i < NSTAGE; ++i) {
      const int st = (fail_stage + i) % NSTAGE;
      if (vq[i] >= 0) mbar_wait(bar0 + st * 8, (st < fail_stage ? round + 1 : round) & 1);
    }
  }

  // ---- merge the warps of the CTA -------------------------------------------------------------
  l_row += __shfl_xor_sync(0xffffffffu, l_row, 1);
  l_row += __shfl_xor_sync(0xffffffffu, l_row, 2);
  ld_row += __shfl_xor_sync(0xffffffffu, ld_row, 1);
  ld_row += __shfl_xor_sync(0xffffffffu, ld_row, 2);
  __syncwarp();
  float* mine = reinterpret_cast<float*>(wbuf);    // [8 heads][D] acc, then [8] max, [8] sum, [8] distant sum
  if (qcol < r) {
#pragma unroll
    for (int cb = 0; cb < D / 16; ++cb) {
      mine[qcol * D + cb * 16 + qrow] = ot[cb][0];
      mine[qcol * D + cb * 16 + 8 + qrow] = ot[cb][2];
      if (qcol + 1 < r) {
        mine[(qcol + 1) * D + cb * 16 + qrow] = ot[cb][1];
        mine[(qcol + 1) * D + cb * 16 + 8 + qrow] = ot[cb][3];
      }
    }
  }
  if ((lane & 3) == 0) { mine[8 * D + qrow] = m_row; mine[8 * D + 8 + qrow] = l_row; mine[8 * D + 16 + qrow] = ld_row; }
  if (sc_write) fence_async_global();    // the stored logits are read through the async proxy
  __syncthreads();
  // all warps of the CTA have finished streaming: its share of the head's logits is stored; the head's DONE
  // count moves below, together with the CTA's ticket (see scores_complete)
  for (int idx = threadIdx.x; idx < r * D; idx += NW * 32) {
    const int h = idx / D, c = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w)
      M = fmaxf(M, reinterpret_cast<const float*>(smem + w * C::WARP_B)[8 * D + h]);
    float a = 0.f, l = 0.f, ld = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float* ow = reinterpret_cast<const float*>(smem + w * C::WARP_B);
      const float mw = ow[8 * D + h];
      const float sc = (mw == -INFINITY) ? 0.f : ex2(mw - M);
      a += ow[h * D + c] * sc;
      l += ow[8 * D + 8 + h] * sc;
      ld += ow[8 * D + 16 + h] * sc;
    }
    const int64_t ph = ((int64_t)b * y.H_q + kvh * r + h) * p.max_splits + split;
    p.part_acc[ph * D + c] = a;
    if (c == 0) *reinterpret_cast<float4*>(p.part_ml + ph * 4) = make_float4(M, l, ld, 0.f);
  }

  // ---- ticket: the CTA that publishes the last partial of this (sequence, KV head) combines ----
  // The barrier orders every thread's partial stores before thread 0's release at GPU scope
  // (cumulative), and the winner's acquire orders them before its reads.
  // Two forms.  General: every CTA takes a ticket and learns from the returned count whether it is the
  // last.  When the whole grid is resident at once (the host knows: closer = 1), the head's first CTA is
  // the one that combines: the others add their ticket without asking for the count and leave at once --
  // their slot on the SM goes to the next kernel a memory round trip earlier -- and the first CTA waits
  // (bounded) until the count is complete.  It cannot wait for a CTA that has no slot yet, because in that
  // mode every CTA of the grid gets one without anyone leaving.
  __shared__ int s_last, s_marks;
  fence_async_global();                  // the partials are read back through the async proxy
  __syncthreads();
  // One release for both of the head's counts: this CTA's logits and partials are visible before either moves.
  if (threadIdx.x == 0) {
    asm volatile("fence.acq_rel.gpu;" ::: "memory");
    if (sc_write && !cta_stale) asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;" ::"l"(sched + SCHED_DONE) : "memory");
  }
  if (p.closer && split != 0) {
    if (threadIdx.x == 0)
      asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;" ::"l"(sched + SCHED_TICKET) : "memory");
    trace_end(p);
    return;
  }
  if (threadIdx.x == 0) {
    int got;
    if (p.closer) {
      got = 0;
      bool all = nsplit == 1;
      for (uint32_t it = 0; it < WAIT_LIMIT && !all; ++it) {
        got = ld_acquire_gpu(sched + SCHED_TICKET);
        all = (got & (REDO_MARK - 1)) == nsplit - 1;
        if (!all) __nanosleep(64);
      }
      if (!all) atomicExch(p.err_flag, 1);                   // (the outputs of this head are then invalid)
      if (nsplit == 1) got = ld_acquire_gpu(sched + SCHED_TICKET);   // this CTA's own marks
    } else {
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(got) : "l"(sched + SCHED_TICKET) : "memory");
    }
    int last = (p.closer || (got & (REDO_MARK - 1)) == nsplit - 1) ? 1 : 0;
    if (last) {                                              // ready for the next launch
      sched[SCHED_TICKET] = 0; *ctr = 0;
      if (p.segment == 1) sched[SCHED_NEED] = 0;             // this CTA's warps set the bits below
      // Every CTA of the head has finished streaming: its stored logits, stashed queries and cache rows are
      // complete, which is what a later launch waits for -- unless a warp found its early copies stale (it added
      // its mark to this word before its CTA took its ticket); then the head is redone first.
      if (got >= REDO_MARK) last = 2;
    }
    s_last = last;
    s_marks = got >> REDO_SHIFT;
  }
  __syncthreads();
  if (!s_last) {
    trace_end(p);
    return;
  }
  if (s_last == 2) {
    if (fused && warp == 0 && lane < D / 4) {     // the new token's rows again, from the final k and v
      const bool isv = lane >= D / 8;
      const int sub = lane % (D / 8);
      *reinterpret_cast<uint4*>(const_cast<uint16_t*>(p.arena) + ((int64_t)(isv ? rowVp : rowKp) + rA) * D + sub * 8) =
          *reinterpret_cast<const uint4*>((isv ? p.new_v : p.new_k) + ((int64_t)b * y.H_kv + kvh) * D + sub * 8);
    }
    __syncthreads();
    redo_head<D>(p.arena, p.q, p.stash, p.out, p.dlse, p.scale_log2, (int64_t)b * y.H_q + kvh * r, r, n_p, n_d, rowKp, rowVp,
                 rowKd, rowVd, sc_base, sc_group_b, is_low, sc_write, q_own, q_st);
    fence_async_global();
    __syncthreads();
    // the logits are rewritten: the DONE counts that the marked CTAs held back
    if (threadIdx.x == 0 && sc_write)
      asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(sched + SCHED_DONE), "r"(s_marks) : "memory");
    trace_end(p);
    return;
  }

  // ---- combine: every warp merges the partials of its own query heads, on its own -----------
  // The (max, sum) pairs and the partial rows of a head come into the warp's ring with bulk
  // copies (one memory round trip); rounds of CROWS rows if a head has more splits than fit.
  constexpr int CPL = D / 32;                 // channels per lane
  const uint32_t w_ml = wbuf_s + C::CML_OFF, w_w = wbuf_s + C::CW_OFF, w_rows = wbuf_s + C::CROW_OFF;
  const int64_t ph0 = ((int64_t)b * y.H_q + kvh * r) * p.max_splits;     // partial row of (head 0, split 0)
  uint32_t cphase = 0;
  bool cfail = false;
  const int need_in = p.segment == 2 ? sched[SCHED_NEED] : 0;   // heads that left a proximal state to merge with
  for (int h = warp; h < r && !cfail; h += NW) {
    if (p.segment == 2 && !((need_in >> h) & 1)) continue;      // this head took its output from the proximal launch
    const int64_t ph = ph0 + (int64_t)h * p.max_splits;
    const int64_t hq = (int64_t)b * y.H_q + kvh * r + h;         // query head
    float acc[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) acc[j] = 0.f;
    float inv = 0.f, m_all = -INFINITY, l_all = 0.f;
    // state of the proximal launch (segment 2): one more partial (max, sum, acc); requested early
    float st_m = -INFINITY, st_l = 0.f, st_w = 0.f, st_acc[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) st_acc[j] = 0.f;
    if (p.segment == 2) {
      st_m = p.state_ml[hq * 2]; st_l = p.state_ml[hq * 2 + 1];
#pragma unroll
      for (int j = 0; j < CPL; ++j) st_acc[j] = p.state_acc[hq * D + lane * CPL + j];
    }
    for (int r0 = 0; r0 < nsplit; r0 += C::CROWS) {
      const int r1 = min(nsplit, r0 + C::CROWS);
      if (lane == 0) {
        fence_async_global();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const uint32_t ml_bytes = (uint32_t)p.max_splits * 16u;
        mbar_expect_tx(cbar, (uint32_t)(r1 - r0) * D * 4u + (r0 == 0 ? ml_bytes : 0u));
        if (r0 == 0) bulk_load(w_ml, p.part_ml + ph * 4, ml_bytes, cbar);
        bulk_load(w_rows, p.part_acc + (ph + r0) * D, (uint32_t)(r1 - r0) * D * 4u, cbar);
      }
      if (!__all_sync(0xffffffffu, mbar_wait(cbar, cphase & 1))) { cfail = true; break; }
      ++cphase;
      if (r0 == 0) {                          // weights 2^(m_s - M) of the splits and 1 / sum, once per head
        float4 ml[MAX_SPLITS_CAP / 32];       // (max, sum, distant part of the sum, -) of a split
        float mloc = st_m;
#pragma unroll
        for (int k = 0; k < MAX_SPLITS_CAP / 32; ++k) {
          const int sp = lane + 32 * k;
          ml[k] = sp < nsplit ? lds_f32x4(w_ml + sp * 16) : make_float4(-INFINITY, 0.f, 0.f, 0.f);
          mloc = fmaxf(mloc, ml[k].x);
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, o2));
        float lloc = 0.f, ldloc = 0.f;
#pragma unroll
        for (int k = 0; k < MAX_SPLITS_CAP / 32; ++k) {
          const int sp = lane + 32 * k;
          const float wgt = (ml[k].x == -INFINITY) ? 0.f : ex2(ml[k].x - mloc);
          if (sp < nsplit) sts_f32(w_w + sp * 4, wgt);
          lloc += ml[k].y * wgt;
          ldloc += ml[k].z * wgt;
        }
#pragma unroll
        for (int o2 = 16; o2 >= 1; o2 >>= 1) {
          lloc += __shfl_xor_sync(0xffffffffu, lloc, o2);
          ldloc += __shfl_xor_sync(0xffffffffu, ldloc, o2);
        }
        st_w = (st_m == -INFINITY) ? 0.f : ex2(st_m - mloc);
        lloc += st_l * st_w;
        m_all = mloc; l_all = lloc;
        inv = lloc > 0.f ? 1.f / lloc : 0.f;
        // the head's lowest layer leaves the log-sum-exp of its distant logits for the gate of the
        // block's other layers (a proximal-only launch sees no distant token: the distant launch writes it)
        if (sc_write && p.segment != 1 && lane == 0) p.dlse[hq] = ldloc > 0.f ? mloc + __log2f(ldloc) : -INFINITY;
        __syncwarp();
      }
      // eight rows per trip, the last trip padded with weight 0 on a valid row
      for (int row = r0; row < r1; row += 8) {
        float v[8][CPL], wg[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const bool in = row + u < r1;
          const int rr = in ? row + u : r0;
          wg[u] = in ? lds_f32(w_w + rr * 4) : 0.f;
          const uint32_t src = w_rows + (uint32_t)(rr - r0) * (D * 4) + lane * (CPL * 4);
          if constexpr (CPL == 4) {
            const float4 x = lds_f32x4(src);
            v[u][0] = x.x; v[u][1] = x.y; v[u][2] = x.z; v[u][3] = x.w;
          } else {
            const float2 x = lds_f32x2(src);
            v[u][0] = x.x; v[u][1] = x.y;
          }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
          for (int j = 0; j < CPL; ++j) acc[j] += v[u][j] * wg[u];
      }
      __syncwarp();                           // the rows are overwritten by the next round
    }
    if (cfail) break;
#pragma unroll
    for (int j = 0; j < CPL; ++j) acc[j] += st_acc[j] * st_w;
    if (p.segment == 1) {
      // Gate of Eq. 2 from the proximal sum of this launch and the distant sum the block's lowest
      // layer left: g = S_P / (S_P + S_D).  A head that reads the block's logits and has g >= tau
      // omits its distant tokens; so does any head without distant tokens.  The others leave their
      // proximal state for the distant launch.
      bool final_out = n_d == 0;
      if (!final_out && sc_read) {
        const float lse_p = m_all + __log2f(l_all), lse_d = p.dlse[hq];
        const float g = 1.f / (1.f + ex2(lse_d - lse_p));
        final_out = g >= p.gate_tau;
      }
      if (!final_out) {
        if (lane == 0) {
          p.state_ml[hq * 2] = m_all; p.state_ml[hq * 2 + 1] = l_all;
          atomicOr(sched + SCHED_NEED, 1 << h);
        }
#pragma unroll
        for (int j = 0; j < CPL; ++j) p.state_acc[hq * D + lane * CPL + j] = acc[j];
        continue;
      }
    }
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + hq * D + lane * CPL;
#pragma unroll
    for (int j = 0; j < CPL; j += 2)
      *reinterpret_cast<__nv_bfloat162*>(dst + j) = __floats2bfloat162_rn(acc[j] * inv, acc[j + 1] * inv);
  }
  if (cfail && lane == 0) atomicExch(p.err_flag, 1);
  __syncthreads();
  trace_end(p);
}

// Outputs of sequences that hold no token are zero (no split CTA exists to write them).
__global__ void pod_zero_empty_kernel(const DecodeParams p) {
  pdl_wait();
  pdl_launch_dependents();
  const int b = blockIdx.x;
  if (p.len[b] != 0) return;
  const int per = p.y.H_q * p.y.D;
  for (int i = threadIdx.x; i < per; i += blockDim.x) p.out[(int64_t)b * per + i] = 0;
}

cudaLaunchConfig_t pdl_config(cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem, cudaStream_t s) {
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cfg;
}

template <int D>
int launch_decode_t(const CUtensorMap& tmap, const DecodeParams& p, int grid_splits, cudaStream_t s) {
  using C = Cfg<D>;
  // the shared-memory attribute is a per-device setting of the kernel
  static bool configured[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaErrorInvalidDevice;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return (int)e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(attr, dim3(p.y.H_kv, grid_splits, p.y.B), dim3(C::NW * 32), C::SMEM, s);
  return (int)cudaLaunchKernelEx(&cfg, pod_decode_splitk_kernel<D>, tmap, p);
}

template <int D>
int resident_t() {
  using C = Cfg<D>;
  cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return 0;
  int nb = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, pod_decode_splitk_kernel<D>, C::NW * 32, C::SMEM);
  return e == cudaSuccess ? nb : 0;
}

}  // namespace

int decode_tile_tokens() { return TOK; }
int decode_warps_per_cta() { return DECODE_WARPS; }

int launch_decode(const CUtensorMap& tmap, const DecodeParams& p, int grid_splits, cudaStream_t s) {
  if (p.tiles_per_chunk < 1 || p.static_eighths < 0 || p.static_eighths > 8 || (p.max_splits & 1)) return (int)cudaErrorInvalidValue;
  if (p.y.D == 128) return launch_decode_t<128>(tmap, p, grid_splits, s);
  if (p.y.D == 64) return launch_decode_t<64>(tmap, p, grid_splits, s);
  return (int)cudaErrorInvalidValue;
}

int launch_zero_empty(const DecodeParams& p, cudaStream_t s) {
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(attr, dim3(p.y.B), dim3(128), 0, s);
  return (int)cudaLaunchKernelEx(&cfg, pod_zero_empty_kernel, p);
}

int decode_resident_ctas_per_sm(int D) {
  if (D == 128) return resident_t<128>();
  if (D == 64) return resident_t<64>();
  return 0;
}

}  // namespace pod
