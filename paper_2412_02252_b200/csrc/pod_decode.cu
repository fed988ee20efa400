// Split-K decode attention over the PoD layout, and the log-sum-exp combine.
//
// Grid (split, KV head, sequence).  A CTA owns a contiguous range of the sequence's tokens in
// "virtual" order -- proximal rows first (sink, then ring slots), distant rows after -- and
// its warps subdivide that range.  Each warp is an independent flash-decoding stream:
//   * lane 0 stages tiles of 16 K rows and 16 V rows into the warp's private shared-memory
//     ring with tiled TMA loads (one tensor map views the whole arena as [rows][d]; 128-byte
//     swizzle, no multicast) that complete on an mbarrier;
//   * logits: S[16 x 16] = Q[16 x d] K^T with mma.sync m16n8k16 (bf16 in, fp32 out).  The rows
//     of Q are the r <= 8 query heads of the KV head, zero-padded to 16; K fragments come from
//     ldmatrix on the swizzled tile, so the bf16 data is never unpacked by ALU instructions;
//   * one online softmax in base 2 runs over proximal and distant rows alike: at the boundary
//     only the Q fragments (own query for proximal rows, the block's lowest-layer query for
//     distant rows) and the tile coordinates change;
//   * values: O[16 x d] += P[16 x 16] V[16 x d], P rounded to bf16 in the accumulator-to-A
//     register layout, V fragments from ldmatrix.trans.
// An earlier CUDA-core version of this kernel (packed fp32 FMAs on unpacked bf16) was bound by
// instruction issue at half the memory rate; the tensor-core form needs about a tenth of the
// instructions and leaves the kernel memory-bound.
// Warps merge through shared memory; the CTA writes one fp32 partial (acc, max, sum) per
// query head.  The log-sum-exp combine of the partials (the gate of Eq. 2 generalised from two
// parts to n_splits parts) runs in the same launch: every CTA takes a ticket of its
// (sequence, KV head) after publishing its partial, and the CTA that draws the last ticket
// merges all of them and writes the bf16 output.  Nobody waits for anybody, so nothing can hang.
// A stand-alone combine kernel is kept for callers that want the two-launch form.
// The kernels are launched with programmatic stream serialization: everything above
// griddepcontrol.wait (barrier setup) overlaps the tail of the previous kernel in the stream.
// Every mbarrier wait is bounded; a wait that gives up raises the cache's error flag.
#include <cuda_bf16.h>

#include "pod_common.h"

namespace pod {

namespace {

constexpr int NW = 4;            // warps per CTA
constexpr int NSTAGE = 3;        // stages of each warp's ring
constexpr int TOK = 16;          // tokens per tile (one mma k-step of P V)
constexpr int CTAS_PER_SM = 2;
constexpr uint32_t WAIT_LIMIT = 1u << 20;

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
// L2 eviction policies.  Rows that are read once per decode step stream through with
// evict_first; the block's shared distant keys are kept with evict_last while later layers of
// the block will read them again in the same step.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ float ld_cg(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float4 ld_cg4(const float* p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
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
  static constexpr int NSUB = D / 64;                 // 128-byte wide sub-tiles per row
  static constexpr int SUB_B = TOK * 128;             // bytes of one sub-tile (1024-byte multiple)
  static constexpr int TILE_B = NSUB * SUB_B;         // bytes of one K (or V) tile
  static constexpr int STAGE_B = 2 * TILE_B;
  static constexpr int WARP_B = NSTAGE * STAGE_B;
  static constexpr int SMEM = NW * WARP_B + NW * NSTAGE * 8 + 1024;   // + slack to align to 1024
  static_assert(NW * WARP_B >= 8 * MAX_SPLITS_CAP * 4, "combine weights must fit the rings");
  static_assert(WARP_B >= (8 * D + 16) * 4, "merge scratch must fit the warp's ring");
};

template <int D>
__global__ void __launch_bounds__(NW * 32, CTAS_PER_SM)
pod_decode_splitk_kernel(const __grid_constant__ CUtensorMap tmap, const DecodeParams p) {
  using C = Cfg<D>;
  const Layout& y = p.y;
  const int r = y.H_q / y.H_kv;   // query heads per KV head (<= 8): rows of the Q operand

  const int b = blockIdx.z, kvh = blockIdx.y, split = blockIdx.x;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);   // swizzle atoms are 1024 B
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* wbuf = smem + warp * C::WARP_B;
  const uint32_t wbuf_s = smem_u32(wbuf);
  const uint32_t bar0 = smem_u32(smem + NW * C::WARP_B) + warp * NSTAGE * 8;
  if (lane == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // Everything below reads what earlier kernels of the stream wrote (lengths, cache rows, stash).
  pdl_wait();
  pdl_launch_dependents();

  const int n = p.by_value ? p.v_len[b] : p.len[b];
  const int64_t cap_d = p.by_value ? (int64_t)p.v_cap_d[b] : (int64_t)y.seq_cap_d[b];
  const int64_t seq_row = p.by_value ? p.v_row_base[b] : y.seq_row_base[b];
  const int nsplit = min(p.max_splits, (n + p.split_tokens - 1) / p.split_tokens);
  if (split >= nsplit) return;

  // ---- token ranges ---------------------------------------------------------------------
  const int n_p = min(n, y.S + y.W);
  const int c0 = (int)((int64_t)n * split / nsplit), c1 = (int)((int64_t)n * (split + 1) / nsplit);
  const int w0 = c0 + (int)((int64_t)(c1 - c0) * warp / NW);
  const int w1 = c0 + (int)((int64_t)(c1 - c0) * (warp + 1) / NW);
  const int pa0 = min(w0, n_p), pa1 = min(w1, n_p);              // proximal rows [pa0, pa1)
  const int da0 = max(w0, n_p) - n_p, da1 = max(w1, n_p) - n_p;  // distant rows  [da0, da1)
  const int ntp = (pa1 - pa0 + TOK - 1) / TOK, ntd = (da1 - da0 + TOK - 1) / TOK;
  const int nt = ntp + ntd;

  // arena rows of this (sequence, layer, head): tile coordinates of the tensor map
  const int rowKp = (int)(seq_row + prox_row(y, p.layer, 0, kvh));
  const int rowVp = (int)(seq_row + prox_row(y, p.layer, 1, kvh));
  const int rowKd = (int)(seq_row + distk_row(y, p.block, kvh, cap_d));
  const int rowVd = (int)(seq_row + distv_row(y, p.layer, kvh, cap_d));

  const uint64_t pol_stream = policy_evict_first();
  const uint64_t pol_distk = p.keep_distk ? policy_evict_last() : pol_stream;

  auto tile_rows = [&](int t) -> int {
    return t < ntp ? min(TOK, pa1 - (pa0 + t * TOK)) : min(TOK, da1 - (da0 + (t - ntp) * TOK));
  };
  auto issue = [&](int t) {   // lane 0 only.  Rows past the piece are other (finite) cache rows
    const int stage = t % NSTAGE;   // or zero fill past the arena; their logits are masked.
    const int yk = t < ntp ? rowKp + pa0 + t * TOK : rowKd + da0 + (t - ntp) * TOK;
    const int yv = t < ntp ? rowVp + pa0 + t * TOK : rowVd + da0 + (t - ntp) * TOK;
    const uint32_t bar = bar0 + stage * 8;
    const uint32_t dst = wbuf_s + stage * C::STAGE_B;
    mbar_expect_tx(bar, C::STAGE_B);
    const uint64_t pol_k = t < ntp ? pol_stream : pol_distk;
#pragma unroll
    for (int s = 0; s < C::NSUB; ++s) {
      tma_load_2d(dst + s * C::SUB_B, &tmap, s * 64, yk, bar, pol_k);
      tma_load_2d(dst + C::TILE_B + s * C::SUB_B, &tmap, s * 64, yv, bar, pol_stream);
    }
  };

  if (lane == 0) {
    for (int t = 0; t < NSTAGE && t < nt; ++t) issue(t);
  }

  // a lowest layer saves its query for the other layers of the block
  if (p.stash != nullptr && split == 0 && warp == 0 && lane < D / 8) {
    for (int h = 0; h < r; ++h) {
      const int64_t o = ((int64_t)b * y.H_q + kvh * r + h) * D + lane * 8;
      *reinterpret_cast<uint4*>(p.stash + o) = *reinterpret_cast<const uint4*>(p.q + o);
    }
  }
  __syncwarp();

  // ---- per-lane state -------------------------------------------------------------------
  const int qrow = lane >> 2;          // query head (row of S and O) owned by this lane's quad
  const int qcol = (lane & 3) * 2;     // first of the two columns this lane holds in a fragment
  uint32_t qa[D / 16][2];              // A fragments of Q: rows 0..7 only (rows 8..15 are zero)
  float o[D / 8][4];                   // O accumulators; [.][2], [.][3] belong to the zero rows
#pragma unroll
  for (int c = 0; c < D / 8; ++c) { o[c][0] = o[c][1] = o[c][2] = o[c][3] = 0.f; }
  float m_row = -INFINITY, l_row = 0.f;
  bool failed = false;

  auto load_q = [&](const uint16_t* qsrc) {
    const uint16_t* base = qsrc + ((int64_t)b * y.H_q + kvh * r + qrow) * D + qcol;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      qa[kk][0] = qrow < r ? *reinterpret_cast<const uint32_t*>(base + kk * 16) : 0u;
      qa[kk][1] = qrow < r ? *reinterpret_cast<const uint32_t*>(base + kk * 16 + 8) : 0u;
    }
  };

  // ldmatrix lane addressing inside a [TOK][128 B] sub-tile with the 128-byte swizzle:
  // 16-byte chunk c of row t lives at t * 128 + ((c ^ (t & 7)) << 4).
  const int lm = lane >> 3, lr = lane & 7;
  // K (non-transposed): matrices (tokens 0-7, chunk 2kk), (0-7, 2kk+1), (8-15, 2kk), (8-15, 2kk+1)
  const int k_tok = (lm >> 1) * 8 + lr, k_chunk = lm & 1;
  // V (transposed): matrices (tokens 0-7, chunk c), (8-15, c), (0-7, c+1), (8-15, c+1)
  const int v_tok = (lm & 1) * 8 + lr, v_chunk = lm >> 1;

  int t = 0;
  for (; t < nt; ++t) {
    if (t == 0 || t == ntp) load_q(t < ntp ? p.q : p.q_low);
    const int stage = t % NSTAGE;
    if (!__all_sync(0xffffffffu, mbar_wait(bar0 + stage * 8, (t / NSTAGE) & 1))) { failed = true; break; }
    const int cnt = tile_rows(t);
    const uint32_t ks = wbuf_s + stage * C::STAGE_B;
    const uint32_t vs = ks + C::TILE_B;

    // ---- S = Q K^T ------------------------------------------------------------------------
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const int chunk = 2 * kk + k_chunk;          // 16-byte chunk of the row
      uint32_t bfr[4];
      ldsm4(ks + (chunk >> 3) * C::SUB_B + k_tok * 128 + (((chunk & 7) ^ (k_tok & 7)) << 4), bfr);
      mma16816(s0, qa[kk][0], 0u, qa[kk][1], 0u, bfr[0], bfr[1]);
      mma16816(s1, qa[kk][0], 0u, qa[kk][1], 0u, bfr[2], bfr[3]);
    }
    // ---- online softmax (base 2) over this lane's row -----------------------------------------
    float a00 = (qcol < cnt) ? s0[0] * p.scale_log2 : -INFINITY;
    float a01 = (qcol + 1 < cnt) ? s0[1] * p.scale_log2 : -INFINITY;
    float a10 = (qcol + 8 < cnt) ? s1[0] * p.scale_log2 : -INFINITY;
    float a11 = (qcol + 9 < cnt) ? s1[1] * p.scale_log2 : -INFINITY;
    float mx = fmaxf(fmaxf(a00, a01), fmaxf(a10, a11));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    if (__any_sync(0xffffffffu, mx > m_row)) {
      const float m_new = fmaxf(m_row, mx);
      const float alpha = ex2(m_row - m_new);       // 0 on the first tile, 1 if unchanged
      m_row = m_new;
      l_row *= alpha;
#pragma unroll
      for (int c = 0; c < D / 8; ++c) { o[c][0] *= alpha; o[c][1] *= alpha; }
    }
    a00 = ex2(a00 - m_row); a01 = ex2(a01 - m_row); a10 = ex2(a10 - m_row); a11 = ex2(a11 - m_row);
    l_row += (a00 + a01) + (a10 + a11);
    const uint32_t pa0 = pack_bf16(a00, a01), pa2 = pack_bf16(a10, a11);
    // ---- O += P V ---------------------------------------------------------------------------
#pragma unroll
    for (int c = 0; c < D / 8; c += 2) {
      const int chunk = c + v_chunk;
      uint32_t bfr[4];
      ldsm4_t(vs + (chunk >> 3) * C::SUB_B + v_tok * 128 + (((chunk & 7) ^ (v_tok & 7)) << 4), bfr);
      mma16816(o[c], pa0, 0u, pa2, 0u, bfr[0], bfr[1]);
      mma16816(o[c + 1], pa0, 0u, pa2, 0u, bfr[2], bfr[3]);
    }
    __syncwarp();                          // all lanes are done reading this stage
    if (lane == 0 && t + NSTAGE < nt) issue(t + NSTAGE);
  }

  if (failed) {
    if (lane == 0) atomicExch(p.err_flag, 1);
    // drain the copies this warp still has in flight before its shared memory is reused
    for (int u = t; u < nt && u < t + NSTAGE; ++u) mbar_wait(bar0 + (u % NSTAGE) * 8, (u / NSTAGE) & 1);
  }

  // ---- merge the warps of the CTA -------------------------------------------------------------
  l_row += __shfl_xor_sync(0xffffffffu, l_row, 1);
  l_row += __shfl_xor_sync(0xffffffffu, l_row, 2);
  __syncwarp();
  float* mine = reinterpret_cast<float*>(wbuf);    // [8][D] acc, then [8] max, [8] sum
#pragma unroll
  for (int c = 0; c < D / 8; ++c)
    *reinterpret_cast<float2*>(mine + qrow * D + c * 8 + qcol) = make_float2(o[c][0], o[c][1]);
  if ((lane & 3) == 0) { mine[8 * D + qrow] = m_row; mine[8 * D + 8 + qrow] = l_row; }
  __syncthreads();

  for (int idx = threadIdx.x; idx < r * D; idx += NW * 32) {
    const int h = idx / D, c = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w)
      M = fmaxf(M, reinterpret_cast<const float*>(smem + w * C::WARP_B)[8 * D + h]);
    float a = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float* ow = reinterpret_cast<const float*>(smem + w * C::WARP_B);
      const float mw = ow[8 * D + h];
      const float sc = (mw == -INFINITY) ? 0.f : ex2(mw - M);
      a += ow[h * D + c] * sc;
      l += ow[8 * D + 8 + h] * sc;
    }
    const int64_t ph = ((int64_t)b * y.H_q + kvh * r + h) * p.max_splits + split;
    p.part_acc[ph * D + c] = a;
    if (c == 0) { p.part_ml[ph * 2] = M; p.part_ml[ph * 2 + 1] = l; }
  }
  if (p.tickets == nullptr) return;      // two-launch form: a combine kernel follows

  // ---- ticket: the CTA that publishes the last partial of this (sequence, KV head) combines ----
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    int* tk = p.tickets + (int64_t)b * y.H_kv + kvh;
    const int got = atomicAdd(tk, 1);
    s_last = (got == nsplit - 1);
    if (s_last) *tk = 0;                 // ready for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  float* s_w = reinterpret_cast<float*>(smem);          // [8][MAX_SPLITS_CAP] split weights
  for (int h = warp; h < r; h += NW) {
    const int64_t ph = ((int64_t)b * y.H_q + kvh * r + h) * p.max_splits;
    float mloc = -INFINITY;
    for (int s = lane; s < nsplit; s += 32) mloc = fmaxf(mloc, ld_cg(p.part_ml + (ph + s) * 2));
#pragma unroll
    for (int o2 = 16; o2 >= 1; o2 >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, o2));
    float lloc = 0.f;
    for (int s = lane; s < nsplit; s += 32) {
      const float ms = ld_cg(p.part_ml + (ph + s) * 2);
      const float wgt = (ms == -INFINITY) ? 0.f : ex2(ms - mloc);
      s_w[h * MAX_SPLITS_CAP + s] = wgt;
      lloc += ld_cg(p.part_ml + (ph + s) * 2 + 1) * wgt;
    }
#pragma unroll
    for (int o2 = 16; o2 >= 1; o2 >>= 1) lloc += __shfl_xor_sync(0xffffffffu, lloc, o2);
    __syncwarp();
    const float inv = lloc > 0.f ? 1.f / lloc : 0.f;
    // each lane owns 4 consecutive channels (d = 128) or 2 (d = 64)
    constexpr int CPL = D / 32;
    float acc[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) acc[j] = 0.f;
    const float* src = p.part_acc + ph * D + lane * CPL;
    int s = 0;
    for (; s + 4 <= nsplit; s += 4) {
      float v[4][CPL];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if constexpr (CPL == 4) {
          const float4 x = ld_cg4(src + (int64_t)(s + u) * D);
          v[u][0] = x.x; v[u][1] = x.y; v[u][2] = x.z; v[u][3] = x.w;
        } else {
#pragma unroll
          for (int j = 0; j < CPL; ++j) v[u][j] = ld_cg(src + (int64_t)(s + u) * D + j);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float wgt = s_w[h * MAX_SPLITS_CAP + s + u];
#pragma unroll
        for (int j = 0; j < CPL; ++j) acc[j] += v[u][j] * wgt;
      }
    }
    for (; s < nsplit; ++s) {
      const float wgt = s_w[h * MAX_SPLITS_CAP + s];
#pragma unroll
      for (int j = 0; j < CPL; ++j) acc[j] += ld_cg(src + (int64_t)s * D + j) * wgt;
    }
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)b * y.H_q + kvh * r + h) * D + lane * CPL;
#pragma unroll
    for (int j = 0; j < CPL; j += 2)
      *reinterpret_cast<__nv_bfloat162*>(dst + j) = __floats2bfloat162_rn(acc[j] * inv, acc[j + 1] * inv);
  }
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

// Merge of the split partials of one (sequence, query head): the gate of Eq. 2 generalised
// from two parts to n_splits parts.  Block = D threads, grid (H_q, B).
template <int D>
__global__ void __launch_bounds__(D) pod_combine_kernel(const DecodeParams p) {
  pdl_wait();
  pdl_launch_dependents();
  const int hq = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const int n = p.len[b];
  const int nsplit = min(p.max_splits, (n + p.split_tokens - 1) / p.split_tokens);
  const int64_t ph = ((int64_t)b * p.y.H_q + hq) * p.max_splits;
  __shared__ float s_w[MAX_SPLITS_CAP];     // weight of each split: 2^(m_s - M)
  __shared__ float s_red[2][4];
  // pass 1: every thread takes some splits' (max, sum); block-wide max
  float mloc = -INFINITY;
  for (int s = c; s < nsplit; s += D) mloc = fmaxf(mloc, p.part_ml[(ph + s) * 2]);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, o));
  if ((c & 31) == 0) s_red[0][c >> 5] = mloc;
  __syncthreads();
  float M = s_red[0][0];
  for (int w = 1; w < D / 32; ++w) M = fmaxf(M, s_red[0][w]);
  float lloc = 0.f;
  for (int s = c; s < nsplit; s += D) {
    const float ms = p.part_ml[(ph + s) * 2];
    const float wgt = (ms == -INFINITY) ? 0.f : ex2(ms - M);
    s_w[s] = wgt;
    lloc += p.part_ml[(ph + s) * 2 + 1] * wgt;
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) lloc += __shfl_xor_sync(0xffffffffu, lloc, o);
  if ((c & 31) == 0) s_red[1][c >> 5] = lloc;
  __syncthreads();
  float l = 0.f;
  for (int w = 0; w < D / 32; ++w) l += s_red[1][w];
  // pass 2: channel c over the splits, loads independent of one another
  float a = 0.f;
  int s = 0;
  for (; s + 4 <= nsplit; s += 4) {
    const float v0 = p.part_acc[(ph + s) * D + c], v1 = p.part_acc[(ph + s + 1) * D + c];
    const float v2 = p.part_acc[(ph + s + 2) * D + c], v3 = p.part_acc[(ph + s + 3) * D + c];
    a += v0 * s_w[s] + v1 * s_w[s + 1] + v2 * s_w[s + 2] + v3 * s_w[s + 3];
  }
  for (; s < nsplit; ++s) a += p.part_acc[(ph + s) * D + c] * s_w[s];
  const float out = (l > 0.f) ? a / l : 0.f;
  reinterpret_cast<__nv_bfloat16*>(p.out)[((int64_t)b * p.y.H_q + hq) * D + c] = __float2bfloat16_rn(out);
}

cudaLaunchAttribute g_pdl_attr[1];
cudaLaunchConfig_t pdl_config(dim3 grid, dim3 block, size_t smem, cudaStream_t s) {
  g_pdl_attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  g_pdl_attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cfg.attrs = g_pdl_attr; cfg.numAttrs = 1;
  return cfg;
}

template <int D>
int launch_decode_t(const CUtensorMap& tmap, const DecodeParams& p, int grid_splits, cudaStream_t s) {
  using C = Cfg<D>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return (int)e;
    configured = true;
  }
  cudaLaunchConfig_t cfg = pdl_config(dim3(grid_splits, p.y.H_kv, p.y.B), dim3(NW * 32), C::SMEM, s);
  return (int)cudaLaunchKernelEx(&cfg, pod_decode_splitk_kernel<D>, tmap, p);
}

template <int D>
int resident_t() {
  using C = Cfg<D>;
  cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return 0;
  int nb = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, pod_decode_splitk_kernel<D>, NW * 32, C::SMEM);
  return e == cudaSuccess ? nb : 0;
}

}  // namespace

int decode_tile_tokens() { return TOK; }

int launch_decode(const CUtensorMap& tmap, const DecodeParams& p, int grid_splits, cudaStream_t s) {
  if (p.y.D == 128) return launch_decode_t<128>(tmap, p, grid_splits, s);
  if (p.y.D == 64) return launch_decode_t<64>(tmap, p, grid_splits, s);
  return (int)cudaErrorInvalidValue;
}

int launch_combine(const DecodeParams& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg = pdl_config(dim3(p.y.H_q, p.y.B), dim3(p.y.D), 0, s);
  if (p.y.D == 128) return (int)cudaLaunchKernelEx(&cfg, pod_combine_kernel<128>, p);
  return (int)cudaLaunchKernelEx(&cfg, pod_combine_kernel<64>, p);
}

int launch_zero_empty(const DecodeParams& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg = pdl_config(dim3(p.y.B), dim3(128), 0, s);
  return (int)cudaLaunchKernelEx(&cfg, pod_zero_empty_kernel, p);
}

int decode_resident_ctas_per_sm(int D) {
  if (D == 128) return resident_t<128>();
  if (D == 64) return resident_t<64>();
  return 0;
}

}  // namespace pod
