// Split-K decode attention over the PoD layout, and the log-sum-exp combine.
//
// Grid (split, KV head, sequence).  A CTA owns a contiguous range of the sequence's tokens in
// "virtual" order -- proximal rows first (sink, then ring slots), distant rows after -- and
// its warps subdivide that range.  Each warp is an independent flash-decoding stream:
//   * lane 0 stages tiles of K rows and V rows into the warp's private shared-memory ring
//     with 1-D bulk async copies (TMA, no multicast) that complete on an mbarrier;
//   * the lanes of a row group each hold 8 of the d channels of q (all r query heads of the
//     KV head) in registers, multiply their 16-byte chunk of a K row against them with packed
//     fp32 FMAs, and a transposing butterfly leaves one (token, head) logit per lane;
//   * one online softmax in base 2 (logits pre-scaled by log2 e) runs over proximal and
//     distant rows alike: only the query registers (own query for proximal rows, the block's
//     lowest-layer query for distant rows) and the K/V base pointers change at the boundary;
//   * probabilities go through a small shared buffer and are applied to the V chunk of
//     each lane with packed fp32 FMAs.
// Warps merge through shared memory; the CTA writes one fp32 partial (acc, max, sum) per
// query head.  A second kernel merges the partials of a (sequence, head) and rounds to bf16.
// Every mbarrier wait is bounded; a wait that gives up raises the cache's error flag.
#include <cuda_bf16.h>

#include "pod_common.h"

namespace pod {

namespace {

constexpr int NW = 8;            // warps per CTA
constexpr int NSTAGE = 3;        // stages of each warp's ring
constexpr int TILE_BYTES = 2048; // bytes of one K (or V) tile of a warp's stage
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
// 1-D bulk copy global -> shared, completing `bytes` on the mbarrier.  Source, destination
// and size are multiples of 16 bytes (rows are 128 or 256 bytes).
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
// two packed bf16 -> two fp32 (exact)
__device__ __forceinline__ float2 bf2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ void unpack8(const uint4& r, float2 (&f)[4]) {
  f[0] = bf2(r.x); f[1] = bf2(r.y); f[2] = bf2(r.z); f[3] = bf2(r.w);
}

template <int D, int R>
struct Cfg {
  static constexpr int LPR = D / 8;            // lanes per row
  static constexpr int NG = 32 / LPR;          // row groups per warp
  static constexpr int TG = LPR / R;           // tokens per row group per iteration
  static constexpr int TOK_IT = NG * TG;       // tokens per iteration (= 32 / R)
  static constexpr int ROWB = D * 2;
  static constexpr int TILE_B = TILE_BYTES;    // bytes of one K (or V) tile
  static constexpr int TOK = TILE_B / ROWB;    // tokens per stage
  static constexpr int ITERS = TOK / TOK_IT;   // softmax iterations per stage
  static constexpr int WARP_B = NSTAGE * 2 * TILE_B;
  static constexpr int PS_FLOATS = 2 * TOK_IT * R;   // double-buffered probabilities
  static constexpr int SMEM = NW * WARP_B + NW * PS_FLOATS * 4 + NW * NSTAGE * 8;
  static_assert(TG >= 1, "r must not exceed d / 8");
  static_assert(ITERS >= 1 && ITERS * TOK_IT == TOK, "a stage holds whole iterations");
  static_assert(WARP_B >= (R * D + 2 * R) * 4, "merge scratch must fit the warp's ring");
};

template <int D, int R>
__global__ void __launch_bounds__(NW * 32, (R > 4 ? 1 : 2)) pod_decode_splitk_kernel(const DecodeParams p) {
  using C = Cfg<D, R>;
  constexpr int LPR = C::LPR, TG = C::TG, TOK_IT = C::TOK_IT, TOK = C::TOK, ROWB = C::ROWB;
  constexpr int ITERS = C::ITERS;
  const Layout& y = p.y;
  const int r = y.H_q / y.H_kv;   // query heads per KV head; R >= r is the compute width

  const int b = blockIdx.z, kvh = blockIdx.y, split = blockIdx.x;
  const int n = p.len[b];
  const int nsplit = min(p.max_splits, (n + p.split_tokens - 1) / p.split_tokens);
  if (split >= nsplit) return;

  extern __shared__ __align__(128) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gi = lane / LPR, sub = lane % LPR;
  unsigned char* wbuf = smem + warp * C::WARP_B;
  float* ps = reinterpret_cast<float*>(smem + NW * C::WARP_B) + warp * C::PS_FLOATS;
  const uint32_t bar0 = smem_u32(smem + NW * C::WARP_B + NW * C::PS_FLOATS * 4) + warp * NSTAGE * 8;
  const uint32_t wbuf_s = smem_u32(wbuf);
  const uint32_t ps_s = smem_u32(ps);

  // ---- token ranges -----------------------------------------------------------------
  const int n_p = min(n, y.S + y.W);
  const int c0 = (int)((int64_t)n * split / nsplit), c1 = (int)((int64_t)n * (split + 1) / nsplit);
  const int w0 = c0 + (int)((int64_t)(c1 - c0) * warp / NW);
  const int w1 = c0 + (int)((int64_t)(c1 - c0) * (warp + 1) / NW);
  const int pa0 = min(w0, n_p), pa1 = min(w1, n_p);              // proximal rows [pa0, pa1)
  const int da0 = max(w0, n_p) - n_p, da1 = max(w1, n_p) - n_p;  // distant rows  [da0, da1)
  const int ntp = (pa1 - pa0 + TOK - 1) / TOK, ntd = (da1 - da0 + TOK - 1) / TOK;
  const int nt = ntp + ntd;

  const int64_t cap_d = y.seq_cap_d[b];
  const uint16_t* seq_base = p.arena + y.seq_row_base[b] * D;
  const uint16_t* Kp = seq_base + prox_row(y, p.layer, 0, kvh) * D;
  const uint16_t* Vp = seq_base + prox_row(y, p.layer, 1, kvh) * D;
  const uint16_t* Kd = seq_base + distk_row(y, p.block, kvh, cap_d) * D;
  const uint16_t* Vd = seq_base + distv_row(y, p.layer, kvh, cap_d) * D;

  auto tile_rows = [&](int t) -> int {
    return t < ntp ? min(TOK, pa1 - (pa0 + t * TOK)) : min(TOK, da1 - (da0 + (t - ntp) * TOK));
  };
  auto issue = [&](int t) {   // lane 0 only
    const int stage = t % NSTAGE;
    const int cnt = tile_rows(t);
    const uint16_t *kp, *vp;
    if (t < ntp) { const int64_t off = pa0 + (int64_t)t * TOK; kp = Kp + off * D; vp = Vp + off * D; }
    else { const int64_t off = da0 + (int64_t)(t - ntp) * TOK; kp = Kd + off * D; vp = Vd + off * D; }
    const uint32_t bar = bar0 + stage * 8;
    const uint32_t bytes = (uint32_t)cnt * ROWB;
    mbar_expect_tx(bar, 2 * bytes);
    bulk_g2s(wbuf_s + stage * 2 * C::TILE_B, kp, bytes, bar);
    bulk_g2s(wbuf_s + stage * 2 * C::TILE_B + C::TILE_B, vp, bytes, bar);
  };

  if (lane == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(bar0 + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int t = 0; t < NSTAGE && t < nt; ++t) issue(t);
  }

  // a lowest layer saves its query for the other layers of the block
  if (p.stash != nullptr && split == 0 && warp == 0 && gi == 0) {
    for (int h = 0; h < r; ++h) {
      const int64_t o = ((int64_t)b * y.H_q + kvh * r + h) * D + sub * 8;
      *reinterpret_cast<uint4*>(p.stash + o) = *reinterpret_cast<const uint4*>(p.q + o);
    }
  }
  __syncwarp();

  // ---- per-lane state -----------------------------------------------------------------
  float2 qr[R][4];            // this lane's 8 channels of the r queries, scaled to log2 units
  float2 acc[R][4];           // this lane's 8 channels of the r outputs (row group partial)
#pragma unroll
  for (int h = 0; h < R; ++h)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[h][j] = make_float2(0.f, 0.f);
  const int own_h = sub % R;  // the (token, head) pair whose logit lands in this lane
  const int own_t = gi * TG + sub / R;
  float m_own = -INFINITY, l_own = 0.f;
  bool failed = false;

  auto load_q = [&](const uint16_t* qsrc) {
#pragma unroll
    for (int h = 0; h < R; ++h) {
      uint4 raw = make_uint4(0u, 0u, 0u, 0u);   // padded heads score 0 and are never written
      if (h < r)
        raw = *reinterpret_cast<const uint4*>(qsrc + ((int64_t)b * y.H_q + kvh * r + h) * D + sub * 8);
      float2 f[4];
      unpack8(raw, f);
#pragma unroll
      for (int j = 0; j < 4; ++j) qr[h][j] = make_float2(f[j].x * p.scale_log2, f[j].y * p.scale_log2);
    }
  };

  int t = 0;
  for (; t < nt; ++t) {
    if (t == 0 || t == ntp) load_q(t < ntp ? p.q : p.q_low);
    const int stage = t % NSTAGE;
    if (!__all_sync(0xffffffffu, mbar_wait(bar0 + stage * 8, (t / NSTAGE) & 1))) { failed = true; break; }
    const int cnt = tile_rows(t);
    const uint32_t ks = wbuf_s + stage * 2 * C::TILE_B + sub * 16;
    const uint32_t vs = ks + C::TILE_B;

#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      if (it * TOK_IT >= cnt) break;
      // ---- logits: TG rows of this row group against r queries -------------------------
      float v[LPR];
#pragma unroll
      for (int tt = 0; tt < TG; ++tt) {
        const int row = min(it * TOK_IT + gi * TG + tt, cnt - 1);
        float2 kf[4];
        unpack8(lds128(ks + row * ROWB), kf);
#pragma unroll
        for (int h = 0; h < R; ++h) {
          float2 a = __fmul2_rn(kf[0], qr[h][0]);
          a = __ffma2_rn(kf[1], qr[h][1], a);
          a = __ffma2_rn(kf[2], qr[h][2], a);
          a = __ffma2_rn(kf[3], qr[h][3], a);
          v[tt * R + h] = a.x + a.y;
        }
      }
      // transposing butterfly over the LPR lanes of the row group: LPR values -> 1 per lane
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < o; ++i) {
          const float send = up ? v[i] : v[i + o];
          const float keep = up ? v[i + o] : v[i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
      }
      float s = (it * TOK_IT + own_t < cnt) ? v[0] : -INFINITY;
      // ---- online softmax ---------------------------------------------------------------
      float mx = s;
#pragma unroll
      for (int o = R; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      if (__any_sync(0xffffffffu, mx > m_own)) {
        const float m_new = fmaxf(m_own, mx);
        const float alpha = ex2(m_own - m_new);     // 0 on the first tile, 1 if unchanged
        l_own *= alpha;
        m_own = m_new;
#pragma unroll
        for (int h = 0; h < R; ++h) {
          const float ah = __shfl_sync(0xffffffffu, alpha, h);
          const float2 a2 = make_float2(ah, ah);
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[h][j] = __fmul2_rn(acc[h][j], a2);
        }
      }
      const float pr = ex2(s - m_own);
      l_own += pr;
      float* psb = ps + (it & 1) * (TOK_IT * R);
      psb[own_t * R + own_h] = pr;
      __syncwarp();
      // ---- values -------------------------------------------------------------------------
      const uint32_t psb_s = ps_s + (it & 1) * (TOK_IT * R * 4);
#pragma unroll
      for (int tt = 0; tt < TG; ++tt) {
        const int row = min(it * TOK_IT + gi * TG + tt, cnt - 1);
        float2 vf[4];
        unpack8(lds128(vs + row * ROWB), vf);
        float pw[R];
        if constexpr (R == 8) {
          const uint4 a = lds128(psb_s + (gi * TG + tt) * R * 4), c = lds128(psb_s + (gi * TG + tt) * R * 4 + 16);
          pw[0] = __uint_as_float(a.x); pw[1] = __uint_as_float(a.y); pw[2] = __uint_as_float(a.z); pw[3] = __uint_as_float(a.w);
          pw[4] = __uint_as_float(c.x); pw[5] = __uint_as_float(c.y); pw[6] = __uint_as_float(c.z); pw[7] = __uint_as_float(c.w);
        } else if constexpr (R == 4) {
          const uint4 a = lds128(psb_s + (gi * TG + tt) * R * 4);
          pw[0] = __uint_as_float(a.x); pw[1] = __uint_as_float(a.y); pw[2] = __uint_as_float(a.z); pw[3] = __uint_as_float(a.w);
        } else {
#pragma unroll
          for (int h = 0; h < R; ++h) pw[h] = psb[(gi * TG + tt) * R + h];
        }
#pragma unroll
        for (int h = 0; h < R; ++h) {
          const float2 p2 = make_float2(pw[h], pw[h]);
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[h][j] = __ffma2_rn(vf[j], p2, acc[h][j]);
        }
      }
    }
    __syncwarp();                          // all lanes are done reading this stage
    if (lane == 0 && t + NSTAGE < nt) issue(t + NSTAGE);
  }

  if (failed) {
    if (lane == 0) atomicExch(p.err_flag, 1);
    // drain the copies this warp still has in flight before its shared memory is reused
    for (int u = t; u < nt && u < t + NSTAGE; ++u) mbar_wait(bar0 + (u % NSTAGE) * 8, (u / NSTAGE) & 1);
  }

  // ---- merge the row groups of the warp, then the warps of the CTA ------------------------
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
    for (int h = 0; h < R; ++h)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        acc[h][j].x += __shfl_xor_sync(0xffffffffu, acc[h][j].x, o);
        acc[h][j].y += __shfl_xor_sync(0xffffffffu, acc[h][j].y, o);
      }
#pragma unroll
  for (int o = R; o < 32; o <<= 1) l_own += __shfl_xor_sync(0xffffffffu, l_own, o);

  __syncwarp();
  float* mine = reinterpret_cast<float*>(wbuf);    // [R][D] acc, then [R] max, [R] sum
  if (gi == 0) {
#pragma unroll
    for (int h = 0; h < R; ++h)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float2*>(mine + h * D + sub * 8 + j * 2) = acc[h][j];
  }
  if (lane < R) { mine[R * D + lane] = m_own; mine[R * D + R + lane] = l_own; }
  __syncthreads();

  for (int idx = threadIdx.x; idx < R * D; idx += NW * 32) {
    const int h = idx / D, c = idx % D;
    if (h >= r) break;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w)
      M = fmaxf(M, reinterpret_cast<const float*>(smem + w * C::WARP_B)[R * D + h]);
    float a = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float* o = reinterpret_cast<const float*>(smem + w * C::WARP_B);
      const float mw = o[R * D + h];
      const float sc = (mw == -INFINITY) ? 0.f : ex2(mw - M);
      a += o[h * D + c] * sc;
      l += o[R * D + R + h] * sc;
    }
    const int64_t ph = ((int64_t)b * y.H_q + kvh * r + h) * p.max_splits + split;
    p.part_acc[ph * D + c] = a;
    if (c == 0) { p.part_ml[ph * 2] = M; p.part_ml[ph * 2 + 1] = l; }
  }
}

// Merge of the split partials of one (sequence, query head): the gate of Eq. 2 generalised
// from two parts to n_splits parts.  Block = D threads, grid (H_q, B).
template <int D>
__global__ void __launch_bounds__(D) pod_combine_kernel(const DecodeParams p) {
  const int hq = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const int n = p.len[b];
  const int nsplit = min(p.max_splits, (n + p.split_tokens - 1) / p.split_tokens);
  const int64_t ph = ((int64_t)b * p.y.H_q + hq) * p.max_splits;
  float M = -INFINITY;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, p.part_ml[(ph + s) * 2]);
  float a = 0.f, l = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = p.part_ml[(ph + s) * 2];
    const float sc = (ms == -INFINITY) ? 0.f : ex2(ms - M);
    a += p.part_acc[(ph + s) * D + c] * sc;
    l += p.part_ml[(ph + s) * 2 + 1] * sc;
  }
  const float o = (l > 0.f) ? a / l : 0.f;
  reinterpret_cast<__nv_bfloat16*>(p.out)[((int64_t)b * p.y.H_q + hq) * D + c] = __float2bfloat16_rn(o);
}

template <int D, int R>
int launch_decode_t(const DecodeParams& p, int grid_splits, cudaStream_t s) {
  using C = Cfg<D, R>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D, R>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return (int)e;
    configured = true;
  }
  dim3 grid(grid_splits, p.y.H_kv, p.y.B);
  pod_decode_splitk_kernel<D, R><<<grid, NW * 32, C::SMEM, s>>>(p);
  return (int)cudaGetLastError();
}

template <int D, int R>
int resident_t() {
  using C = Cfg<D, R>;
  cudaError_t e = cudaFuncSetAttribute(pod_decode_splitk_kernel<D, R>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
  if (e != cudaSuccess) return 0;
  int nb = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, pod_decode_splitk_kernel<D, R>, NW * 32, C::SMEM);
  return e == cudaSuccess ? nb : 0;
}

}  // namespace

int launch_decode(const DecodeParams& p, int grid_splits, cudaStream_t s) {
  const int D = p.y.D, r = p.y.H_q / p.y.H_kv;
  if (D == 128) return r <= 4 ? launch_decode_t<128, 4>(p, grid_splits, s) : launch_decode_t<128, 8>(p, grid_splits, s);
  if (D == 64) return r <= 4 ? launch_decode_t<64, 4>(p, grid_splits, s) : launch_decode_t<64, 8>(p, grid_splits, s);
  return (int)cudaErrorInvalidValue;
}

int launch_combine(const DecodeParams& p, cudaStream_t s) {
  dim3 grid(p.y.H_q, p.y.B);
  if (p.y.D == 128) pod_combine_kernel<128><<<grid, 128, 0, s>>>(p);
  else pod_combine_kernel<64><<<grid, 64, 0, s>>>(p);
  return (int)cudaGetLastError();
}

int decode_resident_ctas_per_sm(int D, int r) {
  if (D == 128) return r <= 4 ? resident_t<128, 4>() : resident_t<128, 8>();
  if (D == 64) return r <= 4 ? resident_t<64, 4>() : resident_t<64, 8>();
  return 0;
}

}  // namespace pod
