// pod_prefill_attn: PoD attention for every position of a sequence (Section 2.2, Eq. 1 and the
// masks of Fig. 2, middle) on the 5th-generation tensor cores: tcgen05.mma with operands staged
// in shared memory by TMA and accumulators in tensor memory.
//
// Position i attends to positions j <= i.  Of those the first n_s and the last n_r are proximal:
// their logits are q_l[i] . k_l[j]; the others are distant: their logits are q_a[i] . k_a[j] with a
// the lowest layer of the head's block (for a head whose block starts at this layer both are the
// same product).  One softmax over both groups weighs layer l's own values.  head_dim is 128 or 64 (a template
// parameter; sizes in these comments are for 128).
//
// One CTA = 256 consecutive query positions of one query head: two softmax groups of four warps (group g
// owns rows 128 g .. 128 g + 127, one thread per row), one warp whose lane 0 issues every tcgen05.mma and
// one warp whose lane 0 issues every TMA load.  Keys and values arrive in tiles of 128 positions through a
// ring of five 32 KiB shared-memory slots (K_0, V_0, K_1, V_1, ...; TMA, 128-byte swizzle); both groups
// use the same tile, so each is fetched once per 256 rows.
// A tile whose keys are all distant for every row of the CTA is scored with Q_a K_a^T, one whose keys are
// all proximal (or whose head does not share) with Q K^T; the few tiles that straddle the edge of the
// window or of the sink are taken twice, once with each product and the other kind of key masked (the
// softmax does not care in how many pieces, or in which order, the keys arrive).  The passes that use the
// lowest layer's product run first, with Q_a in the query buffers; then Q of this layer is loaded over it
// and the other passes follow.  Per pass v and group g, in tensor memory (per group 128 columns for S and
// P, 128 for O):
//   S[128 x 128] = Q K^T  or  Q_a K_a^T      (M = 128, N = 128, K = 16 x 8 steps)
//   each softmax thread reads its row of S in four pieces (tcgen05.ld), takes P = 2^(logit - m) against the
//   row's current reference m, and writes it as packed bf16 over the columns of S it has consumed (tcgen05.st);
//   a first pass, a masked tile or a raise of m reads the row twice (maximum first)
//   O[128 x 128] += P V                       (A = P from tensor memory, B = V MN-major, K = 16 x 8).
// The tensor-core thread alternates between the groups (P V of group g, then its next Q K^T), so one group's
// products run while the other group is in its softmax.  The reference maximum m of a row is only raised
// when the tile's maximum exceeds it by more than 8 (in log2 units): P then stays below 2^8, and the rows of
// O have to be rescaled (tcgen05.ld / st) only on those rare occasions instead of after every tile; row sum
// and O share the same m, so the quotient is exact either way.  Warps hand buffers to one another through
// mbarriers; every wait is bounded (a wait gives up only after seconds, long after every copy in flight has
// landed), a wait that gives up raises the error flag, and the tensor memory is always returned before the
// CTA exits.
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

#include "../../include/pod.h"
#include "pod_common.h"

namespace pod {
namespace {

constexpr int BM = 128;                 // query rows per softmax group
constexpr int NG = 2;                   // softmax groups per CTA
constexpr int BLK = NG * BM;            // query rows per CTA
constexpr int BN = 128;                 // keys per tile
constexpr int NRING = 5;                // slots of the K/V ring
constexpr uint32_t PF_WAIT_LIMIT = 1u << 22;

constexpr int Q_SUB = BM * 128, KV_SUB = BN * 128;   // one [rows][128 B] sub-tile: 64 channels of every row
// shared-memory plan for head_dim PD (64 or 128): one or two sub-tiles per operand tile
template <int PD> struct Plan {
  static constexpr int Q_B = BM * PD * 2;        // 32 KiB at d = 128
  static constexpr int KV_B = BN * PD * 2;       // 32 KiB at d = 128
  static constexpr int OFF_Q = 0;                // per group: Q of the lowest layer, later Q of this layer
  static constexpr int OFF_RING = NG * Q_B;
  static constexpr int OFF_BAR = OFF_RING + NRING * KV_B;
  static constexpr int SMEM = OFF_BAR + 256 + 1024;
};
constexpr int PF_THREADS = BLK + 64;    // eight softmax warps, the tensor-core warp, the load warp
constexpr int TM_COLS = 512;            // per group S / P 128 + O 128 fp32 columns
constexpr int TM_GROUP = 256, TM_O = 128;
constexpr float RESCALE_STEP = 8.f;     // raise a row's reference maximum only past this many log2 units

struct PrefillParams {
  int32_t T, H_q, H_kv, S, W;
  float scale_log2;
  uint32_t share_mask[8];               // bit h: KV head h takes distant logits from the lowest layer's q, k
  uint16_t* out;                        // [T][H_q][head_dim] bf16
  int32_t* err_flag;
};

__device__ __forceinline__ uint32_t s2u(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < PF_WAIT_LIMIT; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
// [rows][64 bf16] box of a [T][H][128] tensor at (channel x, head, row t); x is 0 or 64
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int head, int t, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(head), "r"(t), "r"(bar) : "memory");
}
// Shared-memory matrix descriptor of the tensor cores (128-byte swizzle, descriptor version of
// sm_100): start address, leading and stride byte offsets in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M = 128; B K-major or MN-major
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same with A read from tensor memory (128 lanes x 8 columns of packed bf16 pairs per step)
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// this thread's 32 consecutive fp32 columns of its TMEM lane (valid after tmem_ld_wait)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// the values of earlier tmem_ld32 calls may be used after this
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// 16 consecutive 32-bit columns of this thread's TMEM lane (complete after tmem_st_wait)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void bar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The passes of a CTA in the order they run.  Tiles [low_a, low_b) hold a key that is distant for some row of
// the CTA: they get a pass with the lowest layer's product (these n_low passes come first).  Of those, tiles
// [dis_a, dis_b) are distant for every row and get no other pass; every other tile gets a pass with the
// layer's own product.  mixed: the tile has keys of both kinds, the pass keeps the kind its product is for.
struct PassMap { int n_low, low_a, low_b, dis_a, dis_b; };
struct Pass { int j; bool low, mixed; };
__device__ __forceinline__ Pass pass_of(const PassMap m, int v) {
  Pass c;
  if (v < m.n_low) {
    c.j = m.low_a + v;
    c.low = true;
    c.mixed = !(c.j >= m.dis_a && c.j < m.dis_b);
  } else {
    const int u = v - m.n_low;
    c.j = u < m.dis_a ? u : u + (m.dis_b - m.dis_a);
    c.low = false;
    c.mixed = c.j >= m.low_a && c.j < m.low_b;
  }
  return c;
}
// bit i set for i < n
__device__ __forceinline__ uint32_t low_bits(int n) { return n <= 0 ? 0u : (n >= 32 ? 0xffffffffu : (1u << n) - 1u); }
// Bit i: the pass keeps key c0 + i for row qi.  Causal and inside the sequence; in a tile with both kinds of
// key the own product keeps the proximal keys, the lowest layer's the distant ones (S <= key <= qi - W).
__device__ __forceinline__ uint32_t keep_bits(int c0, int qi, int T, int S, int W, bool mixed, bool low) {
  uint32_t keep = low_bits(min(qi, T - 1) - c0 + 1);
  if (mixed) {
    const uint32_t dist = low_bits(qi - W - c0 + 1) & ~low_bits(S - c0);
    keep &= low ? dist : ~dist;
  }
  return keep;
}
// logits of keys the pass does not keep become -inf
__device__ __forceinline__ void apply_bits(float (&t)[32], uint32_t bits) {
#pragma unroll
  for (int i = 0; i < 32; ++i) t[i] = ((bits >> i) & 1u) ? t[i] : -INFINITY;
}

template <int PD>
__global__ void __launch_bounds__(PF_THREADS, 1)
pod_prefill_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmQl,
                   const __grid_constant__ CUtensorMap tmKl, const PrefillParams p) {
  constexpr int Q_B = Plan<PD>::Q_B, KV_B = Plan<PD>::KV_B, OFF_Q = Plan<PD>::OFF_Q, OFF_RING = Plan<PD>::OFF_RING,
                OFF_BAR = Plan<PD>::OFF_BAR;
  extern __shared__ unsigned char pf_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(pf_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = s2u(smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  const bool producer = warp == BLK / 32, loader = warp == BLK / 32 + 1;   // tensor-core warp, load warp
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x;          // long rows first
  const int hq = blockIdx.y, kvh = hq / (p.H_q / p.H_kv);
  const int q0 = qb * BLK;
  uint32_t share_word = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) share_word = (kvh >> 5) == i ? p.share_mask[i] : share_word;
  const bool shares = (share_word >> (kvh & 31)) & 1u;
  // mbarriers: Q landed; per ring slot: tile landed, slot free; per group: S ready, P written, O complete;
  // the lowest layer's Q no longer needed
  const uint32_t bar_q = sb + OFF_BAR, bar_full = bar_q + 8, bar_free = bar_q + 48, bar_sfull = bar_q + 88,
                 bar_pfull = bar_q + 104, bar_odone = bar_q + 120, bar_qfree = bar_q + 136;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 192);

  // A launch whose waits give up would otherwise spend seconds in every one of its thousands of CTAs: once the
  // error word is set (by this launch or an earlier one, until pod_prefill_status reads it), CTAs return at once.
  __shared__ int s_abort;
  if (tid == 0) s_abort = *reinterpret_cast<volatile int32_t*>(p.err_flag);
  __syncthreads();
  if (s_abort != 0) return;
  if (tid == 0) {
    bar_init(bar_q, 1);
    bar_init(bar_qfree, 1);
    for (int i = 0; i < NRING; ++i) {
      bar_init(bar_full + i * 8, 1);
      bar_init(bar_free + i * 8, 1);
    }
    for (int g = 0; g < NG; ++g) {
      bar_init(bar_sfull + g * 8, 1);
      bar_init(bar_pfull + g * 8, BM / 32);                     // one arrival per softmax warp
      bar_init(bar_odone + g * 8, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (producer) {                                               // all of the SM's tensor memory: S / P and O of both groups
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s2u(tmem_slot)), "r"(TM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = *tmem_slot;

  // keys this CTA needs: positions [0, min(T, q0 + 256)); tile j covers [128 j, 128 j + 128)
  const int k_end = min(p.T, q0 + BLK);
  const int n_tiles = (k_end + BN - 1) / BN;
  PassMap pm{0, 0, 0, 0, 0};
  if (shares) {
    pm.low_a = p.S / BN;                                        // tiles before it lie inside the sink
    const int e = q0 + BLK - 1 - p.W;                           // the last row's newest distant position
    pm.low_b = max(pm.low_a, min(e < 0 ? 0 : e / BN + 1, n_tiles));
    pm.dis_a = (p.S + BN - 1) / BN;
    const int f = q0 - p.W - (BN - 1);                          // tile j is distant for the first row too if 128 j <= f
    pm.dis_b = max(pm.dis_a, min(f < 0 ? 0 : f / BN + 1, pm.low_b));
    pm.n_low = pm.low_b - pm.low_a;
  }
  const int n_low = pm.n_low;
  const int n_pass = n_low + n_tiles - (pm.dis_b - pm.dis_a);
  bool fail = false;

  if (loader) {
    // ---- load warp: one thread requests Q, then keeps the ring full: load 2 v is K of pass v, 2 v + 1 its V ----
    if ((tid & 31) == 0) {
      auto load_q = [&](bool low) {
        bar_expect_tx(bar_q, NG * Q_B);
#pragma unroll
        for (int g = 0; g < NG; ++g)
#pragma unroll
          for (int h = 0; h < PD / 64; ++h)
            tma_load_3d(sb + OFF_Q + g * Q_B + h * Q_SUB, low ? &tmQl : &tmQ, h * 64, hq, q0 + g * BM, bar_q);
      };
      load_q(n_low > 0);
      const int n_loads = 2 * n_pass;
      const int i_switch = n_low > 0 ? 2 * (n_low - 1) : -1;    // the last load whose product reads the lowest layer's Q
      bool switched = n_low == 0;
      for (int i = 0; i < n_loads && !fail; ++i) {
        const int slot = i % NRING;
        if (i >= NRING) {
          if (i - NRING == i_switch) {                          // both groups' last products with Q_a are done
            fail = !bar_wait(bar_qfree, 0);
            if (fail) break;
            load_q(false);
            switched = true;
          }
          fail = !bar_wait(bar_free + slot * 8, ((i / NRING) - 1) & 1);   // the slot's previous tile (load i - 5) has been used
          if (fail) break;
        }
        const Pass c = pass_of(pm, i >> 1);
        const CUtensorMap* map = (i & 1) ? &tmV : (c.low ? &tmKl : &tmK);
        const uint32_t dst = sb + OFF_RING + slot * KV_B, bar = bar_full + slot * 8;
        bar_expect_tx(bar, KV_B);
#pragma unroll
        for (int h = 0; h < PD / 64; ++h) tma_load_3d(dst + h * KV_SUB, map, h * 64, kvh, c.j * BN, bar);
      }
      if (!fail && !switched) {                                 // the ring never came back to that slot
        fail = !bar_wait(bar_qfree, 0);
        if (!fail) load_q(false);
      }
      if (fail) atomicExch(p.err_flag, 1);
    }
  } else if (producer) {
    // ---- tensor-core warp: one thread issues every product -------------------------------------------------
    if ((tid & 31) == 0) {
      constexpr uint32_t IDESC = instr_desc(128, false), IDESC_O = instr_desc(PD, true);
      // Descriptors of the operands' first steps, built once: a later step or slot only adds its byte offset
      // / 16 to the address field (shared-memory addresses stay below 2^18, so the field never carries).
      const uint64_t dq0 = smem_desc(sb + OFF_Q, 16, 1024), dk0 = smem_desc(sb + OFF_RING, 16, 1024);
      const uint64_t dv0 = smem_desc(sb + OFF_RING, KV_SUB, 1024);
      auto issue_qk = [&](int g, int v) {                       // S[g] = Q_g K^T of pass v
        const uint64_t dk = dk0 + (uint64_t)(((2 * v) % NRING) * (KV_B >> 4));
        const uint64_t dq = dq0 + (uint64_t)(g * (Q_B >> 4));
#pragma unroll
        for (int ks = 0; ks < PD / 16; ++ks) {                  // 16 channels per step: 4 per 128-byte sub-tile
          const uint32_t a_off = (ks >> 2) * Q_SUB + (ks & 3) * 32, b_off = (ks >> 2) * KV_SUB + (ks & 3) * 32;
          umma(tm + g * TM_GROUP, dq + (uint64_t)(a_off >> 4), dk + (uint64_t)(b_off >> 4), IDESC, ks > 0);
        }
        umma_commit(bar_sfull + g * 8);
        // A tcgen05.commit in the middle of a run of products costs the pipe a few hundred cycles, one that
        // follows another commit less: V of the pass before is handed back here, next to the commit above
        // (both groups are done with it), and K without a commit at all (see the wait for P below).
        if (g == NG - 1) {
          if (v > 0) umma_commit(bar_free + ((2 * v - 1) % NRING) * 8);
          if (v + 1 == n_low) umma_commit(bar_qfree);           // the last products that read the lowest layer's Q
        }
      };
      auto wait_k = [&](int v) -> bool {                        // K of pass v (and the Q it goes with) has landed
        if (v == 0 && !bar_wait(bar_q, 0)) return false;
        if (v == n_low && n_low > 0 && !bar_wait(bar_q, 1)) return false;
        return bar_wait(bar_full + ((2 * v) % NRING) * 8, ((2 * v) / NRING) & 1);
      };
      fail = !wait_k(0);
      if (!fail) {
        tc_fence_after();
        for (int g = 0; g < NG; ++g) issue_qk(g, 0);
      }
      for (int v = 0; v < n_pass && !fail; ++v) {
        const int iv = 2 * v + 1;                               // the load that brought V of pass v
        fail = !bar_wait(bar_full + (iv % NRING) * 8, (iv / NRING) & 1);
        if (!fail && v + 1 < n_pass) fail = !wait_k(v + 1);
        const uint64_t dv = dv0 + (uint64_t)((iv % NRING) * (KV_B >> 4));
#pragma unroll
        for (int g = 0; g < NG && !fail; ++g) {
          fail = !bar_wait(bar_pfull + g * 8, v & 1);           // P[g] of pass v is written
          if (fail) break;
          // ... so S[g] of pass v was complete: once that is true of the last group, every product that read
          // K of pass v is done and its slot goes back with a plain arrival (its next tile is not due soon)
          if (g == NG - 1) bar_arrive(bar_free + ((2 * v) % NRING) * 8);
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < BN / 16; ++ks)                  // 16 keys per step; O accumulates over the passes
            umma_ts(tm + g * TM_GROUP + TM_O, tm + g * TM_GROUP + ks * 8, dv + (uint64_t)(ks * (2048 >> 4)), IDESC_O,
                    (v > 0 || ks > 0) ? 1u : 0u);
          if (v + 1 < n_pass) issue_qk(g, v + 1);               // overwrites P[g]: in order behind the P V just issued
          else umma_commit(bar_odone + g * 8);
        }
      }
      if (fail) atomicExch(p.err_flag, 1);
    }
  } else {
    // ---- softmax warps: thread r of group g owns query row 128 g + r ----------------------------------
    const int g = warp >> 2, r = tid & (BM - 1);
    const int qg0 = q0 + g * BM, qi = qg0 + r;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;   // this warp's quarter of the TMEM lanes
    const uint32_t tmg = tm + g * TM_GROUP + lane_base;
    float m_used = -INFINITY, l_row = 0.f;
    for (int v = 0; v < n_pass; ++v) {
      const Pass c = pass_of(pm, v);
      fail = !bar_wait(bar_sfull + g * 8, v & 1);               // S of pass v is complete, and so is every earlier P V
      if (__any_sync(0xffffffffu, fail)) { fail = true; break; }
      tc_fence_after();
      const int k0 = c.j * BN;
      // Interior tiles (every key visible to every row of the group) need no per-key decision; tiles on the
      // diagonal get the causal mask, and a pass over a tile with both kinds of key keeps the kind its
      // product is meant for.
      const bool masked = c.mixed || (k0 + BN - 1 > qg0);
      // Common case (no mask): ONE reading of the row.  The exponentials are taken against
      // the reference maximum the row already has while the tile's own maximum is found on the side; P stays
      // in registers until it is known that no row of the warp has to raise its reference, which is nearly
      // always so (a raise needs a logit 8 log2 units above everything seen before).  S is still intact then,
      // so the rare other case simply falls through to the general path below.
      bool done = false;
      if (!masked) {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        float ps4[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pk[BN / 32][16];
        float ta[32], tb[32];
        float m_use = 0.f;
        auto piece = [&](const float (&t)[32], uint32_t (&o)[16]) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            mx4[i & 3] = fmaxf(mx4[i & 3], fmaxf(t[2 * i], t[2 * i + 1]));
            const float p0 = ex2f(fmaf(t[2 * i], p.scale_log2, -m_use));
            const float p1 = ex2f(fmaf(t[2 * i + 1], p.scale_log2, -m_use));
            ps4[i & 3] += p0 + p1;
            __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
            o[i] = *reinterpret_cast<uint32_t*>(&b2);
          }
        };
        tmem_ld32(tmg, ta);                                     // the next piece is on its way while one is worked on
        tmem_ld_wait();
        tmem_ld32(tmg + 32, tb);
        if (m_used == -INFINITY) {                              // a row's first keys: any reference near their maximum will do
          float m0 = ta[0];
#pragma unroll
          for (int i = 1; i < 32; ++i) m0 = fmaxf(m0, ta[i]);
          m_used = m0 * p.scale_log2;                           // finite: nothing is masked in this tile; O and the sum are still 0
        }
        m_use = m_used;
        piece(ta, pk[0]);
        tmem_ld_wait();
        tmem_ld32(tmg + 64, ta);
        piece(tb, pk[1]);
        tmem_ld_wait();
        tmem_ld32(tmg + 96, tb);
        piece(ta, pk[2]);
        tmem_ld_wait();
        piece(tb, pk[3]);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
        const bool raise = mx > m_used + RESCALE_STEP || (m_used == -INFINITY && mx > -INFINITY);
        if (!__any_sync(0xffffffffu, raise)) {
#pragma unroll
          for (int ch = 0; ch < BN / 32; ++ch) tmem_st16(tmg + ch * 16, pk[ch]);
          l_row += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
          done = true;
        }
      }
      if (!done) {
        // General path, two readings of the row: its maximum first.  In a masked tile most pieces of 32 keys
        // are still all kept or all masked for the 32 rows of a warp (the boundaries move with the row); only
        // the others are decided key by key, from the row's keep bits.  These passes are few, so their loops
        // stay rolled up and the kernel's code stays short.
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
        for (int ch = 0; ch < BN / 32; ++ch) {
          const uint32_t kb = masked ? keep_bits(k0 + ch * 32, qi, p.T, p.S, p.W, c.mixed, c.low) : 0xffffffffu;
          if (__all_sync(0xffffffffu, kb == 0u)) continue;
          float t[32];
          tmem_ld32(tmg + ch * 32, t);
          tmem_ld_wait();
          if (!__all_sync(0xffffffffu, kb == 0xffffffffu)) apply_bits(t, kb);
#pragma unroll
          for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], t[i]);
        }
        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        mx *= p.scale_log2;                                     // the scale is positive: it commutes with the maximum
        // raise the row's reference maximum only when the tile exceeds it by more than RESCALE_STEP
        const bool raise = mx > m_used + RESCALE_STEP || (m_used == -INFINITY && mx > -INFINITY);
        float alpha = 1.f;
        if (raise) { alpha = ex2f(m_used - mx); m_used = mx; }  // ex2(-inf) = 0 on the first tile
        if (__any_sync(0xffffffffu, raise) && v > 0) {          // rescale this warp's rows of O (nothing accumulates now)
#pragma unroll 1
          for (int ch = 0; ch < PD / 32; ++ch) {
            float t[32];
            tmem_ld32(tmg + TM_O + ch * 32, t);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) t[i] *= alpha;
            tmem_st32(tmg + TM_O + ch * 32, t);
          }
        }
        l_row *= alpha;
        const float m_use = (m_used == -INFINITY) ? 0.f : m_used;
        // second reading, 32 keys at a time: P as packed bf16 pairs over columns already consumed
        // (keys 32 c .. 32 c + 31 of S sit in columns 32 c .., their P in columns 16 c .. 16 c + 15)
        float ps4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int ch = 0; ch < BN / 32; ++ch) {
          const uint32_t kb = masked ? keep_bits(k0 + ch * 32, qi, p.T, p.S, p.W, c.mixed, c.low) : 0xffffffffu;
          float t[32];
          uint32_t pk[16];
          if (__all_sync(0xffffffffu, kb == 0u)) {               // nothing kept: P = 0
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
          } else {
            tmem_ld32(tmg + ch * 32, t);
            tmem_ld_wait();
            if (!__all_sync(0xffffffffu, kb == 0xffffffffu)) apply_bits(t, kb);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float p0 = ex2f(fmaf(t[2 * i], p.scale_log2, -m_use));
              const float p1 = ex2f(fmaf(t[2 * i + 1], p.scale_log2, -m_use));
              ps4[i & 3] += p0 + p1;
              __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
              pk[i] = *reinterpret_cast<uint32_t*>(&b2);
            }
          }
          tmem_st16(tmg + ch * 16, pk);
        }
        l_row += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if ((tid & 31) == 0) bar_arrive(bar_pfull + g * 8);
    }
    if (!fail) {
      fail = !bar_wait(bar_odone + g * 8, 0);
      fail = __any_sync(0xffffffffu, fail);
    }
    if (fail) {
      if ((tid & 31) == 0) atomicExch(p.err_flag, 1);
    } else {
      tc_fence_after();
      const float inv = l_row > 0.f ? 1.f / l_row : 0.f;
      uint16_t* dst = p.out + ((int64_t)qi * p.H_q + hq) * PD;
#pragma unroll 1
      for (int ch = 0; ch < PD / 32; ++ch) {
        float t[32];
        tmem_ld32(tmg + TM_O + ch * 32, t);                     // warp-collective: rows past T load too
        tmem_ld_wait();
        if (qi < p.T) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              __nv_bfloat162 b2 = __floats2bfloat162_rn(t[c + 2 * i] * inv, t[c + 2 * i + 1] * inv);
              w[i] = *reinterpret_cast<uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(dst + ch * 32 + c) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }
  // return the tensor memory
  tc_fence_before();
  __syncthreads();
  if (producer) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(TM_COLS) : "memory");
  }
}

// Error word of the bounded waits: one per device that loads the library, inside the device image, so that
// nothing is allocated and nothing has to be freed.  In host code the name is only a handle for
// cudaGetSymbolAddress.
static __device__ int32_t g_prefill_err_word;

struct PrefillSetup {
  bool ready = false;
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  int32_t* err = nullptr;       // device address of g_prefill_err_word on that device
};
PrefillSetup g_pf[64];
std::mutex g_pf_mutex;

bool encode_3d(PFN_cuTensorMapEncodeTiled_v12000 enc, CUtensorMap* tm, const void* base, int T, int H, int rows, int PD) {
  cuuint64_t dims[3] = {(cuuint64_t)PD, (cuuint64_t)H, (cuuint64_t)T};
  cuuint64_t strides[2] = {(cuuint64_t)PD * 2, (cuuint64_t)H * PD * 2};
  cuuint32_t box[3] = {64u, 1u, (cuuint32_t)rows};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace pod

using namespace pod;

extern "C" int pod_prefill_attn(int n_tokens, int n_q_heads, int n_kv_heads, int head_dim, int n_sink, int n_recent,
                                float sm_scale, const void* q, const void* k, const void* v, const void* q_low,
                                const void* k_low, const int32_t* head_shares, void* out, void* cuda_stream) {
  if (!q || !k || !v || !out) return POD_ERR_INVALID;
  if ((head_dim != 64 && head_dim != 128) || n_tokens < 1 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads != 0) return POD_ERR_INVALID;
  if (n_sink < 0 || n_recent < 1 || !(sm_scale >= 0.f) || isinf(sm_scale)) return POD_ERR_INVALID;
  if (n_q_heads > 65535) return POD_ERR_INVALID;
  if ((q_low == nullptr) != (k_low == nullptr)) return POD_ERR_INVALID;
  if (q_low != nullptr && n_kv_heads > 256) return POD_ERR_INVALID;     // the sharing mask holds 256 KV heads
  for (const void* ptr : {q, k, v, q_low, k_low, (const void*)out})
    if (((uintptr_t)ptr % 16) != 0) return POD_ERR_INVALID;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return POD_ERR_CUDA;
  PrefillSetup* su = &g_pf[dev];
  {
    std::lock_guard<std::mutex> lock(g_pf_mutex);
    if (!su->ready) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || fn == nullptr)
        return POD_ERR_CUDA;
      void* errp = nullptr;
      if (cudaGetSymbolAddress(&errp, g_prefill_err_word) != cudaSuccess || errp == nullptr) return POD_ERR_CUDA;
      su->err = static_cast<int32_t*>(errp);
      if (cudaMemset(su->err, 0, 4) != cudaSuccess) return POD_ERR_CUDA;
      if (cudaFuncSetAttribute(pod_prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan<128>::SMEM) != cudaSuccess ||
          cudaFuncSetAttribute(pod_prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan<64>::SMEM) != cudaSuccess)
        return POD_ERR_CUDA;
      su->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
      su->ready = true;
    }
  }
  PrefillParams p{};
  p.T = n_tokens; p.H_q = n_q_heads; p.H_kv = n_kv_heads; p.S = n_sink; p.W = n_recent;
  p.scale_log2 = (sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)head_dim)) * 1.4426950408889634f;
  p.out = static_cast<uint16_t*>(out);
  p.err_flag = su->err;
  if (q_low != nullptr)
    for (int h = 0; h < n_kv_heads; ++h)
      if (head_shares == nullptr || head_shares[h] != 0) p.share_mask[h >> 5] |= 1u << (h & 31);
  CUtensorMap tq, tk, tv, tql, tkl;
  const void* ql = q_low ? q_low : q;
  const void* kl = k_low ? k_low : k;
  if (!encode_3d(su->encode, &tq, q, n_tokens, n_q_heads, BM, head_dim) || !encode_3d(su->encode, &tk, k, n_tokens, n_kv_heads, BN, head_dim) ||
      !encode_3d(su->encode, &tv, v, n_tokens, n_kv_heads, BN, head_dim) || !encode_3d(su->encode, &tql, ql, n_tokens, n_q_heads, BM, head_dim) ||
      !encode_3d(su->encode, &tkl, kl, n_tokens, n_kv_heads, BN, head_dim))
    return POD_ERR_INVALID;
  dim3 grid((n_tokens + BLK - 1) / BLK, n_q_heads);
  if (head_dim == 128)
    pod_prefill_kernel<128><<<grid, PF_THREADS, Plan<128>::SMEM, static_cast<cudaStream_t>(cuda_stream)>>>(tq, tk, tv, tql, tkl, p);
  else
    pod_prefill_kernel<64><<<grid, PF_THREADS, Plan<64>::SMEM, static_cast<cudaStream_t>(cuda_stream)>>>(tq, tk, tv, tql, tkl, p);
  return cudaGetLastError() == cudaSuccess ? POD_OK : POD_ERR_CUDA;
}

// POD_ERR_DEVICE if a launch of pod_prefill_attn on the current device gave up a bounded wait since the last call.
extern "C" int pod_prefill_status(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return POD_ERR_CUDA;
  PrefillSetup* su = &g_pf[dev];
  if (!su->ready) return POD_OK;
  int32_t flag = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return POD_ERR_CUDA;
  if (cudaMemcpy(&flag, su->err, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return POD_ERR_CUDA;
  if (flag != 0 && cudaMemset(su->err, 0, 4) != cudaSuccess) return POD_ERR_CUDA;
  return flag ? POD_ERR_DEVICE : POD_OK;
}

// Sets the error word of the current device as a kernel whose wait gave up would (fault injection from the host, for
// tests of the error path): the next launches return without computing until pod_prefill_status has been called.
extern "C" int pod_prefill_inject_error(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return POD_ERR_CUDA;
  PrefillSetup* su = &g_pf[dev];
  if (!su->ready) return POD_ERR_INVALID;                    // no pod_prefill_attn on this device yet
  if (cudaDeviceSynchronize() != cudaSuccess) return POD_ERR_CUDA;
  const int32_t one = 1;
  return cudaMemcpy(su->err, &one, 4, cudaMemcpyHostToDevice) == cudaSuccess ? POD_OK : POD_ERR_CUDA;
}
