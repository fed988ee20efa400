// pod_dense_decode_attn_static: decode attention over a caller-owned dense K/V buffer with the
// split-K scratch held in a fixed device array of this library instead of allocated memory.
//
// The entry point runs the same split-K kernel and in-kernel combine as pod_decode_attn.  A
// dense K/V buffer laid out [2 (K, V)][H_kv][capacity][d] is exactly the PoD arena of a
// one-layer cache with no sink and a recent window of `capacity` rows, so the kernel reads it
// through the same tile coordinates; only the scratch pointers differ.
#include <cudaTypedefs.h>
#include <math.h>

#include <mutex>

#include "../../include/pod.h"
#include "pod_common.h"

using namespace pod;

namespace {

constexpr int STATIC_MAX_Q_HEADS = 64;
constexpr int STATIC_MAX_SPLITS = 64;
constexpr int STATIC_MAX_DEVICES = 64;
constexpr size_t OFF_PACC = 0;                                                         // fp32 [64][64][128]
constexpr size_t OFF_PML = (size_t)STATIC_MAX_Q_HEADS * STATIC_MAX_SPLITS * 128 * 4;   // fp32 [64][64][4]
constexpr size_t SCHED_BYTES = (size_t)STATIC_MAX_Q_HEADS * SCHED_STRIDE * 4;          // int32 [64 KV heads][32]
constexpr size_t OFF_SCHED = OFF_PML + (size_t)STATIC_MAX_Q_HEADS * STATIC_MAX_SPLITS * 4 * 4;
constexpr size_t OFF_ERR = OFF_SCHED + SCHED_BYTES;
constexpr size_t STATIC_BYTES = OFF_ERR + 256;
static_assert(STATIC_BYTES == POD_STATIC_SCRATCH_BYTES, "header and library disagree on the scratch size");

// The scratch itself.  Every device that loads this library holds one copy until the process
// exits.  In host code this name is only a handle for cudaGetSymbolAddress, never a pointer.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_static_scratch on that device
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  int sm_count = 0, resident128 = 0, resident64 = 0;   // resident CTAs per SM of the kernel for head size 128 / 64
};
DeviceSetup g_setup[STATIC_MAX_DEVICES];
std::mutex g_setup_mutex;

// First call on a device: resolve the array's device address and the tensor-map encoder.
int setup_device(int dev, DeviceSetup** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[dev];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return POD_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr)
      return POD_ERR_CUDA;
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return POD_ERR_CUDA;
    // The kernel's shared-memory attribute is a per-device setting: both head sizes are configured here,
    // on this device, and the occupancy the driver reports sizes the grid.
    const int r128 = decode_resident_ctas_per_sm(128), r64 = decode_resident_ctas_per_sm(64);
    if (r128 < 1 || r64 < 1) return POD_ERR_CUDA;
    // the error word starts at zero; afterwards only pod_dense_decode_attn_static_status clears it
    if (cudaMemset(static_cast<unsigned char*>(ptr) + OFF_ERR, 0, 256) != cudaSuccess) return POD_ERR_CUDA;
    s.scratch = static_cast<unsigned char*>(ptr);
    s.encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    s.sm_count = sm;
    s.resident128 = r128; s.resident64 = r64;
    s.ready = true;
  }
  *out = &s;
  return POD_OK;
}

}  // namespace

extern "C" int pod_dense_decode_attn_static(const void* kv_device, int capacity, int n_tokens,
                                            const void* q_device, void* out_device, int n_q_heads,
                                            int n_kv_heads, int head_dim, float sm_scale,
                                            void* cuda_stream) {
  if (!kv_device || !q_device || !out_device) return POD_ERR_INVALID;
  if (((uintptr_t)kv_device % 16) != 0 || ((uintptr_t)q_device % 16) != 0 || ((uintptr_t)out_device % 16) != 0)
    return POD_ERR_INVALID;
  if (head_dim != 64 && head_dim != 128) return POD_ERR_INVALID;
  if (n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads != 0 || n_q_heads / n_kv_heads > 8) return POD_ERR_INVALID;
  if (capacity < 1 || n_tokens < 0 || !(sm_scale >= 0.f) || isinf(sm_scale)) return POD_ERR_INVALID;
  // limits of the fixed scratch: at most 64 query heads (64 splits each), and n_tokens <= capacity
  if (n_q_heads > STATIC_MAX_Q_HEADS || n_tokens > capacity) return POD_ERR_CAPACITY;
  const int64_t total_rows = (int64_t)2 * n_kv_heads * capacity;
  if (total_rows >= ((int64_t)1 << 31)) return POD_ERR_CAPACITY;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return POD_ERR_CUDA;
  DeviceSetup* su = nullptr;
  const int st = setup_device(dev, &su);
  if (st != POD_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t out_bytes = (size_t)n_q_heads * head_dim * 2;
  if (n_tokens == 0) return cudaMemsetAsync(out_device, 0, out_bytes, stream) == cudaSuccess ? POD_OK : POD_ERR_CUDA;

  CUtensorMap tmap;
  cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)total_rows};
  cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)decode_tile_tokens()};
  cuuint32_t estr[2] = {1u, 1u};
  if (su->encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(kv_device), dims, strides, box,
                 estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return POD_ERR_INVALID;

  // one CTA per (split, KV head): about one wave of resident CTAs, at most 64 splits
  int k = (su->sm_count * (head_dim == 128 ? su->resident128 : su->resident64)) / n_kv_heads;
  if (k < 1) k = 1;
  if (k > STATIC_MAX_SPLITS) k = STATIC_MAX_SPLITS;
  int split_tokens = (n_tokens + k - 1) / k;
  if (split_tokens < 64) split_tokens = 64;
  const int grid_splits = (n_tokens + split_tokens - 1) / split_tokens;

  DecodeParams p{};
  p.y.L = 1; p.y.H_kv = n_kv_heads; p.y.H_q = n_q_heads; p.y.D = head_dim;
  p.y.S = 0; p.y.W = capacity; p.y.B = 1; p.y.n_slots = n_kv_heads; p.y.shared = 0;
  p.y.low = nullptr; p.y.slot = nullptr;               // one layer: every layer is its own block
  p.y.seq_row_base = nullptr; p.y.seq_cap_d = nullptr;        // not read: scalars go by value
  p.arena = static_cast<const uint16_t*>(kv_device);
  p.len = nullptr;
  p.q = static_cast<const uint16_t*>(q_device);
  p.stash = nullptr;
  p.part_acc = reinterpret_cast<float*>(su->scratch + OFF_PACC);
  p.part_ml = reinterpret_cast<float*>(su->scratch + OFF_PML);
  p.out = static_cast<uint16_t*>(out_device);
  p.err_flag = reinterpret_cast<int32_t*>(su->scratch + OFF_ERR);
  p.trace = nullptr;
  p.sched = reinterpret_cast<int32_t*>(su->scratch + OFF_SCHED);
  p.layer = 0; p.split_rows = 2 * split_tokens; p.max_splits = STATIC_MAX_SPLITS;
  p.tiles_per_chunk = split_tokens / (decode_tile_tokens() * decode_warps_per_cta() * 16);
  if (p.tiles_per_chunk < 1) p.tiles_per_chunk = 1;
  if (p.tiles_per_chunk > 16) p.tiles_per_chunk = 16;
  p.static_eighths = 5;
  p.scale_log2 = (sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)head_dim)) * 1.4426950408889634f;
  for (int w = 0; w < 8; ++w) p.score_read_mask[w] = 0u;
  p.early_ok = 0; p.optimistic = 0; p.closer = 0; p.seq = 0; p.force_redo = 0; p.keep_logits = 0;
  p.segment = 0; p.gate_tau = 2.f; p.dlse = nullptr; p.state_acc = nullptr; p.state_ml = nullptr;
  p.by_value = 1;
  p.v_len[0] = n_tokens; p.v_cap_d[0] = 0; p.v_row_base[0] = 0;
  p.heads_by_value = 0; p.plans_by_value = 0;

  // The array keeps whatever the previous call left: the chunk counters and the tickets must start at
  // zero.  The error word is left alone: only pod_dense_decode_attn_static_status reads and clears it.
  if (cudaMemsetAsync(su->scratch + OFF_SCHED, 0, SCHED_BYTES, stream) != cudaSuccess) return POD_ERR_CUDA;
  const int e = launch_decode(tmap, p, grid_splits, stream);
  return e == 0 ? POD_OK : POD_ERR_CUDA;
}

// Reads (and clears) the error word of the fixed array on the current device.  No allocation: a plain
// copy through the address cudaGetSymbolAddress gave.
extern "C" int pod_dense_decode_attn_static_status(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return POD_ERR_CUDA;
  DeviceSetup* su = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_setup[dev].ready) return POD_OK;              // nothing has run on this device
    su = &g_setup[dev];
  }
  int32_t flag = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return POD_ERR_CUDA;
  if (cudaMemcpy(&flag, su->scratch + OFF_ERR, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return POD_ERR_CUDA;
  if (flag != 0 && cudaMemset(su->scratch + OFF_ERR, 0, 4) != cudaSuccess) return POD_ERR_CUDA;
  return flag ? POD_ERR_DEVICE : POD_OK;
}

// Sets that error word from the host, as a kernel whose bounded wait gave up would (tests of the error path).
extern "C" int pod_dense_decode_attn_static_inject_error(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return POD_ERR_CUDA;
  DeviceSetup* su = nullptr;
  const int st = setup_device(dev, &su);
  if (st != POD_OK) return st;
  if (cudaDeviceSynchronize() != cudaSuccess) return POD_ERR_CUDA;
  const int32_t one = 1;
  return cudaMemcpy(su->scratch + OFF_ERR, &one, 4, cudaMemcpyHostToDevice) == cudaSuccess ? POD_OK : POD_ERR_CUDA;
}
