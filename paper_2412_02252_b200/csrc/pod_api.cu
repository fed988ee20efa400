// Host side of the PoD library: the C ABI of include/pod.h, argument validation, arena
// carving, length bookkeeping, split planning and kernel launches.
#include <cudaTypedefs.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/pod.h"
#include "pod_common.h"

using namespace pod;

namespace {

constexpr size_t ALIGN = 1024;        // internal offsets
constexpr size_t ARENA_ALIGN = 256;   // what a caller's arena must satisfy
constexpr int TARGET_CTAS_FOR_SPLITS = 148 * 2 * 4;   // used only to size the partial buffers
constexpr int SPLIT_OVERHEAD_TOKENS = 48;             // fixed cost of a CTA in the planner's model

size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

bool config_ok(const pod_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1 || c->batch < 1) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_q_heads % c->n_kv_heads != 0) return false;
  if (c->n_q_heads / c->n_kv_heads > 8) return false;
  if (c->group_size < 1 || c->n_sink < 0 || c->n_recent < 1) return false;
  if (c->n_kv_heads > 65535 || c->batch > 65535) return false;
  if (!(c->sm_scale >= 0.f) || isinf(c->sm_scale)) return false;
  return true;
}

int max_splits_for(const pod_config& c) {
  int per = (TARGET_CTAS_FOR_SPLITS + c.batch * c.n_kv_heads - 1) / (c.batch * c.n_kv_heads);
  if (per < 16) per = 16;
  if (per > MAX_SPLITS_CAP) per = MAX_SPLITS_CAP;
  return (per + 1) & ~1;   // even: the combine's bulk copies move 16-byte multiples
}

// Per-head partition of the layers into blocks of consecutive layers (Section 2.1, Algorithm 1).
struct BlockMap {
  std::vector<int32_t> low;        // [L][H_kv] lowest layer of the block of (layer, head)
  std::vector<int32_t> slot;       // [L][H_kv] key-store index of that block; a head's stores are adjacent
  std::vector<int32_t> head_base;  // [H_kv + 1] first key store of each head
  int n_slots = 0;
  bool shared = false;             // some block has more than one layer
};

// low[l][h] must be l (a block starts) or low[l-1][h] (the block goes on); low[0][h] = 0.
bool build_block_map(const pod_config& c, const int32_t* lowest, BlockMap* m) {
  const int L = c.n_layers, H = c.n_kv_heads;
  m->low.resize((size_t)L * H);
  m->slot.resize((size_t)L * H);
  m->head_base.assign((size_t)H + 1, 0);
  m->shared = false;
  for (int l = 0; l < L; ++l)
    for (int h = 0; h < H; ++h) {
      const int v = lowest ? lowest[(size_t)l * H + h] : l - l % c.group_size;
      const bool ok = v == l || (l > 0 && v == m->low[(size_t)(l - 1) * H + h]);
      if (!ok) return false;
      m->low[(size_t)l * H + h] = v;
      if (v != l) m->shared = true;
    }
  int next = 0;
  for (int h = 0; h < H; ++h) {
    m->head_base[h] = next;
    for (int l = 0; l < L; ++l) {
      if (m->low[(size_t)l * H + h] == l) ++next;
      m->slot[(size_t)l * H + h] = next - 1;
    }
  }
  m->head_base[H] = next;
  m->n_slots = next;
  return true;
}

struct Carve {
  std::vector<int64_t> seq_row_base;   // rows
  std::vector<int32_t> seq_cap_d;
  size_t off_len, off_rowbase, off_capd, off_low, off_slot, off_stash, off_pacc, off_pml, off_dlse, off_sacc, off_sml, off_err, off_sched, total;
  int64_t total_rows;
  int max_splits;
};

bool carve(const pod_config& c, const BlockMap& m, const int32_t* cap, Carve* out) {
  const int64_t row_bytes = (int64_t)c.head_dim * 2;
  out->max_splits = max_splits_for(c);
  out->seq_row_base.resize(c.batch);
  out->seq_cap_d.resize(c.batch);
  int64_t rows = 0;
  const int64_t SW = (int64_t)c.n_sink + c.n_recent;
  for (int b = 0; b < c.batch; ++b) {
    if (cap[b] < 1) return false;
    const int64_t cap_d = cap[b] > SW ? cap[b] - SW : 0;
    out->seq_row_base[b] = rows;
    out->seq_cap_d[b] = (int32_t)cap_d;
    rows += (int64_t)c.n_layers * 2 * c.n_kv_heads * SW + ((int64_t)c.n_layers * c.n_kv_heads + m.n_slots) * cap_d;
    {                                  // shared distant logits (only when some block has several layers)
      Layout y{};
      y.H_q = c.n_q_heads; y.H_kv = c.n_kv_heads; y.D = c.head_dim; y.shared = m.shared ? 1 : 0;
      rows += score_rows_per_seq(y, cap_d);
    }
  }
  if (rows >= ((int64_t)1 << 31)) return false;   // tile coordinates are 32-bit row indices
  out->total_rows = rows;
  size_t off = align_up((size_t)(rows * row_bytes));
  out->off_len = off;      off = align_up(off + (size_t)2 * c.n_layers * c.batch * 4);   // two copies, see len_cur
  out->off_rowbase = off;  off = align_up(off + (size_t)c.batch * 8);
  out->off_capd = off;     off = align_up(off + (size_t)c.batch * 4);
  out->off_low = off;      off = align_up(off + (size_t)c.n_layers * c.n_kv_heads * 4);
  out->off_slot = off;     off = align_up(off + (size_t)c.n_layers * c.n_kv_heads * 4);
  out->off_stash = off;    off = align_up(off + (size_t)m.n_slots * c.batch * (c.n_q_heads / c.n_kv_heads) * row_bytes);
  out->off_pacc = off;     off = align_up(off + (size_t)c.batch * c.n_q_heads * out->max_splits * c.head_dim * 4);
  out->off_pml = off;      off = align_up(off + (size_t)c.batch * c.n_q_heads * out->max_splits * 4 * 4);
  out->off_dlse = off;     off = align_up(off + (size_t)c.batch * c.n_q_heads * 4);
  out->off_sacc = off;     off = align_up(off + (size_t)c.batch * c.n_q_heads * c.head_dim * 4);
  out->off_sml = off;      off = align_up(off + (size_t)c.batch * c.n_q_heads * 2 * 4);
  out->off_err = off;      off = align_up(off + 4);
  out->off_sched = off;    off = align_up(off + (size_t)c.batch * c.n_kv_heads * SCHED_STRIDE * 4);
  out->total = off;
  return true;
}

}  // namespace

struct pod_cache {
  pod_config cfg;
  std::vector<int32_t> cap;            // [B]
  std::vector<int32_t> len;            // host mirror [L][B]
  std::vector<int32_t> stash_len;      // [n_slots][B]: lengths at which a block's q was stashed, -1 = none
  BlockMap bm;
  Carve cv;
  unsigned char* arena = nullptr;
  bool owns_arena = false;
  bool dry = false;
  int last_cuda = 0;
  int sm_count = 148, resident = 2;
  bool keep_logits = false;            // the logit stores are a small part of the L2: they are written and read with evict_last
  int last_decode_layer = -1;          // layer of the previous launch on this cache if it was a decode launch, else -1
  std::vector<int32_t> score_low;      // [H_kv] lowest layer whose distant logits the head's score store holds, -1 = none
  std::vector<int32_t> score_len;      // [H_kv][B] lengths at which they were stored
  std::vector<uint32_t> done_total;    // [B][H_kv] what the head's DONE word reads when all launches so far are through with it
  std::vector<uint32_t> score_done;    // [B][H_kv] done_total right after the launch that stored the head's logits
  int32_t launch_seq = 0;              // decode kernels launched on this cache so far
  bool optimistic = true;              // POD_OPTIMISTIC=0 switches the optimistic start off
  bool closer = true;                  // POD_CLOSER=0: every CTA takes a counted ticket even when the grid fits the GPU
  bool inject_stale = false;           // pod_cache_inject_stale_query: the next launch treats its early q as stale
  int force_split_tokens = 0;          // POD_SPLIT_TOKENS > 0 overrides the planner
  int force_chunk_tiles = 0;           // POD_CHUNK_TILES > 0 overrides the tiles per draw
  int static_eighths = 5;              // POD_STATIC_EIGHTHS: share of a warp's chunks assigned without a draw
  float gate_tau = 2.f;                // gate threshold; above 1 = the distant tokens are never skipped
  float scale = 0.f;
  Layout y{};
  CUtensorMap tmap{};                  // the region rows of the arena as a [rows][d] bf16 tensor
  unsigned long long* trace = nullptr; // caller's device buffer of (start, end) pairs, one per kernel launch
  int trace_cap = 0, trace_n = 0;
  // last launch (diagnostics)
  int32_t last_split_tokens = 0, last_ctas = 0, last_kernels = 0;
  // planner memo
  int64_t memo_sum = -1; int32_t memo_max = -1; int memo_light = -1, memo_segment = -1; DecodePlan memo_plan{};

  // Device lengths are kept twice.  A launch that appends and attends at once reads one copy and
  // writes the other (its CTAs start at different times, so nobody may change what they read);
  // len_cur[layer] says which copy is current.
  std::vector<uint8_t> len_cur;        // [L]
  int32_t* d_len_copy(int layer, int which) const {
    return reinterpret_cast<int32_t*>(arena + cv.off_len) + ((size_t)which * cfg.n_layers + layer) * cfg.batch;
  }
  int32_t* d_len(int layer) const { return d_len_copy(layer, len_cur[layer]); }
  int32_t& h_len(int layer, int b) { return len[(size_t)layer * cfg.batch + b]; }
  int32_t h_len(int layer, int b) const { return len[(size_t)layer * cfg.batch + b]; }
  int low_of(int layer, int head) const { return bm.low[(size_t)layer * cfg.n_kv_heads + head]; }
  int slot_of(int layer, int head) const { return bm.slot[(size_t)layer * cfg.n_kv_heads + head]; }
};

namespace {

int cuda_fail(pod_cache* c, cudaError_t e) {
  c->last_cuda = (int)e;
  return POD_ERR_CUDA;
}

// One tensor map over all region rows: dims (d, rows), box (64 channels, tile rows), 128-byte
// swizzle.  Loads past the last row are zero-filled.
bool make_tensor_map(pod_cache* c) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr)
    return false;
  auto encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  const pod_config& g = c->cfg;
  cuuint64_t dims[2] = {(cuuint64_t)g.head_dim, (cuuint64_t)c->cv.total_rows};
  cuuint64_t strides[1] = {(cuuint64_t)g.head_dim * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)decode_tile_tokens()};
  cuuint32_t estr[2] = {1u, 1u};
  const CUresult r = encode(&c->tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c->arena, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Picks the tokens-per-split that minimises a simple time model: the CTAs run in waves of
// (SMs x resident CTAs), every CTA costs its tokens plus a fixed overhead.
// Picks the rows-per-split that minimises a simple time model: the CTAs run in waves of
// (SMs x resident CTAs), every CTA costs its rows plus a fixed overhead.  A head that reads keys and
// values streams 2 n rows, a head that reads the block's stored logits n + n_p; n_light heads of
// this launch are of the second kind.
DecodePlan plan_decode(pod_cache* c, int layer, int n_light, int segment) {
  const pod_config& g = c->cfg;
  const int n_heavy = g.n_kv_heads - n_light;
  const int64_t SW = (int64_t)g.n_sink + g.n_recent;
  int64_t sum = 0; int32_t nmax = 0;
  for (int b = 0; b < g.batch; ++b) { const int32_t n = c->h_len(layer, b); sum += n; if (n > nmax) nmax = n; }
  if (sum == c->memo_sum && nmax == c->memo_max && n_light == c->memo_light && segment == c->memo_segment)
    return c->memo_plan;
  // segment 1 streams the proximal tokens only, segment 2 the distant tokens only, 0 both
  auto prox = [SW, segment](int64_t n) { return segment == 2 ? (int64_t)0 : (n < SW ? n : SW); };
  auto dist = [SW, segment](int64_t n) { return segment == 1 ? (int64_t)0 : (n > SW ? n - SW : (int64_t)0); };
  auto heavy_rows = [&](int64_t n) { return 2 * (prox(n) + dist(n)); };
  auto light_rows = [&](int64_t n) { return 2 * prox(n) + dist(n); };
  auto count = [&](int64_t st, int64_t* ctas, int64_t* most) {
    *ctas = 0; *most = 0;
    for (int b = 0; b < g.batch; ++b) {
      const int64_t n = c->h_len(layer, b);
      const int64_t kh = (heavy_rows(n) + st - 1) / st, kl = (light_rows(n) + st - 1) / st;
      *ctas += n_heavy * kh + n_light * kl;
      const int64_t m = n_heavy > 0 ? kh : kl;
      if (m > *most) *most = m;
    }
  };
  const int64_t wmax = n_heavy > 0 ? heavy_rows(nmax) : light_rows(nmax);
  DecodePlan best{2, 1, 0};
  if (wmax > 0 && c->force_split_tokens > 0) {      // POD_SPLIT_TOKENS: tuning experiments
    int64_t st = 2 * (int64_t)c->force_split_tokens;
    if (st < (wmax + c->cv.max_splits - 1) / c->cv.max_splits) st = (wmax + c->cv.max_splits - 1) / c->cv.max_splits;
    int64_t ctas, most;
    count(st, &ctas, &most);
    best = DecodePlan{(int32_t)st, (int32_t)most, (int32_t)ctas};
  } else if (wmax > 0) {
    const int64_t slots = (int64_t)c->sm_count * c->resident;
    double best_cost = 1e300;
    int64_t last_st = -1;
    for (int k = 1; k <= c->cv.max_splits; ++k) {
      const int64_t st = (wmax + k - 1) / k;
      if (st == last_st) continue;
      last_st = st;
      int64_t ctas, most;
      count(st, &ctas, &most);
      const int64_t waves = (ctas + slots - 1) / slots;
      const double cost = (double)waves * (st + 2 * SPLIT_OVERHEAD_TOKENS);
      if (cost < best_cost * 0.999) { best_cost = cost; best = DecodePlan{(int32_t)st, (int32_t)most, (int32_t)ctas}; }
      if (st <= 128) break;
    }
  }
  c->memo_sum = sum; c->memo_max = nmax; c->memo_light = n_light; c->memo_segment = segment; c->memo_plan = best;
  return best;
}

}  // namespace

extern "C" {

const char* pod_strerror(int status) {
  switch (status) {
    case POD_OK: return "ok";
    case POD_DRY_RUN: return "host-only cache: validated, nothing launched";
    case POD_ERR_INVALID: return "invalid argument";
    case POD_ERR_CAPACITY: return "sequence capacity exceeded";
    case POD_ERR_ORDER: return "decode order violated: block lengths differ or lowest layer not decoded";
    case POD_ERR_ARENA: return "arena too small or misaligned";
    case POD_ERR_CUDA: return "CUDA runtime error";
    case POD_ERR_DEVICE: return "a kernel gave up a bounded wait";
    default: return "unknown status";
  }
}

static size_t required_bytes_impl(const pod_config* cfg, const int32_t* seq_capacity, const int32_t* lowest) {
  if (!config_ok(cfg) || !seq_capacity) return 0;
  BlockMap bm;
  Carve cv;
  if (!build_block_map(*cfg, lowest, &bm) || !carve(*cfg, bm, seq_capacity, &cv)) return 0;
  return cv.total;
}

size_t pod_cache_required_bytes(const pod_config* cfg, const int32_t* seq_capacity) {
  return required_bytes_impl(cfg, seq_capacity, nullptr);
}

size_t pod_cache_required_bytes_blocks(const pod_config* cfg, const int32_t* seq_capacity,
                                       const int32_t* lowest_layer) {
  return lowest_layer ? required_bytes_impl(cfg, seq_capacity, lowest_layer) : 0;
}

static int create_impl(const pod_config* cfg, const int32_t* seq_capacity, const int32_t* lowest,
                       void* arena_device, size_t arena_bytes, pod_cache** out) {
  if (!out) return POD_ERR_INVALID;
  *out = nullptr;
  if (!config_ok(cfg) || !seq_capacity) return POD_ERR_INVALID;
  pod_cache* c = new (std::nothrow) pod_cache();
  if (!c) return POD_ERR_INVALID;
  c->cfg = *cfg;
  if (!build_block_map(*cfg, lowest, &c->bm) || !carve(*cfg, c->bm, seq_capacity, &c->cv)) { delete c; return POD_ERR_INVALID; }
  c->cap.assign(seq_capacity, seq_capacity + cfg->batch);
  c->len.assign((size_t)cfg->n_layers * cfg->batch, 0);
  c->len_cur.assign((size_t)cfg->n_layers, 0);
  c->score_low.assign((size_t)cfg->n_kv_heads, -1);
  c->score_len.assign((size_t)cfg->n_kv_heads * cfg->batch, -1);
  c->done_total.assign((size_t)cfg->n_kv_heads * cfg->batch, 0u);
  c->score_done.assign((size_t)cfg->n_kv_heads * cfg->batch, 0u);
  c->stash_len.assign((size_t)c->bm.n_slots * cfg->batch, -1);
  c->scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / sqrtf((float)cfg->head_dim);
  c->dry = cfg->device < 0;
  Layout& y = c->y;
  y.L = cfg->n_layers; y.H_kv = cfg->n_kv_heads; y.H_q = cfg->n_q_heads; y.D = cfg->head_dim;
  y.S = cfg->n_sink; y.W = cfg->n_recent; y.B = cfg->batch;
  y.n_slots = c->bm.n_slots; y.shared = c->bm.shared ? 1 : 0;
  if (c->dry) { *out = c; return POD_OK; }

  cudaError_t e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) { delete c; return POD_ERR_CUDA; }
  if (arena_device) {
    if (((uintptr_t)arena_device % ARENA_ALIGN) != 0 || arena_bytes < c->cv.total) { delete c; return POD_ERR_ARENA; }
    c->arena = static_cast<unsigned char*>(arena_device);
  } else {
    void* pmem = nullptr;
    e = cudaMalloc(&pmem, c->cv.total);
    if (e != cudaSuccess) { delete c; return POD_ERR_CUDA; }
    c->arena = static_cast<unsigned char*>(pmem);
    c->owns_arena = true;
  }
  y.seq_row_base = reinterpret_cast<const int64_t*>(c->arena + c->cv.off_rowbase);
  y.seq_cap_d = reinterpret_cast<const int32_t*>(c->arena + c->cv.off_capd);
  y.low = reinterpret_cast<const int32_t*>(c->arena + c->cv.off_low);
  y.slot = reinterpret_cast<const int32_t*>(c->arena + c->cv.off_slot);
  bool ok = true;
  // Tiles of the decode kernel may extend past the rows a head holds into neighbouring rows;
  // their logits are masked, but the rows must hold finite numbers, so the arena starts zeroed.
  ok = ok && cudaMemset(c->arena, 0, c->cv.total) == cudaSuccess;
  ok = ok && make_tensor_map(c);
  ok = ok && cudaMemcpy(c->arena + c->cv.off_rowbase, c->cv.seq_row_base.data(), (size_t)cfg->batch * 8, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->arena + c->cv.off_capd, c->cv.seq_cap_d.data(), (size_t)cfg->batch * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->arena + c->cv.off_low, c->bm.low.data(), c->bm.low.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->arena + c->cv.off_slot, c->bm.slot.data(), c->bm.slot.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  int sm = 0;
  ok = ok && cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess;
  int l2_bytes = 0;
  ok = ok && cudaDeviceGetAttribute(&l2_bytes, cudaDevAttrL2CacheSize, cfg->device) == cudaSuccess;
  const int res = ok ? decode_resident_ctas_per_sm(cfg->head_dim) : 0;
  ok = ok && res > 0 && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    if (c->owns_arena) cudaFree(c->arena);
    delete c;
    return POD_ERR_CUDA;
  }
  c->sm_count = sm; c->resident = res;
  {                                    // all logit stores of the cache at capacity against the L2
    int64_t rows = 0;
    for (int b = 0; b < cfg->batch; ++b) rows += score_rows_per_seq(c->y, c->cv.seq_cap_d[b]);
    c->keep_logits = rows > 0 && rows * cfg->head_dim * 2 <= (int64_t)l2_bytes / 8;
  }
  if (const char* ct = getenv("POD_CHUNK_TILES")) c->force_chunk_tiles = atoi(ct);
  if (const char* se = getenv("POD_STATIC_EIGHTHS")) {
    const int v = atoi(se);
    if (v >= 0 && v <= 8) c->static_eighths = v;
  }
  if (const char* op = getenv("POD_OPTIMISTIC")) c->optimistic = atoi(op) != 0;
  if (const char* cl = getenv("POD_CLOSER")) c->closer = atoi(cl) != 0;
  const char* fst = getenv("POD_SPLIT_TOKENS");
  c->force_split_tokens = fst ? atoi(fst) : 0;
  *out = c;
  return POD_OK;
}

int pod_cache_create(const pod_config* cfg, const int32_t* seq_capacity, void* arena_device,
                     size_t arena_bytes, pod_cache** out) {
  return create_impl(cfg, seq_capacity, nullptr, arena_device, arena_bytes, out);
}

int pod_cache_create_blocks(const pod_config* cfg, const int32_t* seq_capacity, const int32_t* lowest_layer,
                            void* arena_device, size_t arena_bytes, pod_cache** out) {
  if (out) *out = nullptr;
  if (!lowest_layer) return POD_ERR_INVALID;
  return create_impl(cfg, seq_capacity, lowest_layer, arena_device, arena_bytes, out);
}

// Algorithm 1 (Section 2.1): for each head, layer 0 opens a block; each next layer joins the
// current block if its similarity to every layer already in that block reaches the threshold,
// otherwise it opens a new block.
int pod_greedy_layer_blocks(const float* sim, int n_heads, int n_layers, float threshold, int32_t* lowest_layer) {
  if (!sim || !lowest_layer || n_heads < 1 || n_layers < 1) return POD_ERR_INVALID;
  for (int h = 0; h < n_heads; ++h) {
    const float* sh = sim + (size_t)h * n_layers * n_layers;
    int start = 0;                                   // lowest layer of the current block
    lowest_layer[h] = 0;
    for (int l = 1; l < n_layers; ++l) {
      bool similar_to_all = true;
      for (int m = start; m < l && similar_to_all; ++m) similar_to_all = sh[(size_t)l * n_layers + m] >= threshold;
      if (!similar_to_all) start = l;
      lowest_layer[(size_t)l * n_heads + h] = start;
    }
  }
  return POD_OK;
}

// Split of one cache over `world` GPUs by KV head: rank r keeps KV heads [r * H_kv / world, (r + 1) * H_kv / world)
// and the query heads that read them.  Every region is per KV head, so the rank's cache is an ordinary
// cache of H_kv / world heads; outputs of the ranks are disjoint slices of [B][H_q][d].
int pod_shard_config(const pod_config* full, int rank, int world, pod_config* local, int32_t* first_kv_head,
                     int32_t* first_q_head) {
  if (!config_ok(full) || !local || world < 1 || rank < 0 || rank >= world) return POD_ERR_INVALID;
  if (full->n_kv_heads % world != 0) return POD_ERR_INVALID;
  const int per = full->n_kv_heads / world, r = full->n_q_heads / full->n_kv_heads;
  *local = *full;
  local->n_kv_heads = per;
  local->n_q_heads = per * r;
  if (first_kv_head) *first_kv_head = rank * per;
  if (first_q_head) *first_q_head = rank * per * r;
  return POD_OK;
}

int pod_shard_block_map(const pod_config* full, const int32_t* lowest_layer, int rank, int world,
                        int32_t* local_lowest_layer) {
  if (!config_ok(full) || !lowest_layer || !local_lowest_layer || world < 1 || rank < 0 || rank >= world) return POD_ERR_INVALID;
  if (full->n_kv_heads % world != 0) return POD_ERR_INVALID;
  const int H = full->n_kv_heads, per = H / world;
  for (int l = 0; l < full->n_layers; ++l)
    for (int h = 0; h < per; ++h)
      local_lowest_layer[(size_t)l * per + h] = lowest_layer[(size_t)l * H + rank * per + h];
  return POD_OK;
}

int pod_cache_destroy(pod_cache* c) {
  if (!c) return POD_ERR_INVALID;
  int st = POD_OK;
  if (!c->dry) {
    cudaSetDevice(c->cfg.device);
    if (cudaDeviceSynchronize() != cudaSuccess) st = POD_ERR_CUDA;
    if (c->owns_arena && cudaFree(c->arena) != cudaSuccess) st = POD_ERR_CUDA;
  }
  delete c;
  return st;
}

int pod_cache_write(pod_cache* c, int layer, int seq, const void* k, const void* v, int n_tokens,
                    void* stream) {
  if (!c || !k || !v) return POD_ERR_INVALID;
  const pod_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers || seq < -1 || seq >= g.batch || n_tokens < 1) return POD_ERR_INVALID;
  if (seq == -1 && n_tokens != 1) return POD_ERR_INVALID;
  if (((uintptr_t)k % 16) != 0 || ((uintptr_t)v % 16) != 0) return POD_ERR_INVALID;
  const int b0 = seq < 0 ? 0 : seq, b1 = seq < 0 ? g.batch : seq + 1;
  for (int b = b0; b < b1; ++b)
    if ((int64_t)c->h_len(layer, b) + n_tokens > c->cap[b]) return POD_ERR_CAPACITY;
  if (!c->dry) {
    WriteParams p;
    p.y = c->y;
    p.arena = reinterpret_cast<uint16_t*>(c->arena);
    p.k = static_cast<const uint16_t*>(k);
    p.v = static_cast<const uint16_t*>(v);
    p.len = c->d_len(layer);
    p.layer = layer; p.seq = seq; p.n0 = seq < 0 ? 0 : c->h_len(layer, seq); p.T = n_tokens;
    const int e = launch_write(p, static_cast<cudaStream_t>(stream));
    if (e != 0) return cuda_fail(c, (cudaError_t)e);
  }
  for (int b = b0; b < b1; ++b) c->h_len(layer, b) += n_tokens;
  c->memo_sum = -1;
  c->last_decode_layer = -1;
  return c->dry ? POD_DRY_RUN : POD_OK;
}

// pod_decode_attn (k_new == nullptr) and pod_append_decode_attn (k_new, v_new: one new token per
// sequence, appended by the same launch that attends).
static int decode_impl(pod_cache* c, int layer, const void* k_new, const void* v_new, const void* q, void* out,
                       void* stream) {
  if (!c || !q || !out) return POD_ERR_INVALID;
  const bool fused = k_new != nullptr;
  if (fused && (!v_new || ((uintptr_t)k_new % 16) != 0 || ((uintptr_t)v_new % 16) != 0)) return POD_ERR_INVALID;
  const pod_config& g = c->cfg;
  if (layer < 0 || layer >= g.n_layers) return POD_ERR_INVALID;
  if (((uintptr_t)q % 16) != 0 || ((uintptr_t)out % 16) != 0) return POD_ERR_INVALID;
  const int H = g.n_kv_heads;
  const int add = fused ? 1 : 0;
  auto stash_len_of = [&](int head) { return &c->stash_len[(size_t)c->slot_of(layer, head) * g.batch]; };
  if (fused)
    for (int b = 0; b < g.batch; ++b)
      if ((int64_t)c->h_len(layer, b) + 1 > c->cap[b]) return POD_ERR_CAPACITY;
  for (int h = 0; h < H; ++h) {          // every head whose block started at a lower layer
    const int low = c->low_of(layer, h);
    if (low == layer) continue;
    const int32_t* sl = stash_len_of(h);
    for (int b = 0; b < g.batch; ++b) {
      const int32_t n = c->h_len(layer, b) + add;
      if (n != c->h_len(low, b)) return POD_ERR_ORDER;       // block must hold equal lengths
      if (n > 0 && sl[b] != n) return POD_ERR_ORDER;         // lowest layer's q not stashed at this step
    }
  }
  auto note_stash = [&]() {              // heads for which this layer is the lowest of their block
    for (int h = 0; h < H; ++h)
      if (c->low_of(layer, h) == layer) {
        int32_t* sl = stash_len_of(h);
        for (int b = 0; b < g.batch; ++b) sl[b] = c->h_len(layer, b);
      }
  };
  if (fused) {                          // from here on the host lengths are the new ones
    for (int b = 0; b < g.batch; ++b) c->h_len(layer, b) += 1;
    c->memo_sum = -1;
  }
  if (c->dry) {
    note_stash();
    return POD_DRY_RUN;
  }
  DecodeParams p;
  p.y = c->y;
  p.arena = reinterpret_cast<const uint16_t*>(c->arena);
  p.len = c->d_len(layer);
  p.new_k = static_cast<const uint16_t*>(k_new);
  p.new_v = static_cast<const uint16_t*>(v_new);
  p.len_out = fused ? c->d_len_copy(layer, c->len_cur[layer] ^ 1) : nullptr;
  p.q = static_cast<const uint16_t*>(q);
  p.stash = reinterpret_cast<uint16_t*>(c->arena + c->cv.off_stash);
  p.part_acc = reinterpret_cast<float*>(c->arena + c->cv.off_pacc);
  p.part_ml = reinterpret_cast<float*>(c->arena + c->cv.off_pml);
  p.out = static_cast<uint16_t*>(out);
  p.err_flag = reinterpret_cast<int32_t*>(c->arena + c->cv.off_err);
  p.sched = reinterpret_cast<int32_t*>(c->arena + c->cv.off_sched);
  p.layer = layer;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  // Shared distant logits, head by head: the lowest layer of a block of several layers stores them
  // (the kernel decides that from the block tables); a head of another layer reads them if its
  // store holds the logits of its block at exactly these lengths, else it scores the block's keys.
  for (int w = 0; w < 8; ++w) p.score_read_mask[w] = 0u;
  int n_light = 0;                       // heads of this launch that read stored logits
  for (int h = 0; h < H && h < 256; ++h) {
    const int low = c->low_of(layer, h);
    if (low == layer || c->score_low[h] != low) continue;
    bool same = true;
    for (int b = 0; b < g.batch; ++b) same = same && c->score_len[(size_t)h * g.batch + b] == c->h_len(layer, b);
    if (same) { p.score_read_mask[h >> 5] |= 1u << (h & 31); ++n_light; }
  }
  p.dlse = reinterpret_cast<float*>(c->arena + c->cv.off_dlse);
  p.state_acc = reinterpret_cast<float*>(c->arena + c->cv.off_sacc);
  p.state_ml = reinterpret_cast<float*>(c->arena + c->cv.off_sml);
  p.gate_tau = c->gate_tau;
  p.max_splits = c->cv.max_splits;
  p.static_eighths = c->static_eighths;
  p.by_value = g.batch <= SMALL_BATCH ? 1 : 0;
  for (int b = 0; b < SMALL_BATCH; ++b) {
    const bool in = p.by_value && b < g.batch;
    p.v_len[b] = in ? c->h_len(layer, b) : 0;
    p.v_cap_d[b] = in ? c->cv.seq_cap_d[b] : 0;
    p.v_row_base[b] = in ? c->cv.seq_row_base[b] : 0;
  }
  p.heads_by_value = H <= SMALL_HEADS ? 1 : 0;
  p.v_store_mask = 0u;
  for (int h = 0; h < SMALL_HEADS; ++h) {
    const bool in = p.heads_by_value && h < H;
    p.v_low[h] = in ? c->low_of(layer, h) : 0;
    p.v_slot[h] = in ? c->slot_of(layer, h) : 0;
    if (in && c->bm.shared && c->low_of(layer, h) == layer && layer + 1 < g.n_layers && c->low_of(layer + 1, h) == layer)
      p.v_store_mask |= 1u << h;
  }
  // With a gate threshold set, a layer in which some head reads its block's logits runs as two
  // launches: the proximal tokens (which decides, per query head, whether the distant tokens are
  // omitted), then the distant tokens of the KV heads that still need them.
  const bool gated = c->gate_tau <= 1.f && n_light > 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int kernels = 0;
  DecodePlan plan{2, 1, 0};
  for (int pass = 0; pass < (gated ? 2 : 1); ++pass) {
    p.segment = gated ? pass + 1 : 0;
    plan = plan_decode(c, layer, n_light, p.segment);
    p.split_rows = plan.split_rows;
    {
      // A warp sees about split_rows / (2 x tile tokens x warps) tiles; it should make a dozen draws, of two
      // tiles at least (consecutive rows; measured: 0.9 us per launch at 32K against single tiles) unless it
      // has only a handful of tiles.
      const int per_warp = plan.split_rows / (2 * decode_tile_tokens() * decode_warps_per_cta());
      int tch = per_warp / 16;
      if (tch < 2 && per_warp >= 6) tch = 2;
      if (c->force_chunk_tiles > 0) tch = c->force_chunk_tiles;
      p.tiles_per_chunk = tch < 1 ? 1 : (tch > 256 ? 256 : tch);
    }
    // Small launches carry the plan of every (sequence, KV head) by value.
    p.plans_by_value = (g.batch * H <= SMALL_PLANS) ? 1 : 0;
    if (p.plans_by_value) {
      PlanInputs in;
      in.layer = layer; in.segment = p.segment; in.fused = (fused && pass == 0) ? 1 : 0; in.max_splits = p.max_splits;
      in.split_rows = p.split_rows; in.tiles_per_chunk = p.tiles_per_chunk; in.static_eighths = p.static_eighths;
      in.tile_tokens = decode_tile_tokens(); in.warps = decode_warps_per_cta();
      for (int b = 0; b < g.batch; ++b)
        for (int h = 0; h < H; ++h) {
          const int low = c->low_of(layer, h);
          const bool store = c->bm.shared && low == layer && layer + 1 < g.n_layers && c->low_of(layer + 1, h) == layer;
          const bool read = low != layer && h < 256 && ((p.score_read_mask[h >> 5] >> (h & 31)) & 1u);
          HeadPlan& hp = p.v_plan[b * H + h];
          hp = make_head_plan(p.y, in, h, c->h_len(layer, b), c->cv.seq_cap_d[b], c->cv.seq_row_base[b], low,
                              c->slot_of(layer, h), store, read);
          hp.wait_done = (int32_t)c->score_done[(size_t)b * H + h];
        }
    }
    // A launch that appends and attends streams only rows written before this step (the new token's
    // and the displaced token's rows are handled apart); the one launch that may still be running is
    // the previous one on this cache, which touches other rows if it was a decode of another layer.
    // The distant launch of a gated layer follows its own proximal launch, which moved rows: no early start.
    p.early_ok = (fused && pass == 0 && c->last_decode_layer >= 0 && c->last_decode_layer != layer) ? 1 : 0;
    if (pass == 1) {                      // the append is done: the distant launch only attends
      p.new_k = nullptr; p.new_v = nullptr; p.len_out = nullptr;
      p.len = c->d_len(layer);
    }
    if (plan.n_ctas == 0) continue;
    // Optimistic start: for launches that may start early, of caches with few enough heads that the per-head
    // sequence numbers travel by value; not for the two launches of a gated layer.
    p.optimistic = (p.early_ok && !gated && c->optimistic && p.plans_by_value) ? 1 : 0;
    p.seq = ++c->launch_seq;
    // every CTA gets a slot on some SM without another CTA of the grid leaving first
    p.closer = (c->closer && (int64_t)p.y.H_kv * plan.grid_splits * p.y.B <= (int64_t)c->sm_count * c->resident) ? 1 : 0;
    p.force_redo = (c->inject_stale && !gated) ? 1 : 0;
    p.keep_logits = c->keep_logits ? 1 : 0;
    c->inject_stale = false;
    p.trace = (c->trace != nullptr && c->trace_n < c->trace_cap) ? c->trace + 2 * (size_t)c->trace_n++ : nullptr;
    const int e = launch_decode(c->tmap, p, plan.grid_splits, s);
    if (e != 0) {
      if (fused && pass == 0) { for (int b = 0; b < g.batch; ++b) c->h_len(layer, b) -= 1; c->memo_sum = -1; }
      return cuda_fail(c, (cudaError_t)e);
    }
    ++kernels;
    if (fused && pass == 0) c->len_cur[layer] ^= 1;
    if (p.plans_by_value)                 // every CTA of a head that stores its logits adds one to the head's DONE word
      for (int i = 0; i < g.batch * H; ++i)
        if (p.v_plan[i].flags & HP_STORE) c->done_total[i] += (uint32_t)p.v_plan[i].nsplit;
  }
  {
    bool any_empty = false;
    for (int b = 0; b < g.batch; ++b) any_empty = any_empty || c->h_len(layer, b) == 0;
    if (any_empty) {                      // no split CTA exists for an empty sequence
      const int e2 = launch_zero_empty(p, s);
      if (e2 != 0) return cuda_fail(c, (cudaError_t)e2);
      ++kernels;
    }
  }
  note_stash();
  for (int h = 0; h < H; ++h) {          // heads whose block starts here and goes on: their logits are stored now
    if (c->low_of(layer, h) != layer || layer + 1 >= g.n_layers || c->low_of(layer + 1, h) != layer) continue;
    c->score_low[h] = layer;
    for (int b = 0; b < g.batch; ++b) c->score_done[(size_t)b * H + h] = c->done_total[(size_t)b * H + h];
    for (int b = 0; b < g.batch; ++b) c->score_len[(size_t)h * g.batch + b] = c->h_len(layer, b);
  }
  c->last_decode_layer = layer;
  c->last_split_tokens = plan.split_rows / 2; c->last_ctas = plan.n_ctas; c->last_kernels = kernels;   // of the last launch
  return POD_OK;
}

int pod_cache_set_gate_threshold(pod_cache* c, float tau) {
  if (!c || !(tau >= 0.f)) return POD_ERR_INVALID;      // rejects NaN too
  c->gate_tau = tau;
  return c->dry ? POD_DRY_RUN : POD_OK;
}

int pod_decode_attn(pod_cache* c, int layer, const void* q, void* out, void* stream) {
  return decode_impl(c, layer, nullptr, nullptr, q, out, stream);
}

int pod_append_decode_attn(pod_cache* c, int layer, const void* k, const void* v, const void* q, void* out,
                           void* stream) {
  if (!k || !v) return POD_ERR_INVALID;
  return decode_impl(c, layer, k, v, q, out, stream);
}

int64_t pod_cache_bytes(const pod_cache* c, int which) {
  if (!c) return -1;
  const pod_config& g = c->cfg;
  const int64_t row = (int64_t)g.head_dim * 2;
  if (which == POD_BYTES_ALLOCATED) return (int64_t)c->cv.total;
  if (which != POD_BYTES_LIVE && which != POD_BYTES_DENSE_EQUIV) return -1;
  const int64_t SW = (int64_t)g.n_sink + g.n_recent;
  int64_t total = 0;
  for (int b = 0; b < g.batch; ++b) {
    // count what each layer and each block store actually holds
    for (int l = 0; l < g.n_layers; ++l) {
      const int64_t n = c->h_len(l, b);
      const int64_t n_p = n < SW ? n : SW, n_d = n - n_p;
      if (which == POD_BYTES_DENSE_EQUIV) { total += g.n_kv_heads * row * 2 * n; continue; }
      total += g.n_kv_heads * row * (2 * n_p + n_d);
      for (int h = 0; h < g.n_kv_heads; ++h)
        if (c->low_of(l, h) == l) total += row * n_d;       // distant keys are kept once per block
    }
  }
  return total;
}

int pod_cache_seq_len(const pod_cache* c, int seq, int layer) {
  if (!c || seq < 0 || seq >= c->cfg.batch || layer < 0 || layer >= c->cfg.n_layers) return POD_ERR_INVALID;
  return c->h_len(layer, seq);
}

int pod_cache_reset(pod_cache* c, int seq) {
  if (!c || seq < -1 || seq >= c->cfg.batch) return POD_ERR_INVALID;
  const pod_config& g = c->cfg;
  const int b0 = seq < 0 ? 0 : seq, b1 = seq < 0 ? g.batch : seq + 1;
  for (int l = 0; l < g.n_layers; ++l)
    for (int b = b0; b < b1; ++b) c->h_len(l, b) = 0;
  for (int sl = 0; sl < c->bm.n_slots; ++sl)
    for (int b = b0; b < b1; ++b) c->stash_len[(size_t)sl * g.batch + b] = -1;
  c->memo_sum = -1;
  for (auto& x : c->score_low) x = -1;
  c->last_decode_layer = -1;
  if (c->dry) return POD_DRY_RUN;
  cudaError_t e = cudaSetDevice(g.device);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess)
    e = cudaMemcpy(c->arena + c->cv.off_len, c->len.data(), c->len.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess)
    e = cudaMemcpy(c->arena + c->cv.off_len + c->len.size() * 4, c->len.data(), c->len.size() * 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(c, e);
  return POD_OK;
}

int pod_cache_read_region(const pod_cache* c, int region, int layer_or_block, int seq, int kv_head,
                          int first, int count, void* host_dst) {
  if (!c || !host_dst || c->dry) return POD_ERR_INVALID;
  const pod_config& g = c->cfg;
  if (seq < 0 || seq >= g.batch || kv_head < 0 || kv_head >= g.n_kv_heads || first < 0 || count < 0) return POD_ERR_INVALID;
  const bool is_block = (region == POD_REGION_DIST_K);
  const int n_head_blocks = c->bm.head_base[kv_head + 1] - c->bm.head_base[kv_head];
  if (layer_or_block < 0 || layer_or_block >= (is_block ? n_head_blocks : g.n_layers)) return POD_ERR_INVALID;
  const int64_t cap_d = c->cv.seq_cap_d[seq];
  int64_t row, extent;
  switch (region) {
    case POD_REGION_SINK_K: row = prox_row(c->y, layer_or_block, 0, kv_head); extent = g.n_sink; break;
    case POD_REGION_SINK_V: row = prox_row(c->y, layer_or_block, 1, kv_head); extent = g.n_sink; break;
    case POD_REGION_RING_K: row = prox_row(c->y, layer_or_block, 0, kv_head) + g.n_sink; extent = g.n_recent; break;
    case POD_REGION_RING_V: row = prox_row(c->y, layer_or_block, 1, kv_head) + g.n_sink; extent = g.n_recent; break;
    case POD_REGION_DIST_K: row = distk_row(c->y, c->bm.head_base[kv_head] + layer_or_block, cap_d); extent = cap_d; break;
    case POD_REGION_DIST_V: row = distv_row(c->y, layer_or_block, kv_head, cap_d); extent = cap_d; break;
    default: return POD_ERR_INVALID;
  }
  if ((int64_t)first + count > extent) return POD_ERR_INVALID;
  if (count == 0) return POD_OK;
  const size_t row_bytes = (size_t)g.head_dim * 2;
  const unsigned char* src = c->arena + (size_t)(c->cv.seq_row_base[seq] + row + first) * row_bytes;
  cudaError_t e = cudaSetDevice(g.device);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(host_dst, src, (size_t)count * row_bytes, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) { const_cast<pod_cache*>(c)->last_cuda = (int)e; return POD_ERR_CUDA; }
  return POD_OK;
}

int pod_cache_device_status(pod_cache* c) {
  if (!c) return POD_ERR_INVALID;
  if (c->dry) return POD_DRY_RUN;
  int32_t flag = 0;
  cudaError_t e = cudaSetDevice(c->cfg.device);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(&flag, c->arena + c->cv.off_err, 4, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && flag != 0) e = cudaMemset(c->arena + c->cv.off_err, 0, 4);
  if (e != cudaSuccess) return cuda_fail(c, e);
  return flag ? POD_ERR_DEVICE : POD_OK;
}

// Fault injection from the host (tests of the error path): sets the cache's error word as a kernel whose
// bounded wait gave up would.  No kernel is made to fail.
int pod_cache_inject_error(pod_cache* c) {
  if (!c) return POD_ERR_INVALID;
  if (c->dry) return POD_DRY_RUN;
  const int32_t one = 1;
  cudaError_t e = cudaSetDevice(c->cfg.device);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(c->arena + c->cv.off_err, &one, 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(c, e);
  return POD_OK;
}

// Launch trace: the next n_launches kernels of pod_decode_attn / pod_append_decode_attn each record the GPU
// timer at the start of their first CTA and at the end of their last one.
int pod_cache_set_trace(pod_cache* c, void* pairs_device, int n_launches) {
  if (!c || n_launches < 0 || (pairs_device == nullptr) != (n_launches == 0)) return POD_ERR_INVALID;
  if (((uintptr_t)pairs_device % 8) != 0) return POD_ERR_INVALID;
  if (c->dry) return POD_DRY_RUN;
  c->trace = nullptr; c->trace_cap = 0; c->trace_n = 0;
  if (pairs_device == nullptr) return POD_OK;
  std::vector<unsigned long long> init((size_t)2 * n_launches);
  for (int i = 0; i < n_launches; ++i) { init[2 * (size_t)i] = ~0ull; init[2 * (size_t)i + 1] = 0ull; }
  cudaError_t e = cudaSetDevice(c->cfg.device);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(pairs_device, init.data(), init.size() * 8, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(c, e);
  c->trace = static_cast<unsigned long long*>(pairs_device);
  c->trace_cap = n_launches;
  return POD_OK;
}

int pod_cache_trace_count(const pod_cache* c) { return c ? c->trace_n : POD_ERR_INVALID; }

// Test hook of the optimistic start: the next decode launch behaves as if every warp had found its early
// copy of q stale, so every head goes through the recomputation path.  Nothing on the GPU is made to fail.
int pod_cache_inject_stale_query(pod_cache* c) {
  if (!c) return POD_ERR_INVALID;
  c->inject_stale = true;
  return c->dry ? POD_DRY_RUN : POD_OK;
}

int pod_cache_last_cuda_error(const pod_cache* c) { return c ? c->last_cuda : (int)cudaErrorInvalidValue; }

int pod_cache_last_launch(const pod_cache* c, int32_t* split_tokens, int32_t* n_ctas, int32_t* n_kernels) {
  if (!c) return POD_ERR_INVALID;
  if (split_tokens) *split_tokens = c->last_split_tokens;
  if (n_ctas) *n_ctas = c->last_ctas;
  if (n_kernels) *n_kernels = c->last_kernels;
  return POD_OK;
}

}  // extern "C"
