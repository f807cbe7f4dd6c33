// Host side of the C ABI declared in include/kahan_sgd.h: validation, workspace layout,
// launches.  All arithmetic of the update runs in the kernels of kahan_sgd_kernels.cuh.
#include "kahan_sgd.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <utility>
#include <vector>

#include "kahan_sgd_kernels.cuh"
#include "kahan_sgd_momentum_kernels.cuh"
#include "kahan_sgd_adam_kernels.cuh"
#include "kahan_sgd_convert.cuh"

namespace {

using namespace ksgd;

std::atomic<uint64_t> g_launches{0};
thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
  std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return KSGD_ERR_CUDA;
}

#define KSGD_CUDA(call)                                   \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch a step kernel with programmatic stream serialization (see grid_dependency_wait in
// the kernels): its blocks may start their prologue while the preceding kernel of the stream
// finishes.
template <typename... KArgs, typename... Args>
cudaError_t launch_step_kernel(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                               cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Offsets of the workspace regions.  The regions up to stats_end are contiguous so that
// kahan_sgd_amax fetches them with one copy.
struct Layout {
  size_t phase, state, counters, error, stats_end;
  size_t info, grad_ptr, lr, exp_grad /* the optimizers' extra per-tensor word: mu */, chunks, total;
  long long n_chunks;
  int slab;                // records per phase slab (a slab is a multiple of 128 bytes)
};

// The same layout for every optimizer: phase word, three slabs of per-step records (the
// policy's State), counters, error word (all fetched by the read-out in one copy), then the
// tensor table (the policy's Info), the per-step arguments of long lists, the tile table.
Layout make_ring_layout(int32_t n, long long n_chunks, size_t state_bytes, size_t info_bytes, int n_counts) {
  Layout L{};
  L.n_chunks = n_chunks;
  L.slab = (int)(align_up(state_bytes * (size_t)n, 128) / state_bytes);
  size_t o = 0;
  L.phase = o;     o += 128;
  L.state = o;     o += state_bytes * 3 * L.slab;
  L.counters = o;  o += sizeof(unsigned long long) * n_counts * n;
  L.error = o;     o += 8;
  L.stats_end = o;
  o = align_up(o, 16);
  L.info = o;      o += info_bytes * n;
  o = align_up(o, 16);
  L.grad_ptr = o;  o += sizeof(const float*) * n;
  L.lr = o;        o += sizeof(float) * n;
  L.exp_grad = o;  o += sizeof(int) * n;
  o = align_up(o, 16);
  L.chunks = o;    o += sizeof(ChunkRef) * (size_t)n_chunks;
  L.total = align_up(o, 256);
  return L;
}

// What every init needs from the device, and the upload of the finished image.
struct DeviceFacts { int sms = 0, l2_bytes = 0; };
cudaError_t query_device(DeviceFacts& f) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&f.sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&f.l2_bytes, cudaDevAttrL2CacheSize, dev);
  return e;
}

// ---- tile tables ----------------------------------------------------------------------
// A list is cut into tiles of 2^lg elements of one tensor, lg by the tensor's format (the
// rules below).  Block b of a step takes tiles b, b + blocks, ...: when the tile count is not a
// multiple of the block count, the last round over the blocks has work for some of them only,
// and the step ends with a tile's whole latency (load, compute, drain) during which the memory
// system idles: on ResNet-50 shapes 19 of 148 blocks have a 22nd tile.  The builder therefore
// cuts the tiles of that last round into 2^k equal pieces each, k the largest for which the
// pieces still number at most one per block (and a piece has at least 512 elements), so
// that the last round is short and spread over the blocks.  A list with fewer tiles than
// blocks is one such round, which also puts more of the SMs to work on short lists.  The size
// query does not know the device, so a table reserves room for kTailReserve more entries than
// it has whole tiles.
constexpr long long kTailReserve = 1024;   // more than any device has SMs; the pieces are capped to it anyway

inline int lg_plain(const ksgd_tensor_desc& t, int chunk8) { return t.theta_bits == 8 && chunk8 != kChunk ? 14 : 13; }

// Steps on 8-bit gradients move so few bytes per parameter (5 for an 8/8 tensor, 9 for 16/16)
// that what a consumer does per tile, not per element, is a fifth or more of its instructions
// with the tiles above.  Lists long enough get a second tile table for those steps, with
// tiles twice as large as the largest of the first table: 4 * kChunk elements for 8-bit theta
// (12 of the ring's 28 pages with an 8-bit c and an 8-bit gradient; 2 * kChunk with a 16-bit
// c, which would take 16), 2 * kChunk for 16-bit theta (6 to 10 pages).
inline int lg_qgrad(const ksgd_tensor_desc& t) { return t.theta_bits == 8 && t.comp_bits <= 8 ? 15 : 14; }

template <class LgFn>
long long whole_tiles(const ksgd_tensor_desc* d, int32_t n, LgFn lg_of) {
  long long tiles = 0;
  for (int32_t i = 0; i < n; ++i) tiles += (d[i].numel + (1LL << lg_of(d[i])) - 1) >> lg_of(d[i]);
  return tiles;
}

// Writes the table to `out` (nullptr: counts only) and returns the number of entries; sms > 0
// cuts the last round into pieces as described above, sms == 0 leaves whole tiles.
// first_tile (optional) receives the first entry of every tensor, plus the total.
template <class LgFn>
long long build_tile_table(const ksgd_tensor_desc* d, int32_t n, LgFn lg_of, int sms, ChunkRef* out,
                           std::vector<long long>* first_tile) {
  const long long tiles = whole_tiles(d, n, lg_of);
  const long long r = sms > 0 ? tiles % sms : 0;
  int k = 0;
  if (r > 0) {
    const long long room = (long long)sms < kTailReserve ? (long long)sms : kTailReserve;
    while ((r << (k + 1)) <= room) ++k;
  }
  const long long cut_from = tiles - r;      // whole tiles from this one on are cut
  long long c = 0, whole = 0;
  if (first_tile) first_tile->clear();
  for (int32_t i = 0; i < n; ++i) {
    const int lg = lg_of(d[i]);
    const long long nc = (d[i].numel + (1LL << lg) - 1) >> lg;
    if (first_tile) first_tile->push_back(c);
    for (long long j = 0; j < nc; ++j, ++whole) {
      int kk = 0;
      if (whole >= cut_from) {
        kk = k < lg - kMinTileLog2 ? k : lg - kMinTileLog2;
        while (kk > 0 && ((j + 1) << kk) > (1LL << kTileIndexBits)) --kk;    // the index field holds 27 bits
      }
      for (long long q = 0; q < (1LL << kk); ++q) {
        const long long idx = (j << kk) + q;
        if ((idx << (lg - kk)) >= d[i].numel) break;      // the tensor's short last tile: nothing left
        if (out) out[c] = make_chunk_ref(i, idx, lg - kk);
        ++c;
      }
    }
  }
  if (first_tile) first_tile->push_back(c);
  return c;
}

// Tile size for tensors with 8-bit theta in the first table: the large one (2 * kChunk) if the
// list then still has kBigTileMinTiles tiles (about seven per block), so that short lists
// keep every block busy; with one 16-element vector per thread and tile, what a consumer does
// per tile (wait, descriptor, scans, arrive) is a third of its instructions.
int pick_chunk8(const ksgd_tensor_desc* d, int32_t n) {
  const long long tiles = whole_tiles(d, n, [](const ksgd_tensor_desc& t) { return lg_plain(t, 2 * kChunk); });
  return tiles >= kBigTileMinTiles ? 2 * kChunk : kChunk;
}

// Whole tiles of the table for steps on 8-bit gradients, or 0 for none (short lists keep the
// smaller tiles of the first table, with which every block has work).
long long whole_tiles_qgrad(const ksgd_tensor_desc* d, int32_t n) {
  const long long tiles = whole_tiles(d, n, lg_qgrad);
  return tiles >= kBigTileMinTiles ? tiles : 0;
}

// Room for the two tables of the plain optimizer (the second follows the first at
// qgrad_table_offset); reserve_tail: room for the pieces of the last round.
long long plain_table_capacity(const ksgd_tensor_desc* d, int32_t n, int chunk8, bool reserve_tail) {
  return whole_tiles(d, n, [chunk8](const ksgd_tensor_desc& t) { return lg_plain(t, chunk8); }) +
         (reserve_tail ? kTailReserve : 0);
}

// The tile table is the layout's last region.
Layout make_layout(const ksgd_tensor_desc* d, int32_t n, int chunk8, bool with_qgrad_table, bool reserve_tail) {
  const long long q = with_qgrad_table ? whole_tiles_qgrad(d, n) : 0;
  return make_ring_layout(n, plain_table_capacity(d, n, chunk8, reserve_tail) + (q ? q + kTailReserve : 0),
                          sizeof(TensorState), sizeof(TensorInfo), 3);
}

// Device-side view of a workspace at `b`.
void bind_workspace(Workspace& w, char* b, const Layout& L) {
  w.phase = reinterpret_cast<unsigned int*>(b + L.phase);
  w.state = reinterpret_cast<TensorState*>(b + L.state);
  w.slab = L.slab;
  w.counters = reinterpret_cast<unsigned long long*>(b + L.counters);
  w.error = reinterpret_cast<unsigned int*>(b + L.error);
  w.info = reinterpret_cast<TensorInfo*>(b + L.info);
  w.grad_ptr = reinterpret_cast<const float**>(b + L.grad_ptr);
  w.lr = reinterpret_cast<float*>(b + L.lr);
  w.exp_grad = reinterpret_cast<int*>(b + L.exp_grad);
  w.chunks = reinterpret_cast<ChunkRef*>(b + L.chunks);
}

// Host image of a fresh workspace (`img`: L.total zero bytes): phase 0; in the records the
// first step reads (slab 2) the exponents of the stored mantissas and, as overrides, the
// exponents the first step must write; zeroed scans and counters; tensor table; tile
// table (and, if asked for and the list is long enough for one, the table for steps on 8-bit
// gradients, at entry qgrad_offset of the table region).  sms: blocks of a step, for the
// pieces of the tables' last round (0: whole tiles only).
// first_tile (optional) receives the first tile of every tensor, plus the total.
struct TableCounts { long long plain = 0, qgrad = 0, qgrad_offset = 0; };
TableCounts write_initial_image(unsigned char* img, const Layout& L, const ksgd_tensor_desc* descs, int32_t n,
                                const int32_t* exp_comp, const int32_t* exp_comp_next, int chunk8,
                                bool with_qgrad_table, int sms, std::vector<long long>* first_tile) {
  TensorState* last = reinterpret_cast<TensorState*>(img + L.state) + 2 * (size_t)L.slab;
  TensorInfo* info = reinterpret_cast<TensorInfo*>(img + L.info);
  ChunkRef* chunks = reinterpret_cast<ChunkRef*>(img + L.chunks);
  for (int32_t i = 0; i < n; ++i) {
    const ksgd_tensor_desc& t = descs[i];
    last[i].exp_theta = t.exp_theta;
    last[i].ovr_theta = t.exp_theta_next + kOvrBias;
    if (exp_comp) {
      last[i].exp_comp = exp_comp[i];
      last[i].ovr_comp = (exp_comp_next ? exp_comp_next[i] : exp_comp[i]) + kOvrBias;
    }
    info[i].theta = t.theta;
    info[i].comp = t.comp;
    info[i].numel = t.numel;
    info[i].theta_bits = t.theta_bits;
    info[i].comp_bits = t.comp_bits;
    info[i].s = t.comp_bits ? t.comp_bits - 1 - t.overlap_k : 0;
    info[i].pad = 0;
  }
  TableCounts tc;
  tc.plain = build_tile_table(descs, n, [chunk8](const ksgd_tensor_desc& t) { return lg_plain(t, chunk8); }, sms,
                              chunks, first_tile);
  if (with_qgrad_table && whole_tiles_qgrad(descs, n)) {
    tc.qgrad_offset = plain_table_capacity(descs, n, chunk8, sms > 0);
    tc.qgrad = build_tile_table(descs, n, lg_qgrad, sms, chunks + tc.qgrad_offset, nullptr);
  }
  return tc;
}

// The caller's view of a copy of the stats region: scans and exponent of the last finished
// step, the exponent the coming step will write (its override if one is set, else what the
// scan implies: the rule the kernel itself applies), cumulative counters, error word.
int read_stats(const unsigned char* b, const Layout& L, const ksgd_tensor_desc* descs, int32_t n_tensors,
               int amax_mode, bool strict, uint32_t* amax_theta, uint32_t* amax_comp, int32_t* exp_theta_cur,
               int32_t* exp_theta_next, uint64_t* n_sat_theta, uint64_t* n_sat_comp, uint64_t* n_nonfinite,
               int32_t* exp_comp_cur, int32_t* exp_comp_next) {
  const size_t n = (size_t)n_tensors;
  unsigned int ph = 0;
  std::memcpy(&ph, b + L.phase, 4);
  if (ph > 2) return KSGD_ERR_DEVICE;
  const TensorState* last = reinterpret_cast<const TensorState*>(b + L.state) + ((ph + 2) % 3) * (size_t)L.slab;
  for (size_t i = 0; i < n; ++i) {
    const TensorState& r = last[i];
    const int e_next = r.ovr_theta ? r.ovr_theta - kOvrBias
                                   : next_exponent(r.amax[0], descs[i].theta_bits, r.exp_theta, amax_mode);
    if (amax_theta) amax_theta[i] = r.amax[0];
    if (amax_comp) amax_comp[i] = r.amax[1];
    if (exp_theta_cur) exp_theta_cur[i] = r.exp_theta;
    if (exp_theta_next) exp_theta_next[i] = e_next;
    if (strict) {
      if (exp_comp_cur) exp_comp_cur[i] = r.exp_comp;
      if (exp_comp_next)
        exp_comp_next[i] = r.ovr_comp ? r.ovr_comp - kOvrBias
                                      : next_exponent_acc(r.amax[1], descs[i].comp_bits, r.exp_comp, e_next, amax_mode);
    }
  }
  if (n_sat_theta) std::memcpy(n_sat_theta, b + L.counters, 8 * n);
  if (n_sat_comp) std::memcpy(n_sat_comp, b + L.counters + 8 * n, 8 * n);
  if (n_nonfinite) std::memcpy(n_nonfinite, b + L.counters + 16 * n, 8 * n);
  unsigned int dev_err = 0;
  std::memcpy(&dev_err, b + L.error, 4);
  if (dev_err != 0) return KSGD_ERR_DEVICE;
  return KSGD_OK;
}

int validate(const ksgd_tensor_desc* d, int32_t n) {
  if (!d) return KSGD_ERR_NULL;
  if (n <= 0) return KSGD_ERR_NUMEL;
  long long chunks = 0;
  for (int32_t i = 0; i < n; ++i) {
    const ksgd_tensor_desc& t = d[i];
    if (t.theta_bits != 8 && t.theta_bits != 16) return KSGD_ERR_BITS;
    if (t.comp_bits != 0 && t.comp_bits != 8 && t.comp_bits != 16) return KSGD_ERR_BITS;
    if (!t.theta) return KSGD_ERR_NULL;
    if ((t.comp_bits != 0) != (t.comp != nullptr)) return KSGD_ERR_NULL;
    if (t.comp_bits != 0 && (t.overlap_k < 0 || t.overlap_k > t.comp_bits - 1)) return KSGD_ERR_OVERLAP;
    if (t.numel <= 0) return KSGD_ERR_NUMEL;
    if (t.exp_theta < kExpMin || t.exp_theta > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (t.exp_theta_next < kExpMin || t.exp_theta_next > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (std::abs(t.exp_theta_next - t.exp_theta) > kMaxDelta) return KSGD_ERR_EXP_RANGE;
    if (reinterpret_cast<uintptr_t>(t.theta) % 16 || reinterpret_cast<uintptr_t>(t.comp) % 16)
      return KSGD_ERR_ALIGN;
    if (t.numel > (1LL << (kTileIndexBits + kChunkLog2))) return KSGD_ERR_NUMEL;   // the tile table's index field
    chunks += (t.numel + kChunk - 1) / kChunk;
    if (chunks > 0x7fffffffLL - 2 * kTailReserve) return KSGD_ERR_NUMEL;
  }
  return KSGD_OK;
}

}  // namespace

struct ksgd_handle {
  std::vector<ksgd_tensor_desc> descs;
  Layout layout;
  StepParams params;
  char* ws_base;
  cudaStream_t stream;
  int32_t n;
  int grid;
  int sms;
  std::vector<unsigned char> stats_host;   // staging for kahan_sgd_amax
  std::vector<long long> first_tile;       // [n+1] first tile of every tensor
  long long tiles_qgrad = 0;               // entries of the tile table for steps on 8-bit gradients, 0: those
                                           // steps use the first table too
  long long qgrad_offset = 0;              // where that table starts in the table region (in entries)
  bool strict = false;                     // strict Algorithm 1: compensation with its own exponent
  // kahan_sgd_step_host: copy streams and events, created on first use
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  std::vector<cudaEvent_t> events;
};

extern "C" {

size_t kahan_sgd_workspace_bytes(const ksgd_tensor_desc* descs, int32_t n_tensors) {
  if (validate(descs, n_tensors) != KSGD_OK) return 0;
  return make_layout(descs, n_tensors, pick_chunk8(descs, n_tensors), true, true).total;
}

size_t kahan_sgd_workspace_error_offset(const ksgd_tensor_desc* descs, int32_t n_tensors) {
  if (validate(descs, n_tensors) != KSGD_OK) return (size_t)-1;
  return make_layout(descs, n_tensors, pick_chunk8(descs, n_tensors), true, true).error;
}

int64_t kahan_sgd_tile_table(const ksgd_tensor_desc* descs, int32_t n_tensors, int32_t sms, int32_t which,
                             int64_t* out, int64_t capacity) {
  const int v = validate(descs, n_tensors);
  if (v != KSGD_OK) return v;
  if (sms < 0 || (which != 0 && which != 1) || capacity < 0) return KSGD_ERR_MODE;
  const int chunk8 = pick_chunk8(descs, n_tensors);
  if (which == 1 && whole_tiles_qgrad(descs, n_tensors) == 0) return 0;
  auto lg_first = [chunk8](const ksgd_tensor_desc& t) { return lg_plain(t, chunk8); };
  const long long count = which == 0 ? build_tile_table(descs, n_tensors, lg_first, sms, nullptr, nullptr)
                                     : build_tile_table(descs, n_tensors, lg_qgrad, sms, nullptr, nullptr);
  if (!out) return count;
  std::vector<ChunkRef> table((size_t)count);
  if (which == 0) build_tile_table(descs, n_tensors, lg_first, sms, table.data(), nullptr);
  else build_tile_table(descs, n_tensors, lg_qgrad, sms, table.data(), nullptr);
  for (long long i = 0; i < count && i < capacity; ++i) {
    const ChunkRef& c = table[(size_t)i];
    const long long first = chunk_index(c) << chunk_log2(c);
    const long long left = descs[c.tensor].numel - first;
    out[3 * i] = c.tensor;
    out[3 * i + 1] = first;
    out[3 * i + 2] = left < (1LL << chunk_log2(c)) ? left : (1LL << chunk_log2(c));
  }
  return count;
}

}  // extern "C"

namespace {

bool strict_window_ok(int e, int ec) { return e - ec >= -kStrictAbove && e - ec <= kStrictBelow; }

// first_step: also check the exponents the first step writes (init).  The workspace size
// does not depend on them, and c's stored exponent need not lie in the window of theta's
// *next* exponent (a state taken from a running handle has it in the window of the stored
// one only), so the size query checks the stored pair alone.
int validate_strict(const ksgd_tensor_desc* d, const int32_t* ec, const int32_t* ec_next, int32_t n,
                    bool first_step) {
  if (!ec) return KSGD_ERR_NULL;
  for (int32_t i = 0; i < n; ++i) {
    if (d[i].comp_bits == 0) return KSGD_ERR_BITS;          // the accumulator is the point of this mode
    if (ec[i] < kExpMin || ec[i] > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (!strict_window_ok(d[i].exp_theta, ec[i])) return KSGD_ERR_EXP_RANGE;
    if (!first_step) continue;
    const int32_t nx = ec_next ? ec_next[i] : ec[i];
    if (nx < kExpMin || nx > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (!strict_window_ok(d[i].exp_theta_next, nx)) return KSGD_ERR_EXP_RANGE;
    // the device never moves c's exponent by more than 2 * kMaxDelta in one step (its own
    // fit plus theta's move); a larger first-step change would shift past 64 bits
    if (std::abs(nx - ec[i]) > 2 * kMaxDelta) return KSGD_ERR_EXP_RANGE;
  }
  return KSGD_OK;
}

int init_common(ksgd_handle** out, const ksgd_tensor_desc* descs, const int32_t* exp_comp,
                const int32_t* exp_comp_next, bool strict, int32_t n_tensors, ksgd_exp_mode mode,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return KSGD_ERR_NULL;
  *out = nullptr;
  const int v = validate(descs, n_tensors);
  if (v != KSGD_OK) return v;
  if (strict) {
    const int vs = validate_strict(descs, exp_comp, exp_comp_next, n_tensors, true);
    if (vs != KSGD_OK) return vs;
  }
  if (mode != KSGD_EXP_FIXED && mode != KSGD_EXP_AMAX) return KSGD_ERR_MODE;
  if (!workspace) return KSGD_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(workspace) % 256) return KSGD_ERR_ALIGN;
  const int chunk8 = pick_chunk8(descs, n_tensors);
  const Layout L = make_layout(descs, n_tensors, chunk8, true, true);
  if (workspace_bytes < L.total) return KSGD_ERR_WORKSPACE;
  DeviceFacts dev_facts;      // the tile tables depend on the number of blocks a step has
  {
    const cudaError_t eq = query_device(dev_facts);
    if (eq != cudaSuccess) return cuda_fail(eq, "device query");
  }

  ksgd_handle* h = new (std::nothrow) ksgd_handle();
  if (!h) return KSGD_ERR_NULL;
  h->descs.assign(descs, descs + n_tensors);
  h->layout = L;
  h->n = n_tensors;
  h->ws_base = static_cast<char*>(workspace);
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->stats_host.resize(L.stats_end);
  h->strict = strict;

  std::vector<unsigned char> img(L.total, 0);
  const TableCounts tc = write_initial_image(img.data(), L, descs, n_tensors, strict ? exp_comp : nullptr,
                                             exp_comp_next, chunk8, true, dev_facts.sms, &h->first_tile);
  const long long tiles = tc.plain;
  h->tiles_qgrad = tc.qgrad;
  h->qgrad_offset = tc.qgrad_offset;
  char* b = h->ws_base;
  bind_workspace(h->params.ws, b, L);
  h->params.n_tensors = n_tensors;
  h->params.n_chunks = (int)tiles;
  h->params.amax_mode = mode == KSGD_EXP_AMAX ? 1 : 0;
  h->params.inline_args = n_tensors <= kInlineArgs ? 1 : 0;
  h->params.tile_begin = 0;
  h->params.tile_count = (int)tiles;
  h->params.tensor_begin = 0;
  h->params.tensor_count = n_tensors;
  h->params.advance = 1;
  h->params.exp_grad_dev = nullptr;

  // Persistent grid: one block per SM (fewer if the list has fewer tiles).
  const int sms = dev_facts.sms, l2_bytes = dev_facts.l2_bytes;
  cudaError_t e = cudaFuncSetAttribute(ksgd_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(ksgd_step_qgrad_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(ksgd_step_qgrad_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e == cudaSuccess && strict)
    e = cudaFuncSetAttribute(ksgd_strict_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e == cudaSuccess && strict)
    e = cudaFuncSetAttribute(ksgd_strict_step_qgrad_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e == cudaSuccess && strict)
    e = cudaFuncSetAttribute(ksgd_strict_step_qgrad_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kSharedBytes);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "device query");
  }
  h->grid = (int)(tiles < (long long)sms ? tiles : (long long)sms);
  h->sms = sms;
  // theta and c of the whole list against the L2 size: if the state fits (with room for
  // the gradients streaming through), gradient loads are marked evict-first
  double state_bytes = 0.0;
  for (int32_t i = 0; i < n_tensors; ++i)
    state_bytes += (double)descs[i].numel * ((descs[i].theta_bits + descs[i].comp_bits) / 8);
  h->params.state_in_l2 = state_bytes <= 0.8 * (double)l2_bytes ? 1 : 0;

  e = cudaMemcpyAsync(b, img.data(), L.total, cudaMemcpyHostToDevice, h->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "workspace upload");
  }
  *out = h;
  return KSGD_OK;
}

}  // namespace

extern "C" {

int kahan_sgd_init(ksgd_handle** out, const ksgd_tensor_desc* descs, int32_t n_tensors,
                   ksgd_exp_mode mode, void* workspace, size_t workspace_bytes,
                   void* cuda_stream) {
  return init_common(out, descs, nullptr, nullptr, false, n_tensors, mode, workspace, workspace_bytes,
                     cuda_stream);
}

size_t kahan_sgd_strict_workspace_bytes(const ksgd_tensor_desc* descs, const int32_t* exp_comp,
                                        int32_t n_tensors) {
  if (validate(descs, n_tensors) != KSGD_OK) return 0;
  if (validate_strict(descs, exp_comp, nullptr, n_tensors, false) != KSGD_OK) return 0;
  return make_layout(descs, n_tensors, pick_chunk8(descs, n_tensors), true, true).total;
}

int kahan_sgd_strict_init(ksgd_handle** out, const ksgd_tensor_desc* descs, const int32_t* exp_comp,
                          const int32_t* exp_comp_next, int32_t n_tensors, ksgd_exp_mode mode,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return KSGD_ERR_NULL;
  *out = nullptr;
  if (!exp_comp) return KSGD_ERR_NULL;
  return init_common(out, descs, exp_comp, exp_comp_next, true, n_tensors, mode, workspace, workspace_bytes,
                     cuda_stream);
}

static int fetch_stats(ksgd_handle* h) {
  KSGD_CUDA(cudaMemcpyAsync(h->stats_host.data(), h->ws_base, h->layout.stats_end, cudaMemcpyDeviceToHost,
                            h->stream));
  KSGD_CUDA(cudaStreamSynchronize(h->stream));
  return KSGD_OK;
}

int kahan_sgd_strict_exponents(ksgd_handle* h, int32_t* exp_comp_cur, int32_t* exp_comp_next) {
  if (!h) return KSGD_ERR_NULL;
  if (!h->strict) return KSGD_ERR_MODE;
  const int r = fetch_stats(h);
  if (r != KSGD_OK) return r;
  const int rs = read_stats(h->stats_host.data(), h->layout, h->descs.data(), h->n, h->params.amax_mode, true,
                            nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, exp_comp_cur,
                            exp_comp_next);
  return rs == KSGD_ERR_DEVICE ? KSGD_OK : rs;    // the device error word is kahan_sgd_amax's to report
}

static int check_step_args(const ksgd_handle* h, const float* const* grads, const float* lrs) {
  if (!h || !grads || !lrs) return KSGD_ERR_NULL;
  for (int32_t i = 0; i < h->n; ++i) {
    if (!grads[i]) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(grads[i]) % 16) return KSGD_ERR_ALIGN;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
  }
  return KSGD_OK;
}

// Launch the step on tensors [t0, t1) (their tiles are contiguous in the table).
static int launch_step_range(ksgd_handle* h, const InlineArgs* ia, int32_t t0, int32_t t1) {
  StepParams p = h->params;
  p.advance = t1 == h->n ? 1 : 0;     // the groups of one step share its phase; the last one moves it on
  p.tile_begin = (int)h->first_tile[t0];
  p.tile_count = (int)(h->first_tile[t1] - h->first_tile[t0]);
  p.tensor_begin = t0;
  p.tensor_count = t1 - t0;
  const int grid = p.tile_count < h->sms ? p.tile_count : h->sms;
  if (h->strict) ksgd_strict_step_kernel<<<(unsigned)grid, kBlockThreads, kSharedBytes, h->stream>>>(p, *ia);
  else ksgd_step_kernel<<<(unsigned)grid, kBlockThreads, kSharedBytes, h->stream>>>(p, *ia);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

static int launch_step(ksgd_handle* h, const float* const* grads, const float* lrs) {
  static InlineArgs none{};   // parameter placeholder for long lists
  const InlineArgs* ia = &none;
  InlineArgs inl;
  if (h->params.inline_args) {
    for (int32_t i = 0; i < h->n; ++i) { inl.grads[i] = grads[i]; inl.lrs[i] = lrs[i]; }
    for (int32_t i = h->n; i < kInlineArgs; ++i) { inl.grads[i] = nullptr; inl.lrs[i] = 0.0f; }
    ia = &inl;
  } else {
    UploadBatch* ub = new (std::nothrow) UploadBatch;
    if (!ub) return KSGD_ERR_NULL;
    for (int32_t first = 0; first < h->n; first += kUploadBatch) {
      const int count = h->n - first < kUploadBatch ? h->n - first : kUploadBatch;
      for (int i = 0; i < count; ++i) { ub->grads[i] = grads[first + i]; ub->lrs[i] = lrs[first + i]; }
      ksgd_upload_args_kernel<<<1, 256, 0, h->stream>>>(*ub, first, count, h->params.ws.grad_ptr,
                                                        h->params.ws.lr);
      g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    delete ub;
    KSGD_CUDA(cudaGetLastError());
  }
  if (h->strict)
    KSGD_CUDA(launch_step_kernel(ksgd_strict_step_kernel, (unsigned)h->grid, kBlockThreads, kSharedBytes, h->stream,
                                 h->params, *ia));
  else
    KSGD_CUDA(launch_step_kernel(ksgd_step_kernel, (unsigned)h->grid, kBlockThreads, kSharedBytes, h->stream,
                                 h->params, *ia));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

// exp_grad: host array (copied into the launch), or nullptr with exp_grad_dev: a device array
// the kernel reads the exponents from.
static int step_qgrad_common(ksgd_handle* h, const void* const* grads, int32_t grad_bits, const int32_t* exp_grad,
                             const int32_t* exp_grad_dev, const float* lrs) {
  if (!h || !grads || (!exp_grad && !exp_grad_dev) || !lrs) return KSGD_ERR_NULL;
  if (grad_bits != 8 && grad_bits != 16) return KSGD_ERR_BITS;
  if (reinterpret_cast<uintptr_t>(exp_grad_dev) % 4) return KSGD_ERR_ALIGN;
  for (int32_t i = 0; i < h->n; ++i) {
    if (!grads[i]) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(grads[i]) % 16) return KSGD_ERR_ALIGN;
    if (exp_grad && (exp_grad[i] < kExpMin || exp_grad[i] > kExpMax)) return KSGD_ERR_EXP_RANGE;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
  }
  QGradArgs args{};
  if (h->params.inline_args) {
    for (int32_t i = 0; i < h->n; ++i) {
      args.grads[i] = grads[i];
      args.lrs[i] = lrs[i];
      args.exp_grad[i] = exp_grad ? (signed char)exp_grad[i] : 0;
    }
  } else {
    UploadBatch* ub = new (std::nothrow) UploadBatch;
    ExponentBatch* eb = new (std::nothrow) ExponentBatch;
    if (!ub || !eb) { delete ub; delete eb; return KSGD_ERR_NULL; }
    for (int32_t first = 0; first < h->n; first += kUploadBatch) {
      const int count = h->n - first < kUploadBatch ? h->n - first : kUploadBatch;
      for (int i = 0; i < count; ++i) {
        ub->grads[i] = static_cast<const float*>(grads[first + i]);   // only the address travels
        ub->lrs[i] = lrs[first + i];
        eb->exp_next[i] = exp_grad ? exp_grad[first + i] : 0;
      }
      ksgd_upload_args_kernel<<<1, 256, 0, h->stream>>>(*ub, first, count, h->params.ws.grad_ptr,
                                                        h->params.ws.lr);
      g_launches.fetch_add(1, std::memory_order_relaxed);
      if (exp_grad) {
        ksgd_upload_ints_kernel<<<1, 256, 0, h->stream>>>(*eb, first, count, h->params.ws.exp_grad);
        g_launches.fetch_add(1, std::memory_order_relaxed);
      }
    }
    delete ub;
    delete eb;
    KSGD_CUDA(cudaGetLastError());
  }
  StepParams p = h->params;
  p.exp_grad_dev = exp_grad_dev;
  unsigned grid = (unsigned)h->grid;
  if (grad_bits == 8 && h->tiles_qgrad) {       // the table of larger tiles, behind the first one
    p.ws.chunks += h->qgrad_offset;
    p.n_chunks = p.tile_count = (int)h->tiles_qgrad;
    grid = (unsigned)(h->tiles_qgrad < (long long)h->sms ? h->tiles_qgrad : (long long)h->sms);
  }
  auto kernel = h->strict ? (grad_bits == 8 ? ksgd_strict_step_qgrad_kernel<8> : ksgd_strict_step_qgrad_kernel<16>)
                          : (grad_bits == 8 ? ksgd_step_qgrad_kernel<8> : ksgd_step_qgrad_kernel<16>);
  KSGD_CUDA(launch_step_kernel(kernel, grid, kBlockThreads, kSharedBytes, h->stream, p, args));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

int kahan_sgd_step_qgrad(ksgd_handle* h, const void* const* grads, int32_t grad_bits, const int32_t* exp_grad,
                         const float* lrs) {
  if (!exp_grad) return KSGD_ERR_NULL;
  return step_qgrad_common(h, grads, grad_bits, exp_grad, nullptr, lrs);
}

int kahan_sgd_step_qgrad_dev(ksgd_handle* h, const void* const* grads, int32_t grad_bits,
                             const int32_t* exp_grad_dev, const float* lrs) {
  if (!exp_grad_dev) return KSGD_ERR_NULL;
  return step_qgrad_common(h, grads, grad_bits, nullptr, exp_grad_dev, lrs);
}

int kahan_sgd_step(ksgd_handle* h, const float* const* grads, const float* lrs) {
  const int v = check_step_args(h, grads, lrs);
  if (v != KSGD_OK) return v;
  return launch_step(h, grads, lrs);
}

int kahan_sgd_step_host(ksgd_handle* h, void* const* theta_host, void* const* comp_host,
                        const float* const* grads_host, const float* lrs,
                        void* grad_staging, size_t grad_staging_bytes) {
  if (!h || !theta_host || !comp_host || !grads_host || !lrs || !grad_staging) return KSGD_ERR_NULL;
  if (h->strict) return KSGD_ERR_MODE;
  if (reinterpret_cast<uintptr_t>(grad_staging) % 16) return KSGD_ERR_ALIGN;
  size_t need = 0;
  for (int32_t i = 0; i < h->n; ++i) need += align_up((size_t)h->descs[i].numel, 4) * sizeof(float);
  if (grad_staging_bytes < need) return KSGD_ERR_WORKSPACE;
  std::vector<const float*> dev_grads(h->n);
  size_t off = 0;
  for (int32_t i = 0; i < h->n; ++i) {
    const ksgd_tensor_desc& t = h->descs[i];
    if (!theta_host[i] || !grads_host[i] || (t.comp_bits && !comp_host[i])) return KSGD_ERR_NULL;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
    dev_grads[i] = reinterpret_cast<const float*>(static_cast<char*>(grad_staging) + off);
    off += align_up((size_t)t.numel, 4) * sizeof(float);
  }

  // Groups of neighbouring tensors of about 256 MB each travel as a pipeline: while one
  // group is being updated, the next one is on its way to the device and the previous
  // one on its way back (the two copy directions run at the same time).
  constexpr size_t kGroupBytes = 256u << 20;
  std::vector<int32_t> group_start{0};
  size_t acc = 0;
  for (int32_t i = 0; i < h->n; ++i) {
    const ksgd_tensor_desc& t = h->descs[i];
    const size_t b = (size_t)t.numel * ((t.theta_bits + t.comp_bits) / 8 + 4);
    if (acc > 0 && acc + b > kGroupBytes) { group_start.push_back(i); acc = 0; }
    acc += b;
  }
  group_start.push_back(h->n);
  const size_t n_groups = group_start.size() - 1;

  if (!h->h2d_stream) KSGD_CUDA(cudaStreamCreateWithFlags(&h->h2d_stream, cudaStreamNonBlocking));
  if (!h->d2h_stream) KSGD_CUDA(cudaStreamCreateWithFlags(&h->d2h_stream, cudaStreamNonBlocking));
  while (h->events.size() < 2 * n_groups + 1) {
    cudaEvent_t ev;
    KSGD_CUDA(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    h->events.push_back(ev);
  }

  // per-step arguments (device gradient addresses, learning rates)
  static InlineArgs none{};
  const InlineArgs* ia = &none;
  InlineArgs inl;
  if (h->params.inline_args) {
    for (int32_t i = 0; i < h->n; ++i) { inl.grads[i] = dev_grads[i]; inl.lrs[i] = lrs[i]; }
    for (int32_t i = h->n; i < kInlineArgs; ++i) { inl.grads[i] = nullptr; inl.lrs[i] = 0.0f; }
    ia = &inl;
  } else {
    UploadBatch* ub = new (std::nothrow) UploadBatch;
    if (!ub) return KSGD_ERR_NULL;
    for (int32_t first = 0; first < h->n; first += kUploadBatch) {
      const int count = h->n - first < kUploadBatch ? h->n - first : kUploadBatch;
      for (int i = 0; i < count; ++i) { ub->grads[i] = dev_grads[first + i]; ub->lrs[i] = lrs[first + i]; }
      ksgd_upload_args_kernel<<<1, 256, 0, h->stream>>>(*ub, first, count, h->params.ws.grad_ptr,
                                                        h->params.ws.lr);
      g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    delete ub;
    KSGD_CUDA(cudaGetLastError());
  }

  // Neighbouring tensors whose host and device ranges both continue where the previous
  // one ended travel as one copy.
  struct Span { char* dst; const char* src; size_t bytes; };
  auto flush = [&](std::vector<Span>& spans, cudaMemcpyKind kind, cudaStream_t st) -> cudaError_t {
    size_t i = 0;
    while (i < spans.size()) {
      Span sp = spans[i++];
      while (i < spans.size() && spans[i].dst == sp.dst + sp.bytes && spans[i].src == sp.src + sp.bytes)
        sp.bytes += spans[i++].bytes;
      cudaError_t e = cudaMemcpyAsync(sp.dst, sp.src, sp.bytes, kind, st);
      if (e != cudaSuccess) return e;
    }
    spans.clear();
    return cudaSuccess;
  };

  // the copies must not overtake work already queued on the caller's stream
  cudaEvent_t ev_start = h->events[2 * n_groups];
  KSGD_CUDA(cudaEventRecord(ev_start, h->stream));
  KSGD_CUDA(cudaStreamWaitEvent(h->h2d_stream, ev_start, 0));

  std::vector<Span> spans;
  for (size_t g = 0; g < n_groups; ++g) {
    const int32_t t0 = group_start[g], t1 = group_start[g + 1];
    for (int32_t i = t0; i < t1; ++i) {
      const ksgd_tensor_desc& t = h->descs[i];
      spans.push_back({static_cast<char*>(t.theta), static_cast<const char*>(theta_host[i]),
                       (size_t)t.numel * (t.theta_bits / 8)});
    }
    KSGD_CUDA(flush(spans, cudaMemcpyHostToDevice, h->h2d_stream));
    for (int32_t i = t0; i < t1; ++i) {
      const ksgd_tensor_desc& t = h->descs[i];
      if (t.comp_bits)
        spans.push_back({static_cast<char*>(t.comp), static_cast<const char*>(comp_host[i]),
                         (size_t)t.numel * (t.comp_bits / 8)});
    }
    KSGD_CUDA(flush(spans, cudaMemcpyHostToDevice, h->h2d_stream));
    for (int32_t i = t0; i < t1; ++i)
      spans.push_back({const_cast<char*>(reinterpret_cast<const char*>(dev_grads[i])),
                       reinterpret_cast<const char*>(grads_host[i]), (size_t)h->descs[i].numel * sizeof(float)});
    KSGD_CUDA(flush(spans, cudaMemcpyHostToDevice, h->h2d_stream));
    KSGD_CUDA(cudaEventRecord(h->events[2 * g], h->h2d_stream));

    KSGD_CUDA(cudaStreamWaitEvent(h->stream, h->events[2 * g], 0));
    const int r = launch_step_range(h, ia, t0, t1);
    if (r != KSGD_OK) return r;
    KSGD_CUDA(cudaEventRecord(h->events[2 * g + 1], h->stream));

    KSGD_CUDA(cudaStreamWaitEvent(h->d2h_stream, h->events[2 * g + 1], 0));
    for (int32_t i = t0; i < t1; ++i) {
      const ksgd_tensor_desc& t = h->descs[i];
      spans.push_back({static_cast<char*>(theta_host[i]), static_cast<const char*>(t.theta),
                       (size_t)t.numel * (t.theta_bits / 8)});
    }
    KSGD_CUDA(flush(spans, cudaMemcpyDeviceToHost, h->d2h_stream));
    for (int32_t i = t0; i < t1; ++i) {
      const ksgd_tensor_desc& t = h->descs[i];
      if (t.comp_bits)
        spans.push_back({static_cast<char*>(comp_host[i]), static_cast<const char*>(t.comp),
                         (size_t)t.numel * (t.comp_bits / 8)});
    }
    KSGD_CUDA(flush(spans, cudaMemcpyDeviceToHost, h->d2h_stream));
  }
  KSGD_CUDA(cudaStreamSynchronize(h->d2h_stream));
  KSGD_CUDA(cudaStreamSynchronize(h->stream));
  return KSGD_OK;
}

int kahan_sgd_amax(ksgd_handle* h, uint32_t* amax_theta, uint32_t* amax_comp,
                   int32_t* exp_theta_cur, int32_t* exp_theta_next, uint64_t* n_sat_theta,
                   uint64_t* n_sat_comp, uint64_t* n_nonfinite) {
  if (!h) return KSGD_ERR_NULL;
  const int r = fetch_stats(h);
  if (r != KSGD_OK) return r;
  return read_stats(h->stats_host.data(), h->layout, h->descs.data(), h->n, h->params.amax_mode, h->strict,
                    amax_theta, amax_comp, exp_theta_cur, exp_theta_next, n_sat_theta, n_sat_comp, n_nonfinite,
                    nullptr, nullptr);
}

int kahan_sgd_set_exponents(ksgd_handle* h, const int32_t* exp_theta_next) {
  if (!h || !exp_theta_next) return KSGD_ERR_NULL;
  if (h->strict) return KSGD_ERR_MODE;     // the compensation's window hangs on theta's exponent
  for (int32_t i = 0; i < h->n; ++i)
    if (exp_theta_next[i] < kExpMin || exp_theta_next[i] > kExpMax) return KSGD_ERR_EXP_RANGE;
  ExponentBatch* eb = new (std::nothrow) ExponentBatch;
  if (!eb) return KSGD_ERR_NULL;
  for (int32_t first = 0; first < h->n; first += kUploadBatch) {
    const int count = h->n - first < kUploadBatch ? h->n - first : kUploadBatch;
    for (int i = 0; i < count; ++i) eb->exp_next[i] = exp_theta_next[first + i];
    ksgd_set_exponents_kernel<<<1, 256, 0, h->stream>>>(*eb, first, count, h->layout.slab, h->params.ws.phase,
                                                        h->params.ws.state);
    g_launches.fetch_add(1, std::memory_order_relaxed);
  }
  delete eb;
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

int kahan_sgd_destroy(ksgd_handle* h) {
  if (!h) return KSGD_ERR_NULL;
  const cudaError_t e = cudaStreamSynchronize(h->stream);
  for (cudaEvent_t ev : h->events) cudaEventDestroy(ev);
  if (h->h2d_stream) cudaStreamDestroy(h->h2d_stream);
  if (h->d2h_stream) cudaStreamDestroy(h->d2h_stream);
  delete h;
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  return KSGD_OK;
}

// ----------------------------------------------------------------------------------------
// One step without any device allocation by anybody: the scratch that kahan_sgd_init
// otherwise lays out in a caller-provided workspace lives in a fixed array inside this
// library's device image.

static __device__ __align__(256) unsigned char g_static_scratch[KSGD_STATIC_SCRATCH_BYTES];

namespace {
struct StaticDevice {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
  int sms = 0;
  int l2_bytes = 0;
};
constexpr int kMaxDevices = 64;
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mutex;
}  // namespace

int kahan_sgd_step_static(const ksgd_tensor_desc* descs, int32_t n_tensors, ksgd_exp_mode mode,
                          const float* const* grads, const float* lrs, uint32_t* amax_theta,
                          uint32_t* amax_comp, int32_t* exp_theta_cur, int32_t* exp_theta_next,
                          uint64_t* n_sat_theta, uint64_t* n_sat_comp, uint64_t* n_nonfinite,
                          void* cuda_stream) {
  const int v = validate(descs, n_tensors);
  if (v != KSGD_OK) return v;
  if (mode != KSGD_EXP_FIXED && mode != KSGD_EXP_AMAX) return KSGD_ERR_MODE;
  if (!grads || !lrs) return KSGD_ERR_NULL;
  if (n_tensors > KSGD_STATIC_MAX_TENSORS) return KSGD_ERR_WORKSPACE;
  const Layout L = make_layout(descs, n_tensors, kChunk, false, false);
  if (L.total > (size_t)KSGD_STATIC_SCRATCH_BYTES) return KSGD_ERR_WORKSPACE;
  for (int32_t i = 0; i < n_tensors; ++i) {
    if (!grads[i]) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(grads[i]) % 16) return KSGD_ERR_ALIGN;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
  }

  // Once per device, with that device current: the array's name is only a host-side
  // stand-in here, the address a kernel can use has to be asked for.
  int dev = 0;
  KSGD_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return KSGD_ERR_WORKSPACE;
  StaticDevice sd;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice& slot = g_static_dev[dev];
    if (!slot.ready) {
      void* ptr = nullptr;
      KSGD_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
      KSGD_CUDA(cudaDeviceGetAttribute(&slot.sms, cudaDevAttrMultiProcessorCount, dev));
      KSGD_CUDA(cudaDeviceGetAttribute(&slot.l2_bytes, cudaDevAttrL2CacheSize, dev));
      KSGD_CUDA(cudaFuncSetAttribute(ksgd_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kSharedBytes));
      slot.scratch = static_cast<unsigned char*>(ptr);
      slot.ready = true;
    }
    sd = slot;
  }

  // Host image of the scratch, every byte of it: whatever the previous call left in the
  // array (scans, counters, phase and tickets) is overwritten.
  std::vector<unsigned char> img(L.total, 0);
  write_initial_image(img.data(), L, descs, n_tensors, nullptr, nullptr, kChunk, false, 0, nullptr);   // whole tiles of kChunk
  double state_bytes = 0.0;
  for (int32_t i = 0; i < n_tensors; ++i)
    state_bytes += (double)descs[i].numel * ((descs[i].theta_bits + descs[i].comp_bits) / 8);
  const int grid = (int)(L.n_chunks < (long long)sd.sms ? L.n_chunks : (long long)sd.sms);

  StepParams params;
  unsigned char* b = sd.scratch;
  bind_workspace(params.ws, reinterpret_cast<char*>(b), L);
  params.n_tensors = n_tensors;
  params.n_chunks = (int)L.n_chunks;
  params.amax_mode = mode == KSGD_EXP_AMAX ? 1 : 0;
  params.inline_args = 1;
  params.tile_begin = 0;
  params.tile_count = (int)L.n_chunks;
  params.tensor_begin = 0;
  params.tensor_count = n_tensors;
  params.state_in_l2 = state_bytes <= 0.8 * (double)sd.l2_bytes ? 1 : 0;
  params.advance = 1;
  params.exp_grad_dev = nullptr;

  InlineArgs inl;
  for (int32_t i = 0; i < n_tensors; ++i) { inl.grads[i] = grads[i]; inl.lrs[i] = lrs[i]; }
  for (int32_t i = n_tensors; i < kInlineArgs; ++i) { inl.grads[i] = nullptr; inl.lrs[i] = 0.0f; }

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  KSGD_CUDA(cudaMemcpyAsync(b, img.data(), L.total, cudaMemcpyHostToDevice, stream));
  ksgd_step_kernel<<<(unsigned)grid, kBlockThreads, kSharedBytes, stream>>>(params, inl);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  KSGD_CUDA(cudaMemcpyAsync(img.data(), b, L.stats_end, cudaMemcpyDeviceToHost, stream));
  KSGD_CUDA(cudaStreamSynchronize(stream));

  return read_stats(img.data(), L, descs, n_tensors, params.amax_mode, false, amax_theta, amax_comp, exp_theta_cur,
                    exp_theta_next, n_sat_theta, n_sat_comp, n_nonfinite, nullptr, nullptr);
}

// ----------------------------------------------------------------------------------------
// Momentum optimizer with the lazy update.

namespace {

// Per-step arguments of a list longer than kInlineArgs: batches passed by value to the
// upload kernel, which writes them into the workspace (second pass for the momentum
// coefficients, which travel in the batch's lrs field).
int upload_long_list(cudaStream_t stream, int32_t n, const float* const* grads, const float* lrs,
                     const float* mus, const float** grad_ptr, float* lr, float* mu) {
  UploadBatch* ub = new (std::nothrow) UploadBatch;
  if (!ub) return KSGD_ERR_NULL;
  for (int32_t first = 0; first < n; first += kUploadBatch) {
    const int count = n - first < kUploadBatch ? n - first : kUploadBatch;
    for (int i = 0; i < count; ++i) { ub->grads[i] = grads[first + i]; ub->lrs[i] = lrs[first + i]; }
    ksgd_upload_args_kernel<<<1, 256, 0, stream>>>(*ub, first, count, grad_ptr, lr);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (mus) {
      for (int i = 0; i < count; ++i) ub->lrs[i] = mus[first + i];
      ksgd_upload_args_kernel<<<1, 256, 0, stream>>>(*ub, first, count, grad_ptr, mu);
      g_launches.fetch_add(1, std::memory_order_relaxed);
    }
  }
  delete ub;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "argument upload");
  return KSGD_OK;
}

Layout make_mom_layout(const ksgd_tensor_desc* d, int32_t n) {
  return make_ring_layout(n, whole_tiles(d, n, [](const ksgd_tensor_desc&) { return kChunkLog2; }) + kTailReserve,
                          sizeof(mom::TensorState), sizeof(mom::TensorInfo), 4);
}

int validate_momentum(const ksgd_tensor_desc* d, const ksgd_momentum_desc* m, int32_t n) {
  const int v = validate(d, n);
  if (v != KSGD_OK) return v;
  if (!m) return KSGD_ERR_NULL;
  for (int32_t i = 0; i < n; ++i) {
    if (d[i].comp_bits == 0) return KSGD_ERR_BITS;        // momentum goes through the lazy update
    if (m[i].mom_bits != 8 && m[i].mom_bits != 16) return KSGD_ERR_BITS;
    if (!m[i].mom) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(m[i].mom) % 16) return KSGD_ERR_ALIGN;
    if (m[i].exp_mom < kExpMin || m[i].exp_mom > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (m[i].exp_mom_next < kExpMin || m[i].exp_mom_next > kExpMax) return KSGD_ERR_EXP_RANGE;
    if (std::abs(m[i].exp_mom_next - m[i].exp_mom) > kMaxDelta) return KSGD_ERR_EXP_RANGE;
  }
  return KSGD_OK;
}

}  // namespace

struct ksgd_momentum_handle {
  Layout layout;
  std::vector<int32_t> theta_bits, mom_bits;
  mom::StepParams params;
  char* ws_base;
  cudaStream_t stream;
  int32_t n;
  int grid;
  std::vector<unsigned char> stats_host;
};

size_t kahan_sgd_momentum_workspace_bytes(const ksgd_tensor_desc* descs, const ksgd_momentum_desc* mdescs,
                                          int32_t n_tensors) {
  if (validate_momentum(descs, mdescs, n_tensors) != KSGD_OK) return 0;
  return make_mom_layout(descs, n_tensors).total;
}

int kahan_sgd_momentum_init(ksgd_momentum_handle** out, const ksgd_tensor_desc* descs,
                            const ksgd_momentum_desc* mdescs, int32_t n_tensors, ksgd_exp_mode mode,
                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return KSGD_ERR_NULL;
  *out = nullptr;
  const int v = validate_momentum(descs, mdescs, n_tensors);
  if (v != KSGD_OK) return v;
  if (mode != KSGD_EXP_FIXED && mode != KSGD_EXP_AMAX) return KSGD_ERR_MODE;
  if (!workspace) return KSGD_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(workspace) % 256) return KSGD_ERR_ALIGN;
  const Layout L = make_mom_layout(descs, n_tensors);
  if (workspace_bytes < L.total) return KSGD_ERR_WORKSPACE;

  DeviceFacts dev;            // the tile table depends on the number of blocks a step has
  {
    const cudaError_t eq = query_device(dev);
    if (eq != cudaSuccess) return cuda_fail(eq, "device query");
  }
  ksgd_momentum_handle* h = new (std::nothrow) ksgd_momentum_handle();
  if (!h) return KSGD_ERR_NULL;
  h->layout = L;
  h->n = n_tensors;
  h->ws_base = static_cast<char*>(workspace);
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->stats_host.resize(L.stats_end);

  // Host image: phase 0; in the records the first step reads (slab 2) the exponents of the
  // stored mantissas and, as overrides, the exponents the first step must write.
  std::vector<unsigned char> img(L.total, 0);
  mom::TensorState* last = reinterpret_cast<mom::TensorState*>(img.data() + L.state) + 2 * (size_t)L.slab;
  mom::TensorInfo* info = reinterpret_cast<mom::TensorInfo*>(img.data() + L.info);
  ChunkRef* chunks = reinterpret_cast<ChunkRef*>(img.data() + L.chunks);
  double state_bytes = 0.0;
  for (int32_t i = 0; i < n_tensors; ++i) {
    const ksgd_tensor_desc& t = descs[i];
    last[i].exp_theta = t.exp_theta;
    last[i].ovr_theta = t.exp_theta_next + kOvrBias;
    last[i].exp_mom = mdescs[i].exp_mom;
    last[i].ovr_mom = mdescs[i].exp_mom_next + kOvrBias;
    info[i].theta = t.theta;
    info[i].comp = t.comp;
    info[i].mom = mdescs[i].mom;
    info[i].numel = t.numel;
    info[i].theta_bits = t.theta_bits;
    info[i].comp_bits = t.comp_bits;
    info[i].mom_bits = mdescs[i].mom_bits;
    info[i].s = t.comp_bits - 1 - t.overlap_k;
    h->theta_bits.push_back(t.theta_bits);
    h->mom_bits.push_back(mdescs[i].mom_bits);
    state_bytes += (double)t.numel * ((t.theta_bits + t.comp_bits + mdescs[i].mom_bits) / 8);
  }
  const long long tiles = build_tile_table(descs, n_tensors, [](const ksgd_tensor_desc&) { return kChunkLog2; },
                                           dev.sms, chunks, nullptr);

  mom::Workspace& w = h->params.ws;
  char* b = h->ws_base;
  w.phase = reinterpret_cast<unsigned int*>(b + L.phase);
  w.state = reinterpret_cast<mom::TensorState*>(b + L.state);
  w.slab = L.slab;
  w.counters = reinterpret_cast<unsigned long long*>(b + L.counters);
  w.error = reinterpret_cast<unsigned int*>(b + L.error);
  w.info = reinterpret_cast<mom::TensorInfo*>(b + L.info);
  w.chunks = reinterpret_cast<ChunkRef*>(b + L.chunks);
  w.grad_ptr = reinterpret_cast<const float**>(b + L.grad_ptr);
  w.lr = reinterpret_cast<float*>(b + L.lr);
  w.mu = reinterpret_cast<float*>(b + L.exp_grad);
  h->params.n_tensors = n_tensors;
  h->params.tile_begin = 0;
  h->params.tile_count = (int)tiles;
  h->params.amax_mode = mode == KSGD_EXP_AMAX ? 1 : 0;
  h->params.inline_args = n_tensors <= kInlineArgs ? 1 : 0;
  h->params.advance = 1;

  cudaError_t e = cudaFuncSetAttribute(mom::ksgd_momentum_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)mom::kSharedBytes);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "device query");
  }
  h->grid = (int)(tiles < (long long)dev.sms ? tiles : (long long)dev.sms);
  h->params.state_in_l2 = state_bytes <= 0.8 * (double)dev.l2_bytes ? 1 : 0;

  e = cudaMemcpyAsync(b, img.data(), L.total, cudaMemcpyHostToDevice, h->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "workspace upload");
  }
  *out = h;
  return KSGD_OK;
}

int kahan_sgd_momentum_step(ksgd_momentum_handle* h, const float* const* grads, const float* lrs,
                            const float* mus) {
  if (!h || !grads || !lrs || !mus) return KSGD_ERR_NULL;
  for (int32_t i = 0; i < h->n; ++i) {
    if (!grads[i]) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(grads[i]) % 16) return KSGD_ERR_ALIGN;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
    if (!std::isfinite(mus[i]) || !(mus[i] >= 0.0f)) return KSGD_ERR_LR;
  }
  mom::StepArgs args{};
  if (h->params.inline_args) {
    for (int32_t i = 0; i < h->n; ++i) { args.grads[i] = grads[i]; args.lrs[i] = lrs[i]; args.mus[i] = mus[i]; }
  } else {
    const int rc = upload_long_list(h->stream, h->n, grads, lrs, mus, h->params.ws.grad_ptr, h->params.ws.lr,
                                    h->params.ws.mu);
    if (rc != KSGD_OK) return rc;
  }
  KSGD_CUDA(launch_step_kernel(mom::ksgd_momentum_step_kernel, (unsigned)h->grid, mom::kBlock, mom::kSharedBytes,
                               h->stream, h->params, args));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

int kahan_sgd_momentum_amax(ksgd_momentum_handle* h, uint32_t* amax_theta, uint32_t* amax_comp,
                            uint32_t* amax_mom, int32_t* exp_theta_cur, int32_t* exp_theta_next,
                            int32_t* exp_mom_cur, int32_t* exp_mom_next, uint64_t* n_sat_theta,
                            uint64_t* n_sat_comp, uint64_t* n_sat_mom, uint64_t* n_nonfinite) {
  if (!h) return KSGD_ERR_NULL;
  const Layout& L = h->layout;
  KSGD_CUDA(cudaMemcpyAsync(h->stats_host.data(), h->ws_base, L.stats_end, cudaMemcpyDeviceToHost,
                            h->stream));
  KSGD_CUDA(cudaStreamSynchronize(h->stream));
  const unsigned char* b = h->stats_host.data();
  const size_t n = (size_t)h->n;
  unsigned int ph = 0;
  std::memcpy(&ph, b + L.phase, 4);
  if (ph > 2) return KSGD_ERR_DEVICE;
  // the records of the last finished step; the exponents the coming step will write are the
  // overrides if set, else what the scans imply (the rule the kernel applies)
  const mom::TensorState* last = reinterpret_cast<const mom::TensorState*>(b + L.state) + ((ph + 2) % 3) * (size_t)L.slab;
  const int mode = h->params.amax_mode;
  for (size_t i = 0; i < n; ++i) {
    const mom::TensorState& r = last[i];
    if (amax_theta) amax_theta[i] = r.amax[0];
    if (amax_comp) amax_comp[i] = r.amax[1];
    if (amax_mom) amax_mom[i] = r.amax[2];
    if (exp_theta_cur) exp_theta_cur[i] = r.exp_theta;
    if (exp_mom_cur) exp_mom_cur[i] = r.exp_mom;
    if (exp_theta_next)
      exp_theta_next[i] = r.ovr_theta ? r.ovr_theta - kOvrBias : next_exponent(r.amax[0], h->theta_bits[i], r.exp_theta, mode);
    if (exp_mom_next)
      exp_mom_next[i] = r.ovr_mom ? r.ovr_mom - kOvrBias
                                  : mom::next_exponent_velocity(r.amax[2], h->mom_bits[i], r.exp_mom, mode);
  }
  if (n_sat_theta) std::memcpy(n_sat_theta, b + L.counters, 8 * n);
  if (n_sat_comp) std::memcpy(n_sat_comp, b + L.counters + 8 * n, 8 * n);
  if (n_sat_mom) std::memcpy(n_sat_mom, b + L.counters + 16 * n, 8 * n);
  if (n_nonfinite) std::memcpy(n_nonfinite, b + L.counters + 24 * n, 8 * n);
  unsigned int dev_err = 0;
  std::memcpy(&dev_err, b + L.error, 4);
  if (dev_err != 0) return KSGD_ERR_DEVICE;
  return KSGD_OK;
}

int kahan_sgd_momentum_destroy(ksgd_momentum_handle* h) {
  if (!h) return KSGD_ERR_NULL;
  const cudaError_t e = cudaStreamSynchronize(h->stream);
  delete h;
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  return KSGD_OK;
}

// ----------------------------------------------------------------------------------------
// ADAM with the lazy update.

namespace {

Layout make_adam_layout(const ksgd_tensor_desc* d, int32_t n) {
  return make_ring_layout(n, whole_tiles(d, n, [](const ksgd_tensor_desc&) { return kChunkLog2; }) + kTailReserve,
                          sizeof(adam::TensorState), sizeof(adam::TensorInfo), 5);
}

bool exp_pair_ok(int32_t cur, int32_t next) {
  return cur >= kExpMin && cur <= kExpMax && next >= kExpMin && next <= kExpMax &&
         std::abs(next - cur) <= kMaxDelta;
}

int validate_adam(const ksgd_tensor_desc* d, const ksgd_adam_desc* a, int32_t n) {
  const int v = validate(d, n);
  if (v != KSGD_OK) return v;
  if (!a) return KSGD_ERR_NULL;
  for (int32_t i = 0; i < n; ++i) {
    if (d[i].comp_bits == 0) return KSGD_ERR_BITS;        // ADAM goes through the lazy update
    if (!a[i].mom1 || !a[i].mom2) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(a[i].mom1) % 16 || reinterpret_cast<uintptr_t>(a[i].mom2) % 16)
      return KSGD_ERR_ALIGN;
    if (!exp_pair_ok(a[i].exp_m, a[i].exp_m_next) || !exp_pair_ok(a[i].exp_v, a[i].exp_v_next))
      return KSGD_ERR_EXP_RANGE;
  }
  return KSGD_OK;
}

}  // namespace

struct ksgd_adam_handle {
  Layout layout;
  std::vector<int32_t> theta_bits;
  adam::StepParams params;
  char* ws_base;
  cudaStream_t stream;
  int32_t n;
  int grid;
  std::vector<unsigned char> stats_host;
};

size_t kahan_sgd_adam_workspace_bytes(const ksgd_tensor_desc* descs, const ksgd_adam_desc* adescs,
                                      int32_t n_tensors) {
  if (validate_adam(descs, adescs, n_tensors) != KSGD_OK) return 0;
  return make_adam_layout(descs, n_tensors).total;
}

int kahan_sgd_adam_init(ksgd_adam_handle** out, const ksgd_tensor_desc* descs, const ksgd_adam_desc* adescs,
                        int32_t n_tensors, ksgd_exp_mode mode, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
  if (!out) return KSGD_ERR_NULL;
  *out = nullptr;
  const int v = validate_adam(descs, adescs, n_tensors);
  if (v != KSGD_OK) return v;
  if (mode != KSGD_EXP_FIXED && mode != KSGD_EXP_AMAX) return KSGD_ERR_MODE;
  if (!workspace) return KSGD_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(workspace) % 256) return KSGD_ERR_ALIGN;
  const Layout L = make_adam_layout(descs, n_tensors);
  if (workspace_bytes < L.total) return KSGD_ERR_WORKSPACE;

  DeviceFacts dev;            // the tile table depends on the number of blocks a step has
  {
    const cudaError_t eq = query_device(dev);
    if (eq != cudaSuccess) return cuda_fail(eq, "device query");
  }
  ksgd_adam_handle* h = new (std::nothrow) ksgd_adam_handle();
  if (!h) return KSGD_ERR_NULL;
  h->layout = L;
  h->n = n_tensors;
  h->ws_base = static_cast<char*>(workspace);
  h->stream = static_cast<cudaStream_t>(cuda_stream);
  h->stats_host.resize(L.stats_end);

  // Host image: phase 0; in the records the first step reads (slab 2) the exponents of the
  // stored mantissas and, as overrides, the exponents the first step must write.
  std::vector<unsigned char> img(L.total, 0);
  adam::TensorState* last = reinterpret_cast<adam::TensorState*>(img.data() + L.state) + 2 * (size_t)L.slab;
  adam::TensorInfo* info = reinterpret_cast<adam::TensorInfo*>(img.data() + L.info);
  ChunkRef* chunks = reinterpret_cast<ChunkRef*>(img.data() + L.chunks);
  double state_bytes = 0.0;
  for (int32_t i = 0; i < n_tensors; ++i) {
    const ksgd_tensor_desc& t = descs[i];
    last[i].exp_theta = t.exp_theta;
    last[i].ovr_theta = t.exp_theta_next + kOvrBias;
    last[i].exp_m = adescs[i].exp_m;
    last[i].ovr_m = adescs[i].exp_m_next + kOvrBias;
    last[i].exp_v = adescs[i].exp_v;
    last[i].ovr_v = adescs[i].exp_v_next + kOvrBias;
    info[i].theta = t.theta;
    info[i].comp = t.comp;
    info[i].mom1 = adescs[i].mom1;
    info[i].mom2 = adescs[i].mom2;
    info[i].numel = t.numel;
    info[i].theta_bits = t.theta_bits;
    info[i].comp_bits = t.comp_bits;
    info[i].s = t.comp_bits - 1 - t.overlap_k;
    info[i].pad = 0;
    h->theta_bits.push_back(t.theta_bits);
    state_bytes += (double)t.numel * ((t.theta_bits + t.comp_bits + 32) / 8);
  }
  const long long tiles = build_tile_table(descs, n_tensors, [](const ksgd_tensor_desc&) { return kChunkLog2; },
                                           dev.sms, chunks, nullptr);

  adam::Workspace& w = h->params.ws;
  char* b = h->ws_base;
  w.phase = reinterpret_cast<unsigned int*>(b + L.phase);
  w.state = reinterpret_cast<adam::TensorState*>(b + L.state);
  w.slab = L.slab;
  w.counters = reinterpret_cast<unsigned long long*>(b + L.counters);
  w.error = reinterpret_cast<unsigned int*>(b + L.error);
  w.info = reinterpret_cast<adam::TensorInfo*>(b + L.info);
  w.chunks = reinterpret_cast<ChunkRef*>(b + L.chunks);
  w.grad_ptr = reinterpret_cast<const float**>(b + L.grad_ptr);
  w.lr = reinterpret_cast<float*>(b + L.lr);
  h->params.n_tensors = n_tensors;
  h->params.tile_begin = 0;
  h->params.tile_count = (int)tiles;
  h->params.amax_mode = mode == KSGD_EXP_AMAX ? 1 : 0;
  h->params.inline_args = n_tensors <= kInlineArgs ? 1 : 0;
  h->params.advance = 1;

  cudaError_t e = cudaFuncSetAttribute(adam::ksgd_adam_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)adam::kSharedBytes);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "device query");
  }
  h->grid = (int)(tiles < (long long)dev.sms ? tiles : (long long)dev.sms);
  h->params.state_in_l2 = state_bytes <= 0.8 * (double)dev.l2_bytes ? 1 : 0;

  e = cudaMemcpyAsync(b, img.data(), L.total, cudaMemcpyHostToDevice, h->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
  if (e != cudaSuccess) {
    delete h;
    return cuda_fail(e, "workspace upload");
  }
  *out = h;
  return KSGD_OK;
}

int kahan_sgd_adam_step(ksgd_adam_handle* h, const float* const* grads, const float* lrs, float beta1,
                        float beta2, float eps) {
  if (!h || !grads || !lrs) return KSGD_ERR_NULL;
  if (!(beta1 >= 0.0f && beta1 <= 1.0f) || !(beta2 >= 0.0f && beta2 <= 1.0f)) return KSGD_ERR_LR;
  if (!std::isfinite(eps) || !(eps >= 0.0f)) return KSGD_ERR_LR;
  for (int32_t i = 0; i < h->n; ++i) {
    if (!grads[i]) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(grads[i]) % 16) return KSGD_ERR_ALIGN;
    if (!std::isfinite(lrs[i]) || !(lrs[i] > 0.0f)) return KSGD_ERR_LR;
  }
  adam::StepArgs args{};
  if (h->params.inline_args) {
    for (int32_t i = 0; i < h->n; ++i) { args.grads[i] = grads[i]; args.lrs[i] = lrs[i]; }
  } else {
    const int rc = upload_long_list(h->stream, h->n, grads, lrs, nullptr, h->params.ws.grad_ptr,
                                    h->params.ws.lr, nullptr);
    if (rc != KSGD_OK) return rc;
  }
  args.beta1 = beta1;
  args.beta2 = beta2;
  args.eps = eps;
  KSGD_CUDA(launch_step_kernel(adam::ksgd_adam_step_kernel, (unsigned)h->grid, adam::kBlock, adam::kSharedBytes,
                               h->stream, h->params, args));
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

int kahan_sgd_adam_amax(ksgd_adam_handle* h, const ksgd_adam_stats* out) {
  if (!h || !out) return KSGD_ERR_NULL;
  const Layout& L = h->layout;
  KSGD_CUDA(cudaMemcpyAsync(h->stats_host.data(), h->ws_base, L.stats_end, cudaMemcpyDeviceToHost,
                            h->stream));
  KSGD_CUDA(cudaStreamSynchronize(h->stream));
  const unsigned char* b = h->stats_host.data();
  const size_t n = (size_t)h->n;
  unsigned int ph = 0;
  std::memcpy(&ph, b + L.phase, 4);
  if (ph > 2) return KSGD_ERR_DEVICE;
  // the records of the last finished step; the exponents the coming step will write are the
  // overrides if set, else what the scans imply (the rules the kernel applies)
  const adam::TensorState* last = reinterpret_cast<const adam::TensorState*>(b + L.state) + ((ph + 2) % 3) * (size_t)L.slab;
  const int mode = h->params.amax_mode;
  for (size_t i = 0; i < n; ++i) {
    const adam::TensorState& r = last[i];
    if (out->amax_theta) out->amax_theta[i] = r.amax[0];
    if (out->amax_comp) out->amax_comp[i] = r.amax[1];
    if (out->amax_m) out->amax_m[i] = r.amax[2];
    if (out->amax_v) out->amax_v[i] = r.amax[3];
    if (out->exp_theta_cur) out->exp_theta_cur[i] = r.exp_theta;
    if (out->exp_m_cur) out->exp_m_cur[i] = r.exp_m;
    if (out->exp_v_cur) out->exp_v_cur[i] = r.exp_v;
    if (out->exp_theta_next)
      out->exp_theta_next[i] = r.ovr_theta ? r.ovr_theta - kOvrBias
                                           : next_exponent(r.amax[0], h->theta_bits[i], r.exp_theta, mode);
    if (out->exp_m_next)
      out->exp_m_next[i] = r.ovr_m ? r.ovr_m - kOvrBias : adam::next_exponent_moment(r.amax[2], r.exp_m, mode);
    if (out->exp_v_next)
      out->exp_v_next[i] = r.ovr_v ? r.ovr_v - kOvrBias : adam::next_exponent_moment(r.amax[3], r.exp_v, mode);
  }
  auto give = [&](void* dst, size_t off, size_t width) { if (dst) std::memcpy(dst, b + off, width * n); };
  give(out->n_sat_theta, L.counters, 8);
  give(out->n_sat_comp, L.counters + 8 * n, 8);
  give(out->n_sat_m, L.counters + 16 * n, 8);
  give(out->n_sat_v, L.counters + 24 * n, 8);
  give(out->n_nonfinite, L.counters + 32 * n, 8);
  unsigned int dev_err = 0;
  std::memcpy(&dev_err, b + L.error, 4);
  if (dev_err != 0) return KSGD_ERR_DEVICE;
  return KSGD_OK;
}

static __device__ unsigned long long g_selfcheck_mismatches[2];

int kahan_sgd_adam_selfcheck(uint64_t* div_mismatches, uint64_t* sqrt_mismatches, void* cuda_stream) {
  if (!div_mismatches || !sqrt_mismatches) return KSGD_ERR_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long* dev = nullptr;
  KSGD_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&dev), g_selfcheck_mismatches));
  KSGD_CUDA(cudaMemsetAsync(dev, 0, 16, stream));
  // exponents of a (first moment grid) and of b (denominator): corners and inside
  const int combos[][2] = {{0, 0}, {-20, -10}, {-64, -32}, {-64, 40}, {64, -32}, {64, 40}, {-37, 5}, {-1, 1}};
  for (const auto& c : combos) {
    adam::ksgd_adam_selfcheck_div<<<(1u << 23) / 256, 256, 0, stream>>>(c[0], c[1], dev);
    g_launches.fetch_add(1, std::memory_order_relaxed);
  }
  adam::ksgd_adam_selfcheck_sqrt<<<128, 256, 0, stream>>>(dev + 1);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  unsigned long long host[2] = {0, 0};
  KSGD_CUDA(cudaMemcpyAsync(host, dev, 16, cudaMemcpyDeviceToHost, stream));
  KSGD_CUDA(cudaStreamSynchronize(stream));
  *div_mismatches = host[0];
  *sqrt_mismatches = host[1];
  return KSGD_OK;
}

int kahan_sgd_adam_destroy(ksgd_adam_handle* h) {
  if (!h) return KSGD_ERR_NULL;
  const cudaError_t e = cudaStreamSynchronize(h->stream);
  delete h;
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  return KSGD_OK;
}

// ----------------------------------------------------------------------------------------
// fp32 <-> dynamic fixed-point, and the classifier bit-width rule.

}  // extern "C"

namespace {

int check_format(int32_t theta_bits, int32_t comp_bits, int32_t overlap_k) {
  if (theta_bits != 8 && theta_bits != 16) return KSGD_ERR_BITS;
  if (comp_bits != 0 && comp_bits != 8 && comp_bits != 16) return KSGD_ERR_BITS;
  if (comp_bits != 0 && (overlap_k < 0 || overlap_k > comp_bits - 1)) return KSGD_ERR_OVERLAP;
  return KSGD_OK;
}

// Grid of the conversion kernels: blocks of 256 threads, never more than the work (four
// elements per thread and access at least), and at most `per_sm` blocks per SM.  Measured on
// 64 Mi elements: the export is fastest with 64 (0.95-0.99 of the copy peak against 0.87-0.96
// with 16; 128 the same), the two passes of the import with 32 (0.86-0.94; 0.84-0.92 with 16
// or 64, 0.77-0.87 with 128: every block of the scan ends in a reduction and two atomics).
constexpr int kImportBlocksPerSm = 32, kExportBlocksPerSm = 64;
int convert_grid(int64_t numel, int per_sm) {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
    else sms = 148;
  }
  const int64_t blocks = (numel / 4 + convert::kThreads - 1) / convert::kThreads + 1;
  return (int)(blocks < (int64_t)sms * per_sm ? blocks : (int64_t)sms * per_sm);
}

template <int TB>
void launch_quantize_tb(int cb, const float* src, void* theta, void* comp, int64_t numel, const int* exp_dev,
                        int e, int s, cudaStream_t st) {
  const int grid = convert_grid(numel, kImportBlocksPerSm);
  if (cb == 8) convert::quantize_kernel<TB, 8><<<grid, convert::kThreads, 0, st>>>(src, theta, comp, numel, exp_dev, e, s);
  else if (cb == 16) convert::quantize_kernel<TB, 16><<<grid, convert::kThreads, 0, st>>>(src, theta, comp, numel, exp_dev, e, s);
  else convert::quantize_kernel<TB, 0><<<grid, convert::kThreads, 0, st>>>(src, theta, comp, numel, exp_dev, e, s);
}

template <int TB>
void launch_dequantize_tb(int cb, const void* theta, const void* comp, float* dst, int64_t numel, int e, int s,
                          cudaStream_t st) {
  const int grid = convert_grid(numel, kExportBlocksPerSm);
  if (cb == 8) convert::dequantize_kernel<TB, 8><<<grid, convert::kThreads, 0, st>>>(theta, comp, dst, numel, e, s);
  else if (cb == 16) convert::dequantize_kernel<TB, 16><<<grid, convert::kThreads, 0, st>>>(theta, comp, dst, numel, e, s);
  else convert::dequantize_kernel<TB, 0><<<grid, convert::kThreads, 0, st>>>(theta, comp, dst, numel, e, s);
}

// Max scan with the exponent left at exp_dev (device), then the quantization reading it
// from there.  Enqueues two kernels; nothing waits.
int import_auto(const float* src, void* theta, void* comp, int64_t numel, int32_t theta_bits, int32_t comp_bits,
                int32_t overlap_k, int32_t* exp_dev, void* scratch, cudaStream_t st) {
  convert::absmax_fit_kernel<<<convert_grid(numel, kImportBlocksPerSm), convert::kThreads, 0, st>>>(
      src, numel, theta_bits, static_cast<convert::ScanScratch*>(scratch), exp_dev);
  const int s = comp_bits ? comp_bits - 1 - overlap_k : 0;
  if (theta_bits == 8) launch_quantize_tb<8>(comp_bits, src, theta, comp, numel, exp_dev, 0, s, st);
  else launch_quantize_tb<16>(comp_bits, src, theta, comp, numel, exp_dev, 0, s, st);
  g_launches.fetch_add(2, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

}  // namespace

extern "C" {

int kahan_sgd_import(const float* src, void* theta, void* comp, int64_t numel, int32_t theta_bits,
                     int32_t comp_bits, int32_t overlap_k, int32_t exp_theta, int32_t* exp_theta_out,
                     void* scratch, void* cuda_stream) {
  const int f = check_format(theta_bits, comp_bits, overlap_k);
  if (f != KSGD_OK) return f;
  if (!src || !theta || (comp_bits != 0) != (comp != nullptr)) return KSGD_ERR_NULL;
  if (numel <= 0) return KSGD_ERR_NUMEL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int e = exp_theta;
  if (exp_theta == KSGD_EXP_AUTO) {
    // scan and quantization run back to back on the device; the host only waits to hand the
    // exponent back
    if (!scratch) return KSGD_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(scratch) % 4) return KSGD_ERR_ALIGN;
    KSGD_CUDA(cudaMemsetAsync(scratch, 0, 16, st));
    int32_t* exp_dev = static_cast<int32_t*>(scratch) + 2;
    const int r = import_auto(src, theta, comp, numel, theta_bits, comp_bits, overlap_k, exp_dev, scratch, st);
    if (r != KSGD_OK) return r;
    KSGD_CUDA(cudaMemcpyAsync(&e, exp_dev, 4, cudaMemcpyDeviceToHost, st));
    KSGD_CUDA(cudaStreamSynchronize(st));
  } else {
    if (exp_theta < kExpMin || exp_theta > kExpMax) return KSGD_ERR_EXP_RANGE;
    const int s = comp_bits ? comp_bits - 1 - overlap_k : 0;
    if (theta_bits == 8) launch_quantize_tb<8>(comp_bits, src, theta, comp, numel, nullptr, e, s, st);
    else launch_quantize_tb<16>(comp_bits, src, theta, comp, numel, nullptr, e, s, st);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    KSGD_CUDA(cudaGetLastError());
  }
  if (exp_theta_out) *exp_theta_out = e;
  return KSGD_OK;
}

int kahan_sgd_import_dev(const float* src, void* theta, void* comp, int64_t numel, int32_t theta_bits,
                         int32_t comp_bits, int32_t overlap_k, int32_t* exp_theta_dev, void* scratch,
                         void* cuda_stream) {
  const int f = check_format(theta_bits, comp_bits, overlap_k);
  if (f != KSGD_OK) return f;
  if (!src || !theta || (comp_bits != 0) != (comp != nullptr) || !exp_theta_dev || !scratch) return KSGD_ERR_NULL;
  if (numel <= 0) return KSGD_ERR_NUMEL;
  if (reinterpret_cast<uintptr_t>(scratch) % 4 || reinterpret_cast<uintptr_t>(exp_theta_dev) % 4) return KSGD_ERR_ALIGN;
  return import_auto(src, theta, comp, numel, theta_bits, comp_bits, overlap_k, exp_theta_dev, scratch,
                     static_cast<cudaStream_t>(cuda_stream));
}

int kahan_sgd_export(const void* theta, const void* comp, float* dst, int64_t numel, int32_t theta_bits,
                     int32_t comp_bits, int32_t overlap_k, int32_t exp_theta, void* cuda_stream) {
  const int f = check_format(theta_bits, comp_bits, overlap_k);
  if (f != KSGD_OK) return f;
  if (!dst || !theta || (comp_bits != 0) != (comp != nullptr)) return KSGD_ERR_NULL;
  if (numel <= 0) return KSGD_ERR_NUMEL;
  if (exp_theta < kExpMin || exp_theta > kExpMax) return KSGD_ERR_EXP_RANGE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int s = comp_bits ? comp_bits - 1 - overlap_k : 0, e = exp_theta;
  if (theta_bits == 8) launch_dequantize_tb<8>(comp_bits, theta, comp, dst, numel, e, s, st);
  else launch_dequantize_tb<16>(comp_bits, theta, comp, dst, numel, e, s, st);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  KSGD_CUDA(cudaGetLastError());
  return KSGD_OK;
}

int32_t kahan_sgd_classifier_bits(int64_t n_classes, double alpha) {
  if (n_classes < 2 || !(alpha > 0.0) || !(alpha < 1.0)) return 0;
  // Eq. 5: bitwidth > log2(|class| - 1) + log2(2 / alpha); the smallest integer that is
  // strictly larger.  Evaluated on the integers: 2^(b-1) * alpha > |class| - 1.
  for (int32_t b = 2; b <= 64; ++b)
    if (std::ldexp(alpha, b - 1) > (double)(n_classes - 1)) return b;
  return 64;
}

const char* kahan_sgd_strerror(int code) {
  switch (code) {
    case KSGD_OK: return "success";
    case KSGD_ERR_NULL: return "a required pointer is NULL (or comp given with comp_bits == 0)";
    case KSGD_ERR_BITS: return "theta_bits must be 8 or 16 and comp_bits 0, 8 or 16";
    case KSGD_ERR_OVERLAP: return "overlap_k must lie in 0 .. comp_bits-1";
    case KSGD_ERR_EXP_RANGE: return "exponent outside [-64, 64] or more than 8 from the current one";
    case KSGD_ERR_NUMEL: return "numel and n_tensors must be positive (and at most 2^31-1 chunks)";
    case KSGD_ERR_ALIGN: return "device pointers must be 16-byte aligned (workspace: 256)";
    case KSGD_ERR_WORKSPACE: return "workspace or staging buffer too small";
    case KSGD_ERR_LR: return "learning rates must be finite and > 0 (momentum coefficients finite and >= 0)";
    case KSGD_ERR_CUDA: return "CUDA runtime error (see kahan_sgd_last_cuda_error)";
    case KSGD_ERR_MODE: return "unknown exponent mode";
    case KSGD_ERR_DEVICE: return "a bounded wait inside the step kernel ran out; results of that step are invalid";
    default: return "unknown error code";
  }
}

const char* kahan_sgd_last_cuda_error(void) { return g_cuda_error; }

uint64_t kahan_sgd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
