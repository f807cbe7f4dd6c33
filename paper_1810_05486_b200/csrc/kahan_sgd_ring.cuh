// The machinery every step kernel of this library shares (Algorithm 1 of arXiv 1810.05486 in
// the plain optimizer, the momentum optimizer and ADAM): a persistent grid, one block per SM,
// in which one producer thread streams tiles of a ragged tensor list into a paged
// shared-memory ring with bulk asynchronous copies and the consumer warps compute from shared
// memory; the per-tensor max scans gathered on the way; and the state that steps hand to one
// another.  What differs between the optimizers -- how many arrays a tile has, the arithmetic
// of an element, how many scans steer how many exponents -- comes in as a policy class.
//
// Structure.  The tensor list is cut into tiles of kChunk elements (a multiple where the host
// chose larger ones, power-of-two pieces in the table's last round); block b takes tiles b,
// b + gridDim.x, ....  A tile's arrays go into a 224 KB
// ring handed out in 8 KB pages, so a tile takes only what its formats need and two to four
// tiles are resident, independent of registers and occupancy.  The copies of a tile complete
// an mbarrier; the consumers wait on it, compute, store their results straight to global
// memory with 16-byte stores, add their scans to the tile's slot and arrive on a second
// barrier, after which the producer takes the pages back, merges the slot's scans into those
// of the tensor run and publishes a run with one set of global atomics.  No block ever waits
// for another block; every wait inside a block is bounded.
//
// State between steps.  What a step leaves behind for a tensor (the exponents it wrote, its
// max scans, overrides for the next step) is one record per tensor in three rotating slabs
// indexed by the step's phase p = step mod 3 (a word in the workspace).  Step p reads the
// records of slab p-1, derives from them the exponents it writes (every block that meets a
// tensor derives the same values; the block that holds the tensor's first tile stores them
// into slab p), adds its own scans to slab p, and clears the tensor's record in slab p+1,
// which nobody reads or writes until the next step.  So a step needs no pass "after all
// blocks are done": the kernel ends when each block has published its scans.  The phase word
// is advanced by the block that draws the last entry ticket, i.e. after every block of the
// step has read it.
//
// A policy class P provides
//   kStreams            arrays per tile; stream 0 is the gradient (read once)
//   kConsumerWarps      consumer warps per block (one more warp produces)
//   kAmax, kCounts      max scans and counters per tensor
//   kLongStepTiles      tiles per block from which a step beyond L2 limits its tiles in flight
//   kGradEvictFirstBeyondL2   gradient loads carry the L2 evict-first hint also when the state does not fit in L2
//   Params              kernel parameter with: ws.phase, ws.state, ws.slab, ws.counters, ws.error,
//                       ws.info, ws.chunks; n_tensors, tile_begin, tile_count, advance, state_in_l2
//   Info                the tensor table entry (with numel); State: the per-step record, whose
//                       member amax[kAmax] the blocks add their scans to
//   TileDesc, TileScan  what the producer tells the consumers about a tile; the tile's scan
//                       slot: kAmax maxima followed by kCounts counts, 32-bit words
//   Meta                what the producer knows about a tile's tensor (with .ti, the Info)
//   load_meta(p, a, t, ph, ti)   read slab ph-1's record and the per-step arguments, derive exponents
//   record(p, t, ph, m)          store the derived exponents into slab ph, clear the record in slab ph+1
//   streams(m, base, bytes)      global base address and bytes per element of each array (0: absent)
//   fill_desc(td, p, m, tensor, count, n_bulk, page, gptr)   gptr: the tile's first element in each array
//   consume(td, scan, ring, ctid, lane)   one consumer thread's share of a tile, scans included
#pragma once

#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

namespace ksgd {

constexpr int kChunk = 8192;           // elements per tile (twice as many for 8-bit theta in long lists)
constexpr long long kBigTileMinTiles = 1024;   // a list gets the large 8-bit tiles if it still has this many tiles
constexpr int kSlots = 6;              // tiles a block can have in its ring at once
constexpr int kPageBytes = 8192;       // the ring is handed out in pages
static_assert(kChunk == 8192 && kPageBytes == kChunk, "the producer's page arithmetic assumes 8192-element tiles and 8 KB pages");
static_assert(kChunk == 1 << 13, "kChunkLog2");
constexpr int kPages = 28;             // 224 KB of tile data per block
constexpr int kTilesInFlight = 2;      // a step that streams from DRAM keeps this many tiles on their way, and more
constexpr int kPagesInFlight = 18;     // only while they take no more than this many pages together (ring_step)
constexpr int kInlineArgs = 256;     // lists up to this long pass grads/lrs as kernel parameters
constexpr int kUploadBatch = 1024;   // tensors per launch of the argument-upload kernel
constexpr int kDLimit = 1 << 30;     // clamp of the quantized increment, in compensation LSBs
constexpr int kMaxDelta = 8;         // largest exponent change per step
constexpr int kExpMin = -64, kExpMax = 64;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a barrier wait gives up after 2 s

enum DeviceError { kErrNone = 0, kErrFullWait = 1, kErrEmptyWait = 2 };


// One entry of the tile table.  A tile is 2^lg consecutive elements of one tensor (only a
// tensor's last tile is short), lg from kMinTileLog2 to 15, starting at element index << lg.
// Most tiles of a list have the size its tensors' formats ask for (kChunk elements or a
// multiple); the tiles of the table's last, incomplete round over the blocks are cut into
// power-of-two pieces so that the round has about one piece per block (see the host's table
// builder), which is why every entry carries its own size.
struct ChunkRef {
  int tensor;          // index into the tensor list
  unsigned int where;  // index (low kTileIndexBits bits) | lg << kTileIndexBits
};
constexpr int kTileIndexBits = 27;
constexpr int kMinTileLog2 = 9;      // pieces of at least 512 elements (one 16-element vector per consumer thread)
constexpr int kChunkLog2 = 13;
__host__ __device__ __forceinline__ ChunkRef make_chunk_ref(int tensor, long long index, int lg) {
  return ChunkRef{tensor, (unsigned int)index | ((unsigned int)lg << kTileIndexBits)};
}
__host__ __device__ __forceinline__ int chunk_log2(const ChunkRef& c) { return (int)(c.where >> kTileIndexBits); }
__host__ __device__ __forceinline__ long long chunk_index(const ChunkRef& c) {
  return (long long)(c.where & ((1u << kTileIndexBits) - 1u));
}

// Device-side view of the caller's workspace.
// ----------------------------------------------------------------------------------------
// mbarrier / bulk-copy wrappers (PTX)

__device__ __forceinline__ unsigned int smem_addr(const void* p) {
  return static_cast<unsigned int>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(smem_addr(bar))
               : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned int bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(
                   smem_addr(bar)),
               "r"(bytes)
               : "memory");
}

// Announce `bytes` more bytes for the current phase without arriving.
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned int bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned int parity) {
  unsigned int ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: false if the phase did not complete within kWaitLimitNs or another thread
// of the block has already given up.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned int parity,
                                          const volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > kWaitLimitNs) return false;
  }
}

// Global -> shared bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned),
// completion counted in bytes on `bar`.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, unsigned int bytes,
                                          unsigned long long* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_addr(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}

// Same, with an L2 eviction-priority hint for data that is read once per step.
__device__ __forceinline__ void bulk_load_hint(void* dst_smem, const void* src_gmem, unsigned int bytes,
                                               unsigned long long* bar, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_addr(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
      : "memory");
}

// Programmatic dependent launch.  The step kernels are launched with programmatic stream
// serialization: a block of the next kernel in the stream may become resident as soon as an
// SM has room (a block of this kernel has exited) and run its prologue -- barrier set-up,
// its first table entries -- while the rest of this kernel finishes.  Before it touches
// anything an earlier kernel wrote (exponents, mantissas, gradients, per-step arguments in
// the workspace) every thread passes grid_dependency_wait(), which returns once the
// preceding kernel has completed and its writes are visible.  Launched the ordinary way
// both instructions do nothing.  The hardware orders the grids; nothing spins.
__device__ __forceinline__ void grid_dependency_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ unsigned long long l2_policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// ----------------------------------------------------------------------------------------
// Arithmetic helpers

__device__ __forceinline__ float pow2_float(int e) {  // exact 2^e for e in [-126, 127]
  return __int_as_float((e + 127) << 23);
}

// a / 2^r, round to nearest, ties to even (|a| < 2^62).
__device__ __forceinline__ long long rne_shift64(long long a, int r) {
  if (r == 0) return a;
  const long long bias = ((1LL << (r - 1)) - 1) + ((a >> r) & 1LL);
  return (a + bias) >> r;
}

// ----------------------------------------------------------------------------------------
// 16-byte vector helpers.  A Pack holds V elements of B bits (8, 16, 32 or 64 bytes).

template <int BYTES> struct Pack;
template <> struct Pack<8>  { uint2 v; };
template <> struct Pack<16> { uint4 v; };
template <> struct Pack<32> { uint4 v[2]; };
template <> struct Pack<64> { uint4 v[4]; };

template <int BYTES>
__device__ __forceinline__ Pack<BYTES> load_pack(const void* p) {
  Pack<BYTES> r;
  if constexpr (BYTES == 8) {
    r.v = *reinterpret_cast<const uint2*>(p);
  } else if constexpr (BYTES == 16) {
    r.v = *reinterpret_cast<const uint4*>(p);
  } else {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) r.v[i] = reinterpret_cast<const uint4*>(p)[i];
  }
  return r;
}

template <int BYTES>
__device__ __forceinline__ void store_pack(void* p, const Pack<BYTES>& r) {
  if constexpr (BYTES == 8) {
    *reinterpret_cast<uint2*>(p) = r.v;
  } else if constexpr (BYTES == 16) {
    *reinterpret_cast<uint4*>(p) = r.v;
  } else {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) reinterpret_cast<uint4*>(p)[i] = r.v[i];
  }
}

// The same to global memory with the streaming (evict-first) hint: for results that will not
// be read again before they have left L2 anyway, so that they leave it promptly and in order.
template <int BYTES>
__device__ __forceinline__ void store_pack_streaming(void* p, const Pack<BYTES>& r) {
  if constexpr (BYTES == 8) {
    __stcs(reinterpret_cast<uint2*>(p), r.v);
  } else if constexpr (BYTES == 16) {
    __stcs(reinterpret_cast<uint4*>(p), r.v);
  } else {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) __stcs(reinterpret_cast<uint4*>(p) + i, r.v[i]);
  }
}

template <int BYTES>
__device__ __forceinline__ unsigned int pack_word(const Pack<BYTES>& r, int w) {
  if constexpr (BYTES == 8) {
    return w == 0 ? r.v.x : r.v.y;
  } else if constexpr (BYTES == 16) {
    return w == 0 ? r.v.x : (w == 1 ? r.v.y : (w == 2 ? r.v.z : r.v.w));
  } else {
    const uint4& q = r.v[w >> 2];
    const int j = w & 3;
    return j == 0 ? q.x : (j == 1 ? q.y : (j == 2 ? q.z : q.w));
  }
}

template <int BYTES>
__device__ __forceinline__ void set_pack_word(Pack<BYTES>& r, int w, unsigned int x) {
  if constexpr (BYTES == 8) {
    if (w == 0) r.v.x = x; else r.v.y = x;
  } else if constexpr (BYTES == 16) {
    if (w == 0) r.v.x = x; else if (w == 1) r.v.y = x; else if (w == 2) r.v.z = x; else r.v.w = x;
  } else {
    uint4& q = r.v[w >> 2];
    const int j = w & 3;
    if (j == 0) q.x = x; else if (j == 1) q.y = x; else if (j == 2) q.z = x; else q.w = x;
  }
}

// ----------------------------------------------------------------------------------------
// Exact small integers in binary32 (see the step kernels for the technique)

constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23, bits 0x4B400000
constexpr unsigned int kMagicBits = 0x4B400000u;

// M + 2^(BITS-1) + q for element i of a pack whose sign bits have been flipped.
template <int BITS, int BYTES>
__device__ __forceinline__ float magic_elem(const Pack<BYTES>& r, int i) {
  if constexpr (BITS == 8) {
    return __uint_as_float(__byte_perm(pack_word(r, i >> 2), kMagicBits, 0x7640u | (unsigned)(i & 3)));
  } else {
    return __uint_as_float(__byte_perm(pack_word(r, i >> 1), kMagicBits, (i & 1) ? 0x7632u : 0x7610u));
  }
}

// M + q for element i of a pack of signed mantissas, in one instruction: the integer dot
// product with a selector that is 1 at element i sign-extends the mantissa and adds it to
// M's bit pattern (for |q| < 2^22 integer addition on the bits is addition of the values).
// It runs on the FMA pipe; the PRMT form above and the sign flips it needs take the ALU
// pipe, which has half the lanes and also carries the scans and the packing.
template <int BITS, int BYTES>
__device__ __forceinline__ float magic_signed(const Pack<BYTES>& r, int i) {
  if constexpr (BITS == 8) {
    return __int_as_float(__dp4a((int)pack_word(r, i >> 2), 1 << (8 * (i & 3)), (int)kMagicBits));
  } else {
    return __int_as_float(__dp2a_lo((int)pack_word(r, i >> 1), (i & 1) ? 0x0100 : 0x0001, (int)kMagicBits));
  }
}

template <int BITS, int BYTES>
__device__ __forceinline__ void flip_signs(Pack<BYTES>& r) {
  constexpr unsigned int m = BITS == 8 ? 0x80808080u : 0x80008000u;
#pragma unroll
  for (int w = 0; w < BYTES / 4; ++w) set_pack_word(r, w, pack_word(r, w) ^ m);
}

// Low BITS bits of V magic floats, packed.
template <int BITS, int V>
__device__ __forceinline__ Pack<V * BITS / 8> pack_magic(const float (&x)[V]) {
  Pack<V * BITS / 8> r;
  if constexpr (BITS == 8) {
#pragma unroll
    for (int w = 0; w < V / 4; ++w) {
      const unsigned int lo = __byte_perm(__float_as_uint(x[4 * w]), __float_as_uint(x[4 * w + 1]), 0x0040);
      const unsigned int hi = __byte_perm(__float_as_uint(x[4 * w + 2]), __float_as_uint(x[4 * w + 3]), 0x0040);
      set_pack_word(r, w, __byte_perm(lo, hi, 0x5410));
    }
  } else {
#pragma unroll
    for (int w = 0; w < V / 2; ++w)
      set_pack_word(r, w, __byte_perm(__float_as_uint(x[2 * w]), __float_as_uint(x[2 * w + 1]), 0x5410));
  }
  return r;
}

// Three-input maximum / minimum (one instruction on sm_100a).  The .NaN form returns NaN as
// soon as one input is NaN, which is how a NaN product reaches the range check below.
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float d;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Next exponent from the max scan: the tight fit puts the largest mantissa in
// (QMAX/2, QMAX].  With L = bit length of amax and QMAX = 2^(b-1)-1, the change is
// L-(b-1), plus one more when amax still exceeds QMAX*2^change.
__host__ __device__ __forceinline__ int bit_length(unsigned int x) {
#ifdef __CUDA_ARCH__
  return 32 - __clz(x);
#else
  int n = 0;
  while (x) { ++n; x >>= 1; }
  return n;
#endif
}

__host__ __device__ __forceinline__ int next_exponent(unsigned int amax, int bits, int e_out, int amax_mode) {
  if (!amax_mode || amax == 0u) return e_out;
  const int L = bit_length(amax);
  int change = L - (bits - 1);
  if (change >= 1) {
    const unsigned long long cap = (unsigned long long)((1 << (bits - 1)) - 1) << change;
    if ((unsigned long long)amax > cap) ++change;
  }
  change = change < -kMaxDelta ? -kMaxDelta : (change > kMaxDelta ? kMaxDelta : change);
  const int e = e_out + change;
  return e < kExpMin ? kExpMin : (e > kExpMax ? kExpMax : e);
}


constexpr int kOvrBias = 1000;       // an override of e is stored as e + kOvrBias, 0 = none

template <class P>
struct __align__(128) RingShared {
  unsigned long long full[kSlots];     // producer -> consumers: the tile's bytes have landed
  unsigned long long empty[kSlots];    // consumers -> producer: the tile's pages may be reused
  typename P::TileDesc desc[kSlots];
  typename P::TileScan scan[kSlots];
  int slot_pages[kSlots];              // ring pages held by the tile in each slot
  int slot_tensor[kSlots];             // its tensor
  int abort_flag;   // set by the first thread whose bounded wait ran out
  int never;        // stays 0: abort flag for waits that must not be cut short
};

template <class P>
constexpr size_t ring_shared_bytes() { return (size_t)kPages * kPageBytes + sizeof(RingShared<P>); }

template <class P>
constexpr int ring_block_threads() { return 32 * P::kConsumerWarps + 32; }

// Producer side: scans of finished tiles are merged per tensor in registers and go to
// global memory when the tensor changes (one set of atomics per block and tensor run).
template <class P>
struct ScanAcc {
  int tensor = -1;
  unsigned int amax[P::kAmax] = {};
  unsigned int cnt[P::kCounts] = {};
};

template <class P>
__device__ __forceinline__ void publish(const typename P::Params& p, ScanAcc<P>& acc, typename P::State* now) {
  if (acc.tensor >= 0) {
    const int t = acc.tensor, n = p.n_tensors;
#pragma unroll
    for (int i = 0; i < P::kAmax; ++i)
      if (acc.amax[i]) atomicMax(&now[t].amax[i], acc.amax[i]);
#pragma unroll
    for (int i = 0; i < P::kCounts; ++i)
      if (acc.cnt[i]) atomicAdd(&p.ws.counters[(size_t)i * n + t], (unsigned long long)acc.cnt[i]);
  }
  acc = ScanAcc<P>{};
}

template <class P>
__device__ __forceinline__ void take_back(const typename P::Params& p, ScanAcc<P>& acc, typename P::State* now,
                                          typename P::TileScan* scan, int tensor) {
  if (tensor != acc.tensor) {
    publish<P>(p, acc, now);
    acc.tensor = tensor;
  }
  unsigned int* w = reinterpret_cast<unsigned int*>(scan);
#pragma unroll
  for (int i = 0; i < P::kAmax; ++i) { acc.amax[i] = max(acc.amax[i], w[i]); w[i] = 0u; }
#pragma unroll
  for (int i = 0; i < P::kCounts; ++i) { acc.cnt[i] += w[P::kAmax + i]; w[P::kAmax + i] = 0u; }
}

// The whole step of one block.
template <class P, typename Args>
__device__ __forceinline__ void ring_step(const typename P::Params& p, const Args& a) {
  using Shared = RingShared<P>;
  using Meta = typename P::Meta;
  using Info = typename P::Info;
  using State = typename P::State;
  using TileDesc = typename P::TileDesc;
  using TileScan = typename P::TileScan;
  constexpr int S = P::kStreams;
  constexpr int kConsumers = 32 * P::kConsumerWarps;
  static_assert(sizeof(TileScan) % 4 == 0 && sizeof(TileScan) >= 4 * (P::kAmax + P::kCounts), "scan slot layout");

  extern __shared__ __align__(128) unsigned char smem[];
  Shared* sh = reinterpret_cast<Shared*>(smem + (size_t)kPages * kPageBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&sh->full[s], 1u);
      mbar_init(&sh->empty[s], (unsigned)P::kConsumerWarps);
    }
    sh->abort_flag = 0;
    sh->never = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kSlots * (int)(sizeof(TileScan) / 4))
    reinterpret_cast<unsigned int*>(sh->scan)[threadIdx.x] = 0u;
  __syncthreads();

  if (warp == P::kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    // Block b takes tiles b, b + gridDim.x, ...: neighbouring tiles run on neighbouring
    // SMs at the same time, and the tiles of a tensor that needs a slow path are spread
    // evenly over all blocks.  Table entries are fetched two tiles ahead and the tensor's
    // data one tile ahead, so none of these loads sits between a freed page and the copy
    // that refills it.
    if (lane == 0) {
      const int stride = (int)gridDim.x;
      const int n_my = (p.tile_count - (int)blockIdx.x + stride - 1) / stride;
      const int tile0 = p.tile_begin + (int)blockIdx.x;
      const unsigned long long grad_policy = l2_policy_evict_first();
      ScanAcc<P> acc;
      // the tile table and the tensor table are written once at init: read the first
      // entries before waiting for the preceding kernel
      ChunkRef cr = p.ws.chunks[tile0];
      ChunkRef cr1{-1, 0u};
      if (n_my > 1) cr1 = p.ws.chunks[tile0 + stride];
      const Info ti_first = p.ws.info[cr.tensor];
      // The step's phase.  The preceding step moves the word on as soon as all of its blocks
      // have started, long before it ends, so the value read here, before the wait, is
      // normally the right one already: the first record is fetched under it while the word
      // is read again, and only fetched a second time if the two differ.  (The block's entry
      // ticket, which tells the last block that all have read this word, is drawn by a
      // consumer thread once the first tile has landed.)
      int ph = (int)__ldcg(p.ws.phase);
      grid_dependency_wait();
      const int ph_now = (int)__ldcg(p.ws.phase);
      Meta meta = P::load_meta(p, a, cr.tensor, ph, &ti_first);
      if (ph_now != ph) {
        ph = ph_now;
        meta = P::load_meta(p, a, cr.tensor, ph, &ti_first);
      }
      if (chunk_index(cr) == 0) P::record(p, cr.tensor, ph, meta);
      State* now = p.ws.state + (size_t)ph * p.ws.slab;
      int issued = 0;
      // The ring: pages from `head` on are free, tiles are released in the order they were
      // issued, `oldest` is the first tile whose pages have not been taken back yet.
      int head = 0, free_pages = kPages, oldest = 0;
      bool gave_up = false;
      // A step that streams everything from DRAM (state too large to stay in L2, at least
      // P::kLongStepTiles tiles per block) is bound by DRAM, and DRAM serves it faster with
      // fewer requests queued: there kTilesInFlight tiles are on their way at once, and more
      // only while all of them together take at most kPagesInFlight pages (before issuing a
      // tile the producer waits for the oldest tiles in flight to land until that holds).
      // With the state resident in L2 the limit costs about 3 %, so it is left out; the tile
      // count from which it pays is measured per optimizer.  The ring still holds up to three
      // and a half tiles, so landed tiles wait for the consumers as before.  The wait stands
      // before the tile's descriptor is built, not directly before its copies: the few
      // hundred nanoseconds between are part of what the limit buys (measured both ways).
      const bool long_step = n_my >= P::kLongStepTiles && !p.state_in_l2;
      int landed = 0, flight_pages = 0;   // first tile not known to have landed; pages of the tiles from there on
      int last_need = 0;                  // pages of the tile issued last
      for (int i = 0; i < n_my; ++i) {
        const int slot = i % kSlots;
        if (long_step) {
          // the limit on tiles in flight: wait for the oldest of them to land until this one
          // fits (taken to need the pages its predecessor took: the wait comes first)
          while (i - landed >= kTilesInFlight && flight_pages + last_need > kPagesInFlight) {
            if (!mbar_wait(&sh->full[landed % kSlots], (unsigned)(landed / kSlots) & 1u, &sh->abort_flag)) {
              gave_up = true;
              break;
            }
            flight_pages -= sh->slot_pages[landed % kSlots];
            ++landed;
          }
          if (gave_up) {
            // this tile is never issued: its barrier stays open and the consumers leave on the flag
            sh->abort_flag = 1;
            atomicCAS(p.ws.error, 0u, (unsigned)kErrFullWait);
            break;
          }
        }
        ChunkRef cr2{-1, 0u};
        if (i + 2 < n_my) cr2 = p.ws.chunks[tile0 + (i + 2) * stride];
        Meta meta1 = meta;
        if (i + 1 < n_my && cr1.tensor != cr.tensor) {
          meta1 = P::load_meta(p, a, cr1.tensor, ph, nullptr);
          if (chunk_index(cr1) == 0) P::record(p, cr1.tensor, ph, meta1);
        }

        // where the arrays go, and how many pages that takes including those skipped when
        // a run does not fit before the end of the ring (kChunk == kPageBytes: an array of
        // b-byte elements takes b pages, 2b or 4b with the large tiles; the pieces of the
        // table's last round are given the pages of a kChunk tile)
        const int lg = chunk_log2(cr);
        const int big = lg > kChunkLog2 ? lg - kChunkLog2 : 0;
        const int chunk = 1 << lg;
        const unsigned char* base[S];
        int bytes[S];
        P::streams(meta, base, bytes);
        int page[S], h2 = head, need = 0;
#pragma unroll
        for (int r = 0; r < S; ++r) {
          page[r] = 0;
          const int run = bytes[r] << big;
          if (run == 0) continue;
          if (h2 + run > kPages) { need += kPages - h2; h2 = 0; }
          page[r] = h2;
          h2 += run;
          need += run;
        }
        if (h2 == kPages) h2 = 0;
        // take back pages, descriptor slots and scans from the oldest tiles until this one fits
        while (free_pages < need || i - oldest >= kSlots) {
          const int os = oldest % kSlots;
          if (!mbar_wait(&sh->empty[os], (unsigned)(oldest / kSlots) & 1u, &sh->abort_flag)) {
            gave_up = true;
            break;
          }
          take_back<P>(p, acc, now, &sh->scan[os], sh->slot_tensor[os]);
          free_pages += sh->slot_pages[os];
          ++oldest;
        }
        if (gave_up) {
          sh->abort_flag = 1;
          atomicCAS(p.ws.error, 0u, (unsigned)kErrEmptyWait);
          break;
        }
        if (long_step) {
          // tiles taken back have landed: keep the count of those in flight in step (before
          // the slot's page count is overwritten)
          while (landed < oldest) {
            flight_pages -= sh->slot_pages[landed % kSlots];
            ++landed;
          }
          flight_pages += need;
          last_need = need;
        }
        head = h2;
        free_pages -= need;
        sh->slot_pages[slot] = need;
        sh->slot_tensor[slot] = cr.tensor;

        const long long first = chunk_index(cr) << lg;
        const long long left = meta.ti.numel - first;
        const int count = left < (long long)chunk ? (int)left : chunk;
        const int n_bulk = count & ~15;
        const unsigned char* gptr[S];
        int row_bytes = 0;
#pragma unroll
        for (int r = 0; r < S; ++r) {
          gptr[r] = base[r] ? base[r] + first * bytes[r] : nullptr;
          row_bytes += bytes[r];
        }
        auto issue_copies = [&]() {
          if (n_bulk > 0) {
            mbar_expect_tx(&sh->full[slot], (unsigned)(n_bulk * row_bytes));
#pragma unroll
            for (int r = 1; r < S; ++r)
              if (bytes[r])
                bulk_load(smem + page[r] * kPageBytes, gptr[r], (unsigned)(n_bulk * bytes[r]), &sh->full[slot]);
            // Gradients are read once.  When the state of the whole list fits in L2, letting
            // the gradients leave it first keeps the state resident from step to step.  When
            // it does not, the hint makes their lines give way at once instead of ageing out:
            // 1 to 3 % for the plain optimizer, a loss of 2 % with the three or four state
            // arrays of the others (measured), hence the policy's say.
            if (p.state_in_l2 || P::kGradEvictFirstBeyondL2)
              bulk_load_hint(smem + page[0] * kPageBytes, gptr[0], (unsigned)(n_bulk * bytes[0]), &sh->full[slot],
                             grad_policy);
            else
              bulk_load(smem + page[0] * kPageBytes, gptr[0], (unsigned)(n_bulk * bytes[0]), &sh->full[slot]);
          }
        };
        // The tile's barrier completes when its bytes have landed AND the producer has arrived,
        // and it arrives after the descriptor is in place.  For the block's first tile the
        // copies go out before the descriptor is built (the step's start-up latency); for
        // the others after it, which measures better in long steps.
        if (i == 0) issue_copies();
        P::fill_desc(sh->desc[slot], p, meta, cr.tensor, count, n_bulk, page, gptr);
        if (i != 0) issue_copies();
        mbar_arrive(&sh->full[slot]);
        issued = i + 1;
        // With its last tile on the way the block lets the next kernel of the stream go ahead:
        // once every block has said so, blocks of that kernel take over SMs as ours exit, set
        // up and wait (grid_dependency_wait) for this kernel to complete.  Said at the start
        // instead, blocks of the next kernel sit on the early finishers' SMs for a large part
        // of a long step, which measurably slows the blocks still at work.
        if (i == n_my - 1) grid_dependency_launch_dependents();
        cr = cr1;
        cr1 = cr2;
        meta = meta1;
      }
      // Collect the scans of the tiles still in the ring and publish.  The same waits make
      // sure that every copy this block started has landed before the block exits.
      for (int i = oldest; i < issued; ++i) {
        const int os = i % kSlots;
        if (mbar_wait(&sh->empty[os], (unsigned)(i / kSlots) & 1u, &sh->abort_flag))
          take_back<P>(p, acc, now, &sh->scan[os], sh->slot_tensor[os]);
        else
          mbar_wait(&sh->full[os], (unsigned)(i / kSlots) & 1u, &sh->never);
      }
      publish<P>(p, acc, now);
    } else {
      grid_dependency_wait();
    }
  } else {
    // ------------------------------------------------------------------ consumers
    grid_dependency_wait();
    const int ctid = threadIdx.x;
    const int stride = (int)gridDim.x;
    const int n_my = (p.tile_count - (int)blockIdx.x + stride - 1) / stride;
    // Entry ticket (thread 0).  It is drawn after the block's first tile has landed, i.e. after
    // the producer has read the phase word (it arrives on the tile's barrier later than that
    // read returned, and the wait below has seen the arrival); the block that draws the last
    // ticket therefore knows that every block of the step has read the word, and only then
    // moves it on for the next step.  The answer is looked at when the block's tiles are done.
    unsigned int ticket = 0u, ph0 = 0u;
    for (int i = 0; i < n_my; ++i) {
      const int stage = i % kSlots, use = i / kSlots;
      if (!mbar_wait(&sh->full[stage], (unsigned)use & 1u, &sh->abort_flag)) {
        if (lane == 0) {
          sh->abort_flag = 1;
          atomicCAS(p.ws.error, 0u, (unsigned)kErrFullWait);
        }
        break;
      }
      if (i == 0 && threadIdx.x == 0 && p.advance) {
        ph0 = __ldcg(p.ws.phase);
        ticket = atomicAdd(p.ws.phase + 1 + (ph0 >> 8), 1u) + 1u;
      }
      P::consume(&sh->desc[stage], &sh->scan[stage], smem, ctid, lane);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[stage]);
    }
    if (threadIdx.x == 0 && ticket == gridDim.x) {
      p.ws.phase[1] = 0u;
      p.ws.phase[0] = ph0 == 2u ? 0u : ph0 + 1u;
    }
  }
  // Nothing follows: the step is complete when every block's producer has published its
  // scans; the exponents they imply are worked out by the blocks of the next step.
}

}  // namespace ksgd
