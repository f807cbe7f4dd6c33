// Device code of the lazy update (SGD with Kahan summation, Algorithm 1 of
// arXiv 1810.05486) in dynamic fixed-point, for sm_100a.
//
// One launch of ksgd_step_kernel performs, for a ragged list of tensors:
//   - Algorithm 1, statement 1: the fp32 gradient increment is rounded onto the
//     compensation grid (one binary32 multiply + round-to-nearest-even);
//   - statements 2-4: T = theta + c - d is formed exactly in integers, rounded onto
//     theta's grid (theta'), and what the rounding lost is stored back as c';
//   - the per-tensor max scans that dynamic fixed-point needs to choose the next
//     exponent (Section 5): registers -> warp reduce -> one atomicMax per warp and tensor;
//   - the exponent choice for every tensor, made by the blocks of the NEXT step from the
//     finished scans (rotating buffers, see Workspace): no block is ever the last one.
// The pass is bound by HBM traffic: 2*m/8 + 2*n/8 + 4 bytes per parameter.
//
// Structure: a persistent grid, one block per SM.  The tensor list is cut into tiles of
// kChunk elements (2 * kChunk for 8-bit theta in long lists); block b takes tiles b,
// b + gridDim.x, ....  One producer thread streams the tiles of theta, c and g into a 224 KB shared-memory ring with bulk
// asynchronous copies (cp.async.bulk, completion counted on an mbarrier), so the bytes in
// flight do not depend on registers or occupancy; a tile takes only the pages its format
// needs (6 for int8/int8 -- 12 with the large tiles --, 8 for int16/int16), so two to four
// tiles are resident.
// Sixteen consumer warps compute from shared memory and store theta' and c' straight to
// global memory with 16-byte stores.
// No block ever waits for another block; every wait inside a block is bounded.
//
// State between steps.  The per-tensor state a step leaves behind (the exponent it wrote,
// its max scans) lives in three rotating buffers indexed by the step's phase p = step mod 3
// (a word in the workspace).  Step p reads buffer p-1 (exponent of the stored mantissas,
// finished scans), derives from it the exponent it writes (every block that meets a tensor
// derives the same value and stores it into buffer p: idempotent), accumulates its own scans
// into buffer p, and clears buffer p+1, which nobody reads or writes until the next step.
// So a step needs no pass "after all blocks are done": the kernel ends when each block has
// published its scans, and the next launch finds everything it needs.  The phase word is
// advanced by the block that draws the last entry ticket, i.e. after every block of the
// step has read it.
#pragma once

#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

namespace ksgd {

constexpr int kChunk = 8192;           // elements per tile (twice as many for 8-bit theta in long lists)
constexpr long long kBigTileMinTiles = 1024;   // a list gets the large 8-bit tiles if it still has this many tiles
constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kBlockThreads = kConsumers + 32;   // + one producer warp
constexpr int kSlots = 6;              // tiles a block can have in its ring at once
constexpr int kPageBytes = 8192;       // the ring is handed out in pages
static_assert(kChunk == 8192 && kPageBytes == kChunk, "the producer's page arithmetic assumes 8192-element tiles and 8 KB pages");
constexpr int kPages = 28;             // 224 KB of tile data per block
constexpr int kInlineArgs = 256;     // lists up to this long pass grads/lrs as kernel parameters
constexpr int kUploadBatch = 1024;   // tensors per launch of the argument-upload kernel
constexpr int kDLimit = 1 << 30;     // clamp of the quantized increment, in compensation LSBs
constexpr int kMaxDelta = 8;         // largest exponent change per step
constexpr int kExpMin = -64, kExpMax = 64;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a barrier wait gives up after 2 s

enum DeviceError { kErrNone = 0, kErrFullWait = 1, kErrEmptyWait = 2 };

struct TensorInfo {
  void* theta;
  void* comp;
  long long numel;
  int theta_bits;
  int comp_bits;
  int s;       // grid distance: exp_comp = exp_theta - s  (0 in plain mode)
  int pad;
};

struct ChunkRef {
  int tensor;  // index into the tensor list
  int index;   // tile number inside that tensor: elements [index*chunk, ...), chunk = the tensor's tile size
};

// Device-side view of the caller's workspace.
// What a step leaves behind for one tensor: everything the next step needs to know about it,
// in one 32-byte record (one load).
struct __align__(32) TensorState {
  int exp_theta;          // exponent of theta's mantissas as this step wrote them
  int exp_comp;           // strict mode: the same for the compensation's own exponent
  unsigned int amax_t;    // this step's max scans (blocks add to them while the step runs)
  unsigned int amax_c;
  int ovr_theta;          // exponent the NEXT step must write instead of the one the scans give:
  int ovr_comp;           //   value + kOvrBias, 0 = none (init, kahan_sgd_set_exponents; comp: init only)
  int pad[2];
};

struct Workspace {
  unsigned int* phase;             // [0] phase of the coming step (0..2); [1] entry tickets drawn in the running step
  // [3][slab] records, one slab per phase; a slab starts on a 128-byte boundary, so that the
  // slab all blocks add their scans to shares no cache line with the one they read.
  TensorState* state;
  int slab;                        // records per slab
  unsigned long long* counters;    // [3n] cumulative: sat_theta | sat_comp | nonfinite
  unsigned int* error;             // [1] first DeviceError seen (0 = none), sticky
  TensorInfo* info;                // [n]
  const float** grad_ptr;          // [n] per-step arguments for lists longer than kInlineArgs
  float* lr;                       // [n]
  int* exp_grad;                   // [n] the same, exponents of fixed-point gradients
  ChunkRef* chunks;                // [n_chunks]
};
constexpr int kOvrBias = 1000;

struct StepParams {
  Workspace ws;
  int n_tensors;
  int n_chunks;
  int amax_mode;     // 1: exponents follow the max scan, 0: fixed
  int inline_args;   // 1: grads/lrs are in the InlineArgs parameter
  int grad_evict_first;  // 1: gradient loads carry the L2 evict-first hint
  const int* exp_grad_dev;   // fixed-point gradients: device array of their exponents (as a scan on the
                             // device left them), or nullptr: the exponents come with the per-step arguments
  int advance;           // 1: this launch ends a step (the phase word moves on); 0: more launches of the
                         //    same step follow (the host-buffer entry point updates groups of tensors in turn)
  // The launch covers tiles [tile_begin, tile_begin + tile_count), which are all the tiles
  // of tensors [tensor_begin, tensor_begin + tensor_count): the whole list for an ordinary
  // step, one group of tensors when the host-buffer entry point pipelines its copies.
  int tile_begin, tile_count, tensor_begin, tensor_count;
  // Elements per tile of tensors with 8-bit theta: kChunk, or 2 * kChunk for lists long
  // enough to keep every block busy with the larger tiles (one vector per thread and tile
  // leaves the per-tile work of a consumer -- wait, descriptor, scans, arrive -- a third of
  // its instructions).  Tensors with 16-bit theta always take kChunk.
  int chunk8;
};

struct InlineArgs {
  const float* grads[kInlineArgs];
  float lrs[kInlineArgs];
};

// Per-step arguments when the gradients are dynamic fixed-point tensors themselves (8- or
// 16-bit mantissas, one exponent per tensor).
struct QGradArgs {
  const void* grads[kInlineArgs];
  float lrs[kInlineArgs];
  signed char exp_grad[kInlineArgs];
};

struct UploadBatch {
  const float* grads[kUploadBatch];
  float lrs[kUploadBatch];
};

struct ExponentBatch {
  int exp_next[kUploadBatch];
};

// What the consumers need to know about a tensor for this step.
struct StepCoef {
  float scale;   // lr * 2^-(e_out - s): gradient -> compensation LSBs of the output grid
  int s;         // grid distance
  int delta;     // e_out - e_in
  int sh_t;      // theta mantissa  -> fine grid
  int sh_c;      // comp mantissa   -> fine grid
  int sh_d;      // increment       -> fine grid
  int r_t;       // fine grid -> theta output grid (rounding shift)
  int r_c;       // fine grid -> comp output grid (rounding shift)
  int qmax_t;    // 2^(m-1) - 1
  int qmax_c;    // 2^(n-1) - 1
  int gb;        // gradient storage: 32 = binary32, 8 / 16 = fixed-point mantissas
  int eg;        // exponent of fixed-point gradient mantissas (0 for binary32)
  int strict;    // 1: every statement of Algorithm 1 rounds into the stored format
  int delta_c;   // ec_out - ec_in
};

// One tile as the producer describes it to the consumers (lives in shared memory).  The
// first 48 bytes are all the steady-state path reads (three 16-byte loads).
struct __align__(16) TileDesc {
  float scale;          // lr * 2^-(e_out - s), times 2^eg for fixed-point gradients
  float pow2s_neg;      // -2^s
  float inv2s;          // 2^-s
  float pow2dc;         // strict mode: 2^(ec_in - ec_out), c's old units in new ones; else 1
  void* theta;          // global address of the tile's first theta mantissa
  void* comp;           // same for the compensation (unused in plain mode)
  int tensor;
  int n_bulk;           // elements that arrived through the bulk copies (multiple of 16)
  int count;            // valid elements in the tile
  int flags;            // kFlag* | format id
  StepCoef coef;        // for the general path
  const void* grad;     // global address of the tile's first gradient
};
constexpr int kFlagFormatMask = 7;   // 0..5 = (8,0) (8,8) (8,16) (16,0) (16,8) (16,16)
constexpr int kFlagSteady = 8;       // no exponent change: the exact-fp32 path applies
constexpr int kFlagRegrid = 16;      // theta's exponent changes: the exact-fp32 re-gridding path applies
constexpr int kFlagThetaPageShift = 8;   // 5 bits each: first ring page of theta, c, g
constexpr int kFlagCompPageShift = 13;
constexpr int kFlagGradPageShift = 18;

// Max scans and counters of one tile, gathered in shared memory: the consumer warps add to
// it, the producer publishes it when it takes the tile's stage back.
struct TileScan {
  unsigned int amax_t, amax_c, n_sat_t, n_sat_c, n_nonfinite, pad[3];
};

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
// Arithmetic

__device__ __forceinline__ float pow2_float(int e) {  // exact 2^e for e in [-126, 127]
  return __int_as_float((e + 127) << 23);
}

// a / 2^r, round to nearest, ties to even (|a| < 2^62).
__device__ __forceinline__ long long rne_shift64(long long a, int r) {
  if (r == 0) return a;
  const long long bias = ((1LL << (r - 1)) - 1) + ((a >> r) & 1LL);
  return (a + bias) >> r;
}

__device__ __forceinline__ int quantize_increment(float g, float scale) {
  const float x = __fmul_rn(g, scale);   // one binary32 multiply, never contracted
  int d = __float2int_rn(x);             // nearest-even; saturates; NaN -> 0
  return max(min(d, kDLimit), -kDLimit);
}

// Shifts between the four grids of a step (theta's and c's, each read at *_in and written at
// *_out) and the finest of them, f.  In the ordinary mode c's exponent is tied to theta's
// (ec = e - s); in strict mode it is the tensor's own.
__device__ __forceinline__ StepCoef make_coef(const TensorInfo& ti, int e_in, int e_out, int ec_in, int ec_out,
                                              float lr, int gb, int eg, int strict) {
  StepCoef k;
  k.gb = gb;
  k.eg = eg;
  k.strict = strict;
  const int f = min(min(e_in, e_out), min(ec_in, ec_out));
  k.s = e_out - ec_out;
  k.delta = e_out - e_in;
  k.delta_c = ec_out - ec_in;
  k.sh_t = e_in - f;
  k.sh_c = ec_in - f;
  k.sh_d = ec_out - f;
  k.r_t = e_out - f;
  k.r_c = ec_out - f;
  k.qmax_t = (1 << (ti.theta_bits - 1)) - 1;
  k.qmax_c = ti.comp_bits ? (1 << (ti.comp_bits - 1)) - 1 : 0;
  k.scale = __fmul_rn(lr, pow2_float(-ec_out));   // |ec_out| <= 100: exact power of two
  return k;
}

// Algorithm 1 for elements [first, first+n) with 64-bit intermediates, in place on arrays
// that may live in a shared-memory stage or in global memory.  This is the general path:
// exponent changes, vectors in which theta saturates or a gradient is not finite (or very
// large), and ragged tails.  It is kept out of line, one copy for all formats, so that it
// costs the steady-state path no registers.
__device__ __noinline__ void update_general(const StepCoef* coef, int tb, int cb, void* theta,
                                            void* comp, const void* grad, int first, int n,
                                            TileScan* slots) {
  const StepCoef k = *coef;
  unsigned int amax_t = 0, amax_c = 0, n_sat_t = 0, n_sat_c = 0, n_nf = 0;
#pragma unroll 1
  for (int e = first; e < first + n; ++e) {
    const int qt = tb == 8 ? (int)static_cast<const signed char*>(theta)[e]
                           : (int)static_cast<const short*>(theta)[e];
    int qc = 0;
    if (cb == 8) qc = (int)static_cast<const signed char*>(comp)[e];
    else if (cb == 16) qc = (int)static_cast<const short*>(comp)[e];
    float g;       // a fixed-point gradient Q * 2^eg is exact in binary32
    if (k.gb == 32) g = static_cast<const float*>(grad)[e];
    else if (k.gb == 8) g = __fmul_rn((float)static_cast<const signed char*>(grad)[e], pow2_float(k.eg));
    else g = __fmul_rn((float)static_cast<const short*>(grad)[e], pow2_float(k.eg));
    const int d = quantize_increment(g, k.scale);
    long long T;
    if (k.strict) {
      // statement 1 rounds into the n-bit accumulator before theta sees it
      const long long C1 = rne_shift64((long long)qc * (1LL << k.sh_c) - (long long)d * (1LL << k.sh_d), k.r_c);
      const long long C1c = C1 > k.qmax_c ? k.qmax_c : (C1 < -k.qmax_c ? -k.qmax_c : C1);
      unsigned long long a1 = (unsigned long long)(C1 < 0 ? -C1 : C1);
      if (a1 > 0x7fffffffULL) a1 = 0x7fffffffULL;
      amax_c = max(amax_c, (unsigned int)a1);
      n_sat_c += (C1 != C1c);
      T = (long long)qt * (1LL << k.sh_t) + C1c * (1LL << k.r_c);
    } else {
      T = (long long)qt * (1LL << k.sh_t) + (long long)qc * (1LL << k.sh_c) - (long long)d * (1LL << k.sh_d);
    }
    const long long P = rne_shift64(T, k.r_t);
    const long long Pc = P > k.qmax_t ? k.qmax_t : (P < -k.qmax_t ? -k.qmax_t : P);
    unsigned long long aP = (unsigned long long)(P < 0 ? -P : P);
    if (aP > 0x7fffffffULL) aP = 0x7fffffffULL;
    amax_t = max(amax_t, (unsigned int)aP);
    n_sat_t += (P != Pc);
    if (tb == 8) static_cast<signed char*>(theta)[e] = (signed char)Pc;
    else static_cast<short*>(theta)[e] = (short)Pc;
    if (cb) {
      const long long R = T - Pc * (1LL << k.r_t);
      const long long Rq = rne_shift64(R, k.r_c);
      const long long Rc = Rq > k.qmax_c ? k.qmax_c : (Rq < -k.qmax_c ? -k.qmax_c : Rq);
      unsigned long long aR = (unsigned long long)(Rq < 0 ? -Rq : Rq);
      if (aR > 0x7fffffffULL) aR = 0x7fffffffULL;
      amax_c = max(amax_c, (unsigned int)aR);
      n_sat_c += (Rq != Rc);
      if (cb == 8) static_cast<signed char*>(comp)[e] = (signed char)Rc;
      else static_cast<short*>(comp)[e] = (short)Rc;
    }
    n_nf += ((__float_as_uint(g) & 0x7f800000u) == 0x7f800000u);
  }
  if (amax_t) atomicMax(&slots->amax_t, amax_t);
  if (amax_c) atomicMax(&slots->amax_c, amax_c);
  if (n_sat_t) atomicAdd(&slots->n_sat_t, n_sat_t);
  if (n_sat_c) atomicAdd(&slots->n_sat_c, n_sat_c);
  if (n_nf) atomicAdd(&slots->n_nonfinite, n_nf);
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
// Steady state (no exponent change): one vector of V elements on the FP32 pipe, used as an
// exact integer unit.  With M = 1.5 * 2^23 every float in [2^23, 2^24) is an integer whose
// low mantissa bits are that integer in two's complement relative to M, an addition that
// lands there rounds to nearest-even on the integer grid, and sums, differences and FMAs
// of integers below 2^24 are exact.  Per element:
//   qtM = M + qt, qcM = M + qc          the signed mantissa added to M's bit pattern by one
//                                         integer dot-product instruction (magic_signed)
//   y   = g*scale + M                   = M + d, d = rne(g*scale)            (stmt 1)
//   u   = qcM - y                       = qc - d
//   Pb  = fma(u, 2^-s, qtM)             = M + rne((qt*2^s + u) / 2^s) = M + P
//                                         (stmt 2; M is even, so the tie falls on the parity
//                                         of P itself)
//   w   = Pb - qtM                      = P - qt
//   r0  = fma(w, -2^s, u)               = T - P*2^s                       (stmt 3)
// theta' is the low bits of Pb (two's complement of P under M's exponent), c' the low bits
// of r0 + M.
// The vector is handed to update_general instead (returns false, nothing stored) when some
// |g*scale| exceeds 4e6 (y must stay below 2^24) or is Inf or NaN, or some |P| exceeds QMAX:
// exactly the cases in which the magnitudes above could leave the exact range or a clamp is
// needed.

// Strict mode (STRICT): u is statement 1's rounded result C1 = rne(qc * 2^(ec_in-ec_out) - d),
// formed by one FMA onto M - d, so a change of c's exponent stays on this path; the vector
// also leaves the path when |C1| or |r0| exceeds c's n bits (the clamps of statements 1, 3).

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

struct SteadyCoef {
  float scale;      // lr * 2^-(e - s)
  float pow2s_neg;  // -2^s
  float inv2s;      // 2^-s
  float pow2dc;     // 2^(ec_in - ec_out) (strict mode)
};

struct TileHot {       // the consumers' copy of the first 48 bytes of a TileDesc
  SteadyCoef k;
  unsigned char* theta;
  unsigned char* comp;
  int tensor, n_bulk, count, flags;
};

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

// The scans take two elements per instruction: the largest and smallest Pb give max|P|, and
// |x|, |r0| go through three-input maxima.
template <int TB, int CB, int V, int GB, bool STRICT>
__device__ __forceinline__ bool update_vector(const Pack<V * TB / 8>& pt, const Pack<(CB ? V * CB / 8 : 8)>& pc,
                                              const Pack<V * GB / 8>& pg, const SteadyCoef& k,
                                              Pack<V * TB / 8>& ot, Pack<(CB ? V * CB / 8 : 8)>& oc,
                                              float& amax_t, float& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int CBS = CB ? CB : 8;
  constexpr int GBS = GB == 32 ? 8 : GB;
  float Pm[V], rm[V], xa[2], ra[2], ua[2];
  float aX = 0.0f, hiP = kMagic, loP = kMagic, aR = 0.0f, aU = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const float qtM = magic_signed<TB>(pt, i);
    float g;       // binary32 gradient, or the gradient mantissa (k.scale then carries 2^eg)
    if constexpr (GB == 32) g = __uint_as_float(pack_word(pg, i));
    else g = __fadd_rn(magic_signed<GBS>(pg, i), -kMagic);
    const float x = __fmul_rn(g, k.scale);              // the one binary32 multiply
    float u;
    if constexpr (STRICT) {
      // statement 1 with c's own exponent: C1 = rne(Q_c * 2^(ec_in-ec_out) - d), one rounding
      // (the FMA lands in [2^23, 2^24), where floats are the integers)
      const float d = __fadd_rn(__fadd_rn(x, kMagic), -kMagic);
      const float qc = __fadd_rn(magic_signed<CBS>(pc, i), -kMagic);
      u = __fadd_rn(__fmaf_rn(qc, k.pow2dc, __fadd_rn(kMagic, -d)), -kMagic);
    } else {
      const float y = __fadd_rn(x, kMagic);               // rounds x to nearest-even integer
      if constexpr (HAS_COMP) u = __fadd_rn(magic_signed<CBS>(pc, i), -y);
      else u = __fadd_rn(kMagic, -y);
    }
    const float P = __fmaf_rn(u, k.inv2s, qtM);
    const float w = __fadd_rn(P, -qtM);
    const float r0 = __fmaf_rn(w, k.pow2s_neg, u);
    Pm[i] = P;
    rm[i] = __fadd_rn(r0, kMagic);
    xa[i & 1] = fabsf(x);
    ra[i & 1] = fabsf(r0);
    ua[i & 1] = fabsf(u);
    if (i & 1) {
      aX = max3_nan(aX, xa[0], xa[1]);                  // NaN if any product is
      hiP = max3(hiP, Pm[i - 1], P);
      loP = min3(loP, Pm[i - 1], P);
      if constexpr (HAS_COMP) aR = max3(aR, ra[0], ra[1]);
      if constexpr (STRICT) aU = max3(aU, ua[0], ua[1]);  // u = c - d is statement 1's result
    }
  }
  const float aP = fmaxf(__fadd_rn(hiP, -kMagic), __fadd_rn(kMagic, -loP));
  constexpr float qmax_t = (float)((1 << (TB - 1)) - 1);
  if (!(aX <= 4000000.0f) | (aP > qmax_t)) return false;   // also Inf and NaN products
  if constexpr (STRICT) {
    // both accumulator results must fit their n bits, or the vector needs the clamps
    constexpr float qmax_c = (float)((1 << (CBS - 1)) - 1);
    aR = fmaxf(aR, aU);
    if (aR > qmax_c) return false;
  }
  amax_t = fmaxf(amax_t, aP);
  if constexpr (HAS_COMP) amax_c = fmaxf(amax_c, aR);
  ot = pack_magic<TB, V>(Pm);
  if constexpr (HAS_COMP) oc = pack_magic<CB, V>(rm);
  return true;
}

// The step in which theta's exponent changes by delta = e_out - e_in (ordinary mode: c's grid
// moves with theta's), again on the FP32 pipe with every intermediate an exact integer below
// 2^24.  k.pow2dc = 2^-delta.  d = rne(g*scale) is on the output compensation grid as always.
//
// Finer grid (delta < 0, a = -delta): the stored mantissas scale up exactly,
//   base = M + qt*2^a (both even, so exact even beyond 2^24),  u = qc*2^a - d,
//   Pb = fma(u, 2^-s, base) = M + P,  w = Pb - base,  r0 = fma(w, -2^s, u) = Rq  (no second rounding).
// Coarser grid (delta > 0, a = delta, s' = s + a): theta's mantissa is split with two integer
// operations per packed word, qt = A*2^a + B with 0 <= B < 2^a (on the sign-flipped lanes the
// split is a logical shift and a mask), so that
//   T = A*2^s' + v,  v = B*2^s + qc - d*2^a   (exact: |d|*2^a <= 4e6 is checked)
//   Pb = fma(v, 2^-s', M + A) = M + P,  w = Pb - (M + A),  R = fma(w, -2^s', v),
//   Rm = fma(R, 2^-a, M) = M + Rq   (the second rounding of the coarser grid, ties on Rq's parity).
// In both cases |Rq| <= 2^(s-1) whenever P needs no clamp, so c never clamps on this path.
// Returns false (nothing stored: the vector goes to update_general) when some product is too
// large, Inf or NaN, or some |P| exceeds QMAX.  A coarser change needs a <= TB - 1 (the
// producer checks).
template <int TB, int CB, int V, int GB>
__device__ __forceinline__ bool update_vector_regrid(Pack<V * TB / 8> pt, Pack<(CB ? V * CB / 8 : 8)> pc,
                                                     Pack<V * GB / 8> pg, const SteadyCoef& k,
                                                     Pack<V * TB / 8>& ot, Pack<(CB ? V * CB / 8 : 8)>& oc,
                                                     float& amax_t, float& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int CBS = CB ? CB : 8;
  constexpr int GBS = GB == 32 ? 8 : GB;
  constexpr float bias_t = (float)(1 << (TB - 1));
  const bool finer = k.pow2dc > 1.0f;
  // 2^a and 2^-a
  const float up = finer ? k.pow2dc : __int_as_float(0x7f000000 - __float_as_int(k.pow2dc));
  const float down = finer ? __int_as_float(0x7f000000 - __float_as_int(k.pow2dc)) : k.pow2dc;
  Pack<V * TB / 8> pA = pt, pB = pt;
  float inv2sp = k.inv2s, pow2sp_neg = k.pow2s_neg, biasA = bias_t, pow2s = -k.pow2s_neg;
  if (!finer) {
    // split on the sign-flipped (unsigned) lanes: a logical shift and a mask per word
    flip_signs<TB>(pA);
    const int a = 127 - (int)(__float_as_uint(k.pow2dc) >> 23);
    constexpr unsigned int lanes = TB == 8 ? 0x01010101u : 0x00010001u;
    constexpr unsigned int full = TB == 8 ? 0xffu : 0xffffu;
    const unsigned int maskA = (full >> a) * lanes, maskB = ((1u << a) - 1u) * lanes;
#pragma unroll
    for (int w = 0; w < V * TB / 32; ++w) {
      const unsigned int x = pack_word(pA, w);
      set_pack_word(pA, w, (x >> a) & maskA);
      set_pack_word(pB, w, x & maskB);
    }
    inv2sp = __fmul_rn(k.inv2s, down);          // 2^-s'
    pow2sp_neg = __fmul_rn(k.pow2s_neg, up);    // -2^s'
    biasA = __fmul_rn(bias_t, down);            // what the shifted lanes still carry of the sign flip
  }
  float Pm[V], rm[V], xa[2], ra[2];
  float aX = 0.0f, hiP = kMagic, loP = kMagic, aR = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    float g;
    if constexpr (GB == 32) g = __uint_as_float(pack_word(pg, i));
    else g = __fadd_rn(magic_signed<GBS>(pg, i), -kMagic);
    const float x = __fmul_rn(g, k.scale);              // the one binary32 multiply
    const float y = __fadd_rn(x, kMagic);               // M + d
    float qc = 0.0f;
    if constexpr (HAS_COMP) qc = __fadd_rn(magic_signed<CBS>(pc, i), -kMagic);
    float P, r;
    if (finer) {
      const float qt = __fadd_rn(magic_signed<TB>(pt, i), -kMagic);
      const float base = __fmaf_rn(qt, up, kMagic);
      const float u = __fmaf_rn(qc, up, __fadd_rn(kMagic, -y));
      P = __fmaf_rn(u, inv2sp, base);
      const float w = __fadd_rn(P, -base);
      r = __fmaf_rn(w, pow2sp_neg, u);
      rm[i] = __fadd_rn(r, kMagic);
    } else {
      const float base = __fadd_rn(magic_elem<TB>(pA, i), -biasA);       // M + A
      const float B = __fadd_rn(magic_elem<TB>(pB, i), -kMagic);
      const float d = __fadd_rn(y, -kMagic);
      const float v = __fmaf_rn(d, -up, __fmaf_rn(B, pow2s, qc));
      P = __fmaf_rn(v, inv2sp, base);
      const float w = __fadd_rn(P, -base);
      const float R = __fmaf_rn(w, pow2sp_neg, v);
      rm[i] = __fmaf_rn(R, down, kMagic);
      r = __fadd_rn(rm[i], -kMagic);
    }
    Pm[i] = P;
    xa[i & 1] = fabsf(x);
    ra[i & 1] = fabsf(r);
    if (i & 1) {
      aX = max3_nan(aX, xa[0], xa[1]);                  // NaN if any product is
      hiP = max3(hiP, Pm[i - 1], P);
      loP = min3(loP, Pm[i - 1], P);
      if constexpr (HAS_COMP) aR = max3(aR, ra[0], ra[1]);
    }
  }
  const float aP = fmaxf(__fadd_rn(hiP, -kMagic), __fadd_rn(kMagic, -loP));
  constexpr float qmax_t = (float)((1 << (TB - 1)) - 1);
  const float x_limit = finer ? 4000000.0f : __fmul_rn(4000000.0f, down);   // |d| * 2^a stays exact
  if (!(aX <= x_limit) | (aP > qmax_t)) return false;   // also Inf and NaN products
  amax_t = fmaxf(amax_t, aP);
  if constexpr (HAS_COMP) amax_c = fmaxf(amax_c, aR);
  ot = pack_magic<TB, V>(Pm);
  if constexpr (HAS_COMP) oc = pack_magic<CB, V>(rm);
  return true;
}

// All vectors of one tile that belong to this consumer thread (V consecutive elements,
// 16 bytes of theta, per vector).  Returns true if the general path wrote into the stage.
template <int TB, int CB, int GB, bool STRICT>
__device__ __forceinline__ bool consume_tile(const TileHot& h, const TileDesc* td, unsigned char* ring,
                                             int ctid, TileScan* slots, float& amax_t, float& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int V = (TB == 8) ? 16 : 8;
  constexpr int TBYTES = V * TB / 8;
  constexpr int CBYTES = HAS_COMP ? V * CB / 8 : 8;
  constexpr int GBYTES = V * GB / 8;
  const bool steady = (h.flags & kFlagSteady) != 0;
  unsigned char* theta_s = ring + ((h.flags >> kFlagThetaPageShift) & 31) * kPageBytes;
  unsigned char* comp_s = ring + ((h.flags >> kFlagCompPageShift) & 31) * kPageBytes;
  const unsigned char* grad_s = ring + ((h.flags >> kFlagGradPageShift) & 31) * kPageBytes;
  bool wrote_stage = false;
  const int n_vec = h.n_bulk / V;
  for (int v = ctid; v < n_vec; v += kConsumers) {
    Pack<TBYTES> ot;
    Pack<CBYTES> oc;
    bool done = false;
    if (steady) {
      const Pack<TBYTES> pt = load_pack<TBYTES>(theta_s + v * TBYTES);
      Pack<CBYTES> pc{};
      if constexpr (HAS_COMP) pc = load_pack<CBYTES>(comp_s + v * CBYTES);
      const Pack<GBYTES> pg = load_pack<GBYTES>(grad_s + v * GBYTES);
      done = update_vector<TB, CB, V, GB, STRICT>(pt, pc, pg, h.k, ot, oc, amax_t, amax_c);
    }
    if (!done) {
      // general path, in place in the stage; then the vector goes out like any other
      update_general(&td->coef, TB, CB, theta_s, comp_s, grad_s, v * V, V, slots);
      ot = load_pack<TBYTES>(theta_s + v * TBYTES);
      if constexpr (HAS_COMP) oc = load_pack<CBYTES>(comp_s + v * CBYTES);
      wrote_stage = true;
    }
    store_pack<TBYTES>(h.theta + (size_t)v * TBYTES, ot);
    if constexpr (HAS_COMP) store_pack<CBYTES>(h.comp + (size_t)v * CBYTES, oc);
  }
  // ragged tail (fewer than 16 elements) that the bulk copies did not bring: in place in
  // global memory
  const int e = h.n_bulk + ctid;
  if (e < h.count) update_general(&td->coef, TB, CB, h.theta, h.comp, td->grad, e, 1, slots);
  return wrote_stage;
}

// Add a consumer warp's steady-path scans of the tile it just finished to the tile's slot.
__device__ __forceinline__ void add_warp_scans(TileScan* scan, int lane, float& amax_t, float& amax_c) {
  const unsigned int full = 0xffffffffu;
  // the steady path's scans are exact integers below 2^23 held in floats
  const unsigned int at = __reduce_max_sync(full, (unsigned int)amax_t);
  const unsigned int ac = __reduce_max_sync(full, (unsigned int)amax_c);
  amax_t = 0.0f;
  amax_c = 0.0f;
  if (lane == 0) {
    if (at) atomicMax(&scan->amax_t, at);
    if (ac) atomicMax(&scan->amax_c, ac);
  }
}

// A whole tile of a tensor whose exponent changes in this step, for one consumer thread:
// update_vector_regrid per vector (update_general for the vectors it declines), stores, the
// ragged tail, and the warp's scans added to the tile's slot.  Kept out of line, like update_general: it is called once per
// tile with next to nothing live around the call, and the registers its arithmetic needs
// then cost the tiles whose exponent does not change (the common case, inline in the
// kernel) nothing.
template <int TB, int CB, int GB>
__device__ __forceinline__ bool regrid_tile_format(const TileHot& h, const TileDesc* td, unsigned char* ring,
                                                   int ctid, TileScan* slots, float& amax_t, float& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int V = (TB == 8) ? 16 : 8;
  constexpr int TBYTES = V * TB / 8;
  constexpr int CBYTES = HAS_COMP ? V * CB / 8 : 8;
  constexpr int GBYTES = V * GB / 8;
  unsigned char* theta_s = ring + ((h.flags >> kFlagThetaPageShift) & 31) * kPageBytes;
  unsigned char* comp_s = ring + ((h.flags >> kFlagCompPageShift) & 31) * kPageBytes;
  const unsigned char* grad_s = ring + ((h.flags >> kFlagGradPageShift) & 31) * kPageBytes;
  bool wrote_stage = false;
  const int n_vec = h.n_bulk / V;
  for (int v = ctid; v < n_vec; v += kConsumers) {
    Pack<TBYTES> ot;
    Pack<CBYTES> oc;
    const Pack<TBYTES> pt = load_pack<TBYTES>(theta_s + v * TBYTES);
    Pack<CBYTES> pc{};
    if constexpr (HAS_COMP) pc = load_pack<CBYTES>(comp_s + v * CBYTES);
    const Pack<GBYTES> pg = load_pack<GBYTES>(grad_s + v * GBYTES);
    if (!update_vector_regrid<TB, CB, V, GB>(pt, pc, pg, h.k, ot, oc, amax_t, amax_c)) {
      update_general(&td->coef, TB, CB, theta_s, comp_s, grad_s, v * V, V, slots);
      ot = load_pack<TBYTES>(theta_s + v * TBYTES);
      if constexpr (HAS_COMP) oc = load_pack<CBYTES>(comp_s + v * CBYTES);
      wrote_stage = true;
    }
    store_pack<TBYTES>(h.theta + (size_t)v * TBYTES, ot);
    if constexpr (HAS_COMP) store_pack<CBYTES>(h.comp + (size_t)v * CBYTES, oc);
  }
  const int e = h.n_bulk + ctid;
  if (e < h.count) update_general(&td->coef, TB, CB, h.theta, h.comp, td->grad, e, 1, slots);
  return wrote_stage;
}

__device__ __forceinline__ TileHot load_tile_hot(const TileDesc* td) {
  TileHot h;
  const uint4* q = reinterpret_cast<const uint4*>(td);
  const uint4 q0 = q[0], q1 = q[1], q2 = q[2];
  h.k.scale = __uint_as_float(q0.x);
  h.k.pow2s_neg = __uint_as_float(q0.y);
  h.k.inv2s = __uint_as_float(q0.z);
  h.k.pow2dc = __uint_as_float(q0.w);
  h.theta = reinterpret_cast<unsigned char*>(((unsigned long long)q1.y << 32) | q1.x);
  h.comp = reinterpret_cast<unsigned char*>(((unsigned long long)q1.w << 32) | q1.z);
  h.tensor = (int)q2.x;
  h.n_bulk = (int)q2.y;
  h.count = (int)q2.z;
  h.flags = (int)q2.w;
  return h;
}

template <int GB>
__device__ __noinline__ void regrid_tile(const TileDesc* td, TileScan* slots, unsigned char* ring) {
  const TileHot h = load_tile_hot(td);
  const int ctid = threadIdx.x;
  float amax_t = 0.0f, amax_c = 0.0f;
  bool wrote_stage;
  switch (h.flags & kFlagFormatMask) {
    case 0: wrote_stage = regrid_tile_format<8, 0, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
    case 1: wrote_stage = regrid_tile_format<8, 8, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
    case 2: wrote_stage = regrid_tile_format<8, 16, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
    case 3: wrote_stage = regrid_tile_format<16, 0, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
    case 4: wrote_stage = regrid_tile_format<16, 8, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
    default: wrote_stage = regrid_tile_format<16, 16, GB>(h, td, ring, ctid, slots, amax_t, amax_c); break;
  }
  add_warp_scans(slots, threadIdx.x & 31, amax_t, amax_c);
  // if the general path wrote into the stage, order those writes before the bulk copy that
  // refills it
  if (wrote_stage) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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

// Strict mode: the compensation's own next exponent.  The tight fit of its scan; an empty
// scan (every increment rounded away, or none came) makes the grid 8 binades finer; the
// result stays within [e_next - 36, e_next + 8] of theta's next exponent, which keeps every
// sum of the step within 64 bits.
constexpr int kStrictBelow = 36, kStrictAbove = 8;
__host__ __device__ __forceinline__ int next_exponent_acc(unsigned int amax, int bits, int ec_out, int e_next,
                                                          int amax_mode) {
  int ec = next_exponent(amax, bits, ec_out, amax_mode);
  if (amax_mode && amax == 0u) ec = ec_out - kMaxDelta;
  ec = ec < e_next - kStrictBelow ? e_next - kStrictBelow : (ec > e_next + kStrictAbove ? e_next + kStrictAbove : ec);
  return ec < kExpMin ? kExpMin : (ec > kExpMax ? kExpMax : ec);
}

struct __align__(128) BlockShared {
  unsigned long long full[kSlots];     // producer -> consumers: the tile's bytes have landed
  unsigned long long empty[kSlots];    // consumers -> producer: the tile's pages may be reused
  TileDesc desc[kSlots];
  TileScan scan[kSlots];
  int slot_pages[kSlots];              // ring pages held by the tile in each slot
  int abort_flag;   // set by the first thread whose bounded wait ran out
  int never;        // stays 0: abort flag for waits that must not be cut short
};

constexpr size_t kSharedBytes = (size_t)kPages * kPageBytes + sizeof(BlockShared);

// Producer side: scans of finished tiles are merged per tensor in registers and go to
// global memory when the tensor changes (one set of atomics per block and tensor run).
struct ScanAcc {
  int tensor = -1;
  unsigned int amax_t = 0, amax_c = 0, n_sat_t = 0, n_sat_c = 0, n_nonfinite = 0;
};

__device__ __forceinline__ void publish(const StepParams& p, ScanAcc& acc, TensorState* now) {
  if (acc.tensor >= 0) {
    const int t = acc.tensor, n = p.n_tensors;
    if (acc.amax_t) atomicMax(&now[t].amax_t, acc.amax_t);
    if (acc.amax_c) atomicMax(&now[t].amax_c, acc.amax_c);
    if (acc.n_sat_t) atomicAdd(&p.ws.counters[t], (unsigned long long)acc.n_sat_t);
    if (acc.n_sat_c) atomicAdd(&p.ws.counters[n + t], (unsigned long long)acc.n_sat_c);
    if (acc.n_nonfinite) atomicAdd(&p.ws.counters[2 * n + t], (unsigned long long)acc.n_nonfinite);
  }
  acc = ScanAcc{};
}

__device__ __forceinline__ void take_back(const StepParams& p, ScanAcc& acc, TensorState* now,
                                          TileScan* scan, int tensor) {
  if (tensor != acc.tensor) {
    publish(p, acc, now);
    acc.tensor = tensor;
  }
  acc.amax_t = max(acc.amax_t, scan->amax_t);
  acc.amax_c = max(acc.amax_c, scan->amax_c);
  acc.n_sat_t += scan->n_sat_t;
  acc.n_sat_c += scan->n_sat_c;
  acc.n_nonfinite += scan->n_nonfinite;
  scan->amax_t = scan->amax_c = scan->n_sat_t = scan->n_sat_c = scan->n_nonfinite = 0u;
}

// What the producer reads about a tile's tensor, fetched one tile ahead.
struct TensorMeta {
  TensorInfo ti;
  const void* grad;
  float lr;
  int e_in, e_out;
  int ec_in, ec_out;   // the compensation's exponents: e - s, or its own in strict mode
  int eg;              // exponent of a fixed-point gradient, 0 for binary32
};

// The exponents tensor t reads and writes in the step of phase `ph`, derived from what the
// preceding step left in buffer ph-1; the result goes into buffer ph and buffer ph+1 is cleared
// for the step after this one.  Every block that meets the tensor does the same and stores the
// same values.
__device__ __forceinline__ void step_exponents(const StepParams& p, int t, int ph, bool strict, TensorMeta& m) {
  const int prev = ph == 0 ? 2 : ph - 1;
  // one 32-byte load (L2: the record was written by other SMs during the preceding step)
  const int4* rec = reinterpret_cast<const int4*>(&p.ws.state[(size_t)prev * p.ws.slab + t]);
  const int4 r0 = __ldcg(rec), r1 = __ldcg(rec + 1);
  m.e_in = r0.x;
  m.e_out = r1.x ? r1.x - kOvrBias : next_exponent((unsigned)r0.z, m.ti.theta_bits, m.e_in, p.amax_mode);
  if (strict) {
    m.ec_in = r0.y;
    m.ec_out = r1.y ? r1.y - kOvrBias : next_exponent_acc((unsigned)r0.w, m.ti.comp_bits, m.ec_in, m.e_out, p.amax_mode);
  } else {
    m.ec_in = m.e_in - m.ti.s;
    m.ec_out = m.e_out - m.ti.s;
  }
}

// Every block that meets a tensor derives the same exponents; the one that holds the tensor's
// first tile records them and clears the record of the step after this one.  (This step's
// own record was cleared a step ago; only its exponent fields are written here, the scans
// other blocks may already have added to it stay.)
__device__ __forceinline__ void record_exponents(const StepParams& p, int t, int ph, bool strict,
                                                 const TensorMeta& m) {
  const int next = ph == 2 ? 0 : ph + 1;
  TensorState* now = &p.ws.state[(size_t)ph * p.ws.slab + t];
  now->exp_theta = m.e_out;
  now->exp_comp = strict ? m.ec_out : 0;
  int4* nx = reinterpret_cast<int4*>(&p.ws.state[(size_t)next * p.ws.slab + t]);
  nx[0] = make_int4(0, 0, 0, 0);
  nx[1] = make_int4(0, 0, 0, 0);
}

// ti: the tensor's table entry if the caller has it already (the table never changes).
__device__ __forceinline__ TensorMeta load_meta(const StepParams& p, const InlineArgs& a, int t, int ph, bool strict,
                                                bool owner, const TensorInfo* ti = nullptr) {
  TensorMeta m;
  m.ti = ti ? *ti : p.ws.info[t];
  m.grad = p.inline_args ? a.grads[t] : p.ws.grad_ptr[t];
  m.lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];
  m.eg = 0;
  step_exponents(p, t, ph, strict, m);
  if (owner) record_exponents(p, t, ph, strict, m);
  return m;
}

__device__ __forceinline__ TensorMeta load_meta(const StepParams& p, const QGradArgs& a, int t, int ph, bool strict,
                                                bool owner, const TensorInfo* ti = nullptr) {
  TensorMeta m;
  m.ti = ti ? *ti : p.ws.info[t];
  m.grad = p.inline_args ? a.grads[t] : static_cast<const void*>(p.ws.grad_ptr[t]);
  m.lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];
  if (p.exp_grad_dev) m.eg = max(kExpMin, min(kExpMax, __ldcg(p.exp_grad_dev + t)));
  else m.eg = p.inline_args ? (int)a.exp_grad[t] : p.ws.exp_grad[t];
  step_exponents(p, t, ph, strict, m);
  if (owner) record_exponents(p, t, ph, strict, m);
  return m;
}

// The whole step.  GB = 32: binary32 gradients; 8 / 16: fixed-point gradients (one or two
// bytes per parameter instead of four on the gradient stream).
// STRICT: every statement of Algorithm 1 rounds into the stored format and the compensation
// has its own exponent (comp_bits != 0 for every tensor).
template <int GB, bool STRICT, typename Args>
__device__ __forceinline__ void step_body(const StepParams& p, const Args& a) {
  extern __shared__ __align__(128) unsigned char smem[];
  BlockShared* sh = reinterpret_cast<BlockShared*>(smem + (size_t)kPages * kPageBytes);
  grid_dependency_launch_dependents();   // the next step's blocks may take over SMs as ours exit

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&sh->full[s], 1u);
      mbar_init(&sh->empty[s], (unsigned)kConsumerWarps);
    }
    sh->abort_flag = 0;
    sh->never = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kSlots * (int)(sizeof(TileScan) / 4))
    reinterpret_cast<unsigned int*>(sh->scan)[threadIdx.x] = 0u;
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    // Block b takes tiles b, b + gridDim.x, ...: neighbouring tiles run on neighbouring
    // SMs at the same time, and the tiles of a tensor that needs the general path are
    // spread evenly over all blocks.  Table entries are fetched two tiles ahead and the
    // tensor's data one tile ahead, so none of these loads sits between a freed stage and
    // the copy that refills it.
    if (lane == 0) {
      const int stride = (int)gridDim.x;
      const int n_my = (p.tile_count - (int)blockIdx.x + stride - 1) / stride;
      const int tile0 = p.tile_begin + (int)blockIdx.x;
      const unsigned long long grad_policy = l2_policy_evict_first();
      ScanAcc acc;
      // the tile table is written once at init: read the first entries before waiting for
      // the preceding kernel
      ChunkRef cr = p.ws.chunks[tile0];
      ChunkRef cr1{-1, -1};
      if (n_my > 1) cr1 = p.ws.chunks[tile0 + stride];
      const TensorInfo ti_first = p.ws.info[cr.tensor];       // the tensor table never changes either
      // The step's phase.  The preceding step moves the word on as soon as all of its blocks
      // have started, long before it ends, so the value read here, before the wait, is
      // normally the right one already: the first record is fetched under it while the word
      // is read again, and only fetched a second time if the two differ.  (The block's entry
      // ticket, which tells the last block that all have read this word, is drawn by a
      // consumer thread once the first tile has landed.)
      int ph = (int)__ldcg(p.ws.phase);
      grid_dependency_wait();
      const int ph_now = (int)__ldcg(p.ws.phase);
      TensorMeta meta = load_meta(p, a, cr.tensor, ph, STRICT, false, &ti_first);
      if (ph_now != ph) {
        ph = ph_now;
        meta = load_meta(p, a, cr.tensor, ph, STRICT, false, &ti_first);
      }
      if (cr.index == 0) record_exponents(p, cr.tensor, ph, STRICT, meta);
      TensorState* amax_now = p.ws.state + (size_t)ph * p.ws.slab;
      int issued = 0;
      // The ring: pages from `head` on are free, tiles are released in the order they were
      // issued, `oldest` is the first tile whose pages have not been taken back yet.
      int head = 0, free_pages = kPages, oldest = 0;
      bool gave_up = false;
      for (int i = 0; i < n_my; ++i) {
        const int slot = i % kSlots;
        ChunkRef cr2{-1, -1};
        if (i + 2 < n_my) cr2 = p.ws.chunks[tile0 + (i + 2) * stride];
        TensorMeta meta1 = meta;
        if (i + 1 < n_my && cr1.tensor != cr.tensor) meta1 = load_meta(p, a, cr1.tensor, ph, STRICT, cr1.index == 0);

        const TensorInfo& ti = meta.ti;
        const int tbytes = ti.theta_bits >> 3, cbytes = ti.comp_bits >> 3;
        // where the three arrays go (g, theta, c), and how many pages that takes including
        // those skipped when a run does not fit before the end of the ring
        constexpr int gbytes = GB / 8;
        // kChunk == kPageBytes: an array of b-byte elements takes b pages (2b with the large tiles)
        const int big = (ti.theta_bits == 8 && p.chunk8 != kChunk) ? 1 : 0;
        const int chunk = kChunk << big;
        const int run[3] = {gbytes << big, tbytes << big, cbytes << big};
        int page[3] = {0, 0, 0}, h2 = head, need = 0;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          if (run[r] == 0) continue;
          if (h2 + run[r] > kPages) { need += kPages - h2; h2 = 0; }
          page[r] = h2;
          h2 += run[r];
          need += run[r];
        }
        if (h2 == kPages) h2 = 0;
        // take back pages, descriptor slots and scans from the oldest tiles until this one fits
        while (free_pages < need || i - oldest >= kSlots) {
          const int os = oldest % kSlots;
          if (!mbar_wait(&sh->empty[os], (unsigned)(oldest / kSlots) & 1u, &sh->abort_flag)) {
            gave_up = true;
            break;
          }
          take_back(p, acc, amax_now, &sh->scan[os], sh->desc[os].tensor);
          free_pages += sh->slot_pages[os];
          ++oldest;
        }
        if (gave_up) {
          sh->abort_flag = 1;
          atomicCAS(p.ws.error, 0u, (unsigned)kErrEmptyWait);
          break;
        }
        head = h2;
        free_pages -= need;
        sh->slot_pages[slot] = need;

        const long long first = (long long)cr.index << (13 + big);
        const long long left = ti.numel - first;
        const int count = left < (long long)chunk ? (int)left : chunk;
        const int n_bulk = count & ~15;
        // The copies go out first and the descriptor is written while they are on their way:
        // the tile's barrier completes only when the bytes have landed AND the producer has
        // arrived, and it arrives after the descriptor is in place.
        unsigned char* const theta_g = static_cast<unsigned char*>(ti.theta) + first * tbytes;
        unsigned char* const comp_g = ti.comp ? static_cast<unsigned char*>(ti.comp) + first * cbytes : nullptr;
        const unsigned char* const grad_g = static_cast<const unsigned char*>(meta.grad) + first * gbytes;
        if (n_bulk > 0) {
          mbar_expect_tx(&sh->full[slot], (unsigned)(n_bulk * (tbytes + cbytes + gbytes)));
          bulk_load(smem + page[1] * kPageBytes, theta_g, (unsigned)(n_bulk * tbytes), &sh->full[slot]);
          if (cbytes)
            bulk_load(smem + page[2] * kPageBytes, comp_g, (unsigned)(n_bulk * cbytes), &sh->full[slot]);
          // Gradients are read once.  When theta and c of the whole list fit in L2, letting
          // the gradients leave it first keeps the state resident from step to step.
          if (p.grad_evict_first)
            bulk_load_hint(smem + page[0] * kPageBytes, grad_g, (unsigned)(n_bulk * gbytes), &sh->full[slot],
                           grad_policy);
          else
            bulk_load(smem + page[0] * kPageBytes, grad_g, (unsigned)(n_bulk * gbytes), &sh->full[slot]);
        }
        const StepCoef coef = make_coef(ti, meta.e_in, meta.e_out, meta.ec_in, meta.ec_out, meta.lr, GB, meta.eg,
                                        STRICT ? 1 : 0);
        // fixed-point gradients: the exact-fp32 path multiplies the mantissa by scale * 2^eg,
        // which must itself be exact (a normal number); otherwise the tile takes the general path
        float scale_hot = coef.scale;
        bool scale_ok = true;
        if constexpr (GB != 32) {
          const int ex = (int)((__float_as_uint(coef.scale) >> 23) & 0xffu);
          scale_ok = ex != 0 && ex + meta.eg >= 1 && ex + meta.eg <= 254;
          if (scale_ok) scale_hot = __int_as_float(__float_as_int(coef.scale) + (meta.eg << 23));
        }
        TileDesc& td = sh->desc[slot];
        td.scale = scale_hot;
        td.pow2s_neg = -pow2_float(coef.s);
        td.inv2s = pow2_float(-coef.s);
        td.pow2dc = pow2_float(-coef.delta_c);
        td.theta = theta_g;
        td.comp = comp_g;
        td.tensor = cr.tensor;
        td.n_bulk = n_bulk;
        td.count = count;
        td.flags = ((ti.theta_bits == 16 ? 3 : 0) + (ti.comp_bits >> 3)) |
                   ((coef.delta == 0 && scale_ok && (!STRICT || coef.s >= 0)) ? kFlagSteady : 0) |
                   // a coarser grid splits theta's mantissa at bit delta: that needs delta <= theta_bits - 1
                   ((!STRICT && coef.delta != 0 && scale_ok && coef.delta <= ti.theta_bits - 1) ? kFlagRegrid : 0) |
                   (page[1] << kFlagThetaPageShift) |
                   (page[2] << kFlagCompPageShift) | (page[0] << kFlagGradPageShift);
        td.coef = coef;
        td.grad = grad_g;
        mbar_arrive(&sh->full[slot]);
        issued = i + 1;
        cr = cr1;
        cr1 = cr2;
        meta = meta1;
      }
      // Collect the scans of the tiles still in the ring and publish.  The same waits make
      // sure that every copy this block started has landed before the block exits.
      for (int i = oldest; i < issued; ++i) {
        const int os = i % kSlots;
        if (mbar_wait(&sh->empty[os], (unsigned)(i / kSlots) & 1u, &sh->abort_flag))
          take_back(p, acc, amax_now, &sh->scan[os], sh->desc[os].tensor);
        else
          mbar_wait(&sh->full[os], (unsigned)(i / kSlots) & 1u, &sh->never);
      }
      publish(p, acc, amax_now);
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
    // read returned, and the wait above has seen the arrival); the block that draws the last
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
      const TileDesc* td = &sh->desc[stage];
      TileScan* scan = &sh->scan[stage];
      unsigned char* st = smem;
      if (!STRICT && (td->flags & kFlagRegrid)) {
        regrid_tile<GB>(td, scan, st);
      } else {
        const TileHot h = load_tile_hot(td);
        float amax_t = 0.0f, amax_c = 0.0f;
        bool wrote_stage;
        switch (h.flags & kFlagFormatMask) {
          case 0: wrote_stage = consume_tile<8, 0, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
          case 1: wrote_stage = consume_tile<8, 8, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
          case 2: wrote_stage = consume_tile<8, 16, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
          case 3: wrote_stage = consume_tile<16, 0, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
          case 4: wrote_stage = consume_tile<16, 8, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
          default: wrote_stage = consume_tile<16, 16, GB, STRICT>(h, td, st, ctid, scan, amax_t, amax_c); break;
        }
        add_warp_scans(scan, lane, amax_t, amax_c);
        // if the general path wrote into the stage, order those writes before the bulk copy
        // that refills it
        if (wrote_stage) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
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

__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  step_body<32, false>(p, a);
}

template <int GB>
__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_step_qgrad_kernel(const __grid_constant__ StepParams p, const __grid_constant__ QGradArgs a) {
  step_body<GB, false>(p, a);
}

__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_strict_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  step_body<32, true>(p, a);
}

template <int GB>
__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_strict_step_qgrad_kernel(const __grid_constant__ StepParams p, const __grid_constant__ QGradArgs a) {
  step_body<GB, true>(p, a);
}

// Per-step arguments of long lists: written to the workspace from kernel parameters.
__global__ void ksgd_upload_args_kernel(const __grid_constant__ UploadBatch b, int first, int count,
                                        const float** grad_ptr, float* lr) {
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    grad_ptr[first + i] = b.grads[i];
    lr[first + i] = b.lrs[i];
  }
}

__global__ void ksgd_upload_ints_kernel(const __grid_constant__ ExponentBatch b, int first, int count,
                                       int* dst) {
  for (int i = threadIdx.x; i < count; i += blockDim.x) dst[first + i] = b.exp_next[i];
}

// Caller-chosen exponents for the coming step, limited to kMaxDelta around the current one:
// written as overrides into the record the coming step reads.
__global__ void ksgd_set_exponents_kernel(const __grid_constant__ ExponentBatch b, int first,
                                          int count, int slab, const unsigned int* phase, TensorState* state) {
  const int ph = (int)phase[0], prev = ph == 0 ? 2 : ph - 1;
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    TensorState* rec = &state[(size_t)prev * slab + first + i];
    const int cur = rec->exp_theta;
    int e = max(kExpMin, min(kExpMax, b.exp_next[i]));
    e = max(cur - kMaxDelta, min(cur + kMaxDelta, e));
    rec->ovr_theta = e + kOvrBias;
  }
}

}  // namespace ksgd
