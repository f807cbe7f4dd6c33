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
//   - in the last block to finish, the exponent choice itself for every tensor.
// The pass is bound by HBM traffic: 2*m/8 + 2*n/8 + 4 bytes per parameter.
//
// Structure: a persistent grid, one block per SM.  The tensor list is cut into tiles of
// kChunk elements; each block owns a contiguous run of tiles.  One producer thread
// streams the tiles of theta, c and g into a ring of shared-memory stages with bulk
// asynchronous copies (cp.async.bulk, completion counted on an mbarrier), so the bytes in
// flight do not depend on registers or occupancy; sixteen consumer warps compute from
// shared memory and store theta' and c' straight to global memory with 16-byte stores.
// No block ever waits for another block; every wait inside a block is bounded.
#pragma once

#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

namespace ksgd {

constexpr int kChunk = 8192;           // elements per tile
constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kBlockThreads = kConsumers + 32;   // + one producer warp
constexpr int kStages = 3;
constexpr int kStageBytes = kChunk * 8;          // theta <= 2 B, c <= 2 B, g 4 B per element
constexpr int kStageThetaOff = 0;
constexpr int kStageCompOff = kChunk * 2;
constexpr int kStageGradOff = kChunk * 4;
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
  int index;   // tile number inside that tensor: elements [index*kChunk, ...)
};

// Device-side view of the caller's workspace.
struct Workspace {
  int* exp_cur;                    // [n] exponent of the stored mantissas
  int* exp_next;                   // [n] exponent the coming step writes
  unsigned int* amax_last;         // [2n] max scans of the last finished step (theta | comp)
  unsigned long long* counters;    // [3n] cumulative: sat_theta | sat_comp | nonfinite
  unsigned int* error;             // [1] first DeviceError seen (0 = none), sticky
  unsigned int* amax_acc;          // [2n] max scans being accumulated by the running step
  TensorInfo* info;                // [n]
  const float** grad_ptr;          // [n] per-step arguments for lists longer than kInlineArgs
  float* lr;                       // [n]
  ChunkRef* chunks;                // [n_chunks]
  unsigned int* ticket;            // blocks finished in the running step
};

struct StepParams {
  Workspace ws;
  int n_tensors;
  int n_chunks;
  int amax_mode;     // 1: exponents follow the max scan, 0: fixed
  int inline_args;   // 1: grads/lrs are in the InlineArgs parameter
};

struct InlineArgs {
  const float* grads[kInlineArgs];
  float lrs[kInlineArgs];
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
};

// One tile as the producer describes it to the consumers (lives in shared memory).
struct TileDesc {
  StepCoef coef;
  void* theta;          // global address of the tile's first theta mantissa
  void* comp;           // same for the compensation (unused in plain mode)
  const float* grad;    // same for the gradient
  int tensor;
  int count;            // valid elements in the tile
  int n_bulk;           // elements that arrived through the bulk copies (multiple of 16)
  int theta_bits;
  int comp_bits;
  int pad;
};

// Max scans and counters of the rare path, one set per consumer warp (shared memory).
struct WarpSlots {
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

__device__ __forceinline__ StepCoef make_coef(const TensorInfo& ti, int e_in, int e_out, float lr) {
  StepCoef k;
  const int delta = e_out - e_in;
  k.s = ti.s;
  k.delta = delta;
  k.sh_t = ti.s + max(0, -delta);
  k.sh_c = max(0, -delta);
  k.sh_d = max(0, delta);
  k.r_t = ti.s + max(0, delta);
  k.r_c = max(0, delta);
  k.qmax_t = (1 << (ti.theta_bits - 1)) - 1;
  k.qmax_c = ti.comp_bits ? (1 << (ti.comp_bits - 1)) - 1 : 0;
  k.scale = __fmul_rn(lr, pow2_float(ti.s - e_out));   // |s - e_out| <= 79: exact power of two
  return k;
}

// Algorithm 1 for elements [first, first+n) of a tile with 64-bit intermediates, straight
// from and to global memory.  This is the rare path: exponent changes, vectors in which
// theta saturates or a gradient is not finite, and ragged tails.  It is kept out of line
// (one copy for all formats) so that it costs the steady-state path no registers.
__device__ __noinline__ void update_general(const TileDesc* td, int first, int n, WarpSlots* slots) {
  const StepCoef k = td->coef;
  const int tb = td->theta_bits, cb = td->comp_bits;
  unsigned int amax_t = 0, amax_c = 0, n_sat_t = 0, n_sat_c = 0, n_nf = 0;
  for (int e = first; e < first + n; ++e) {
    const int qt = tb == 8 ? (int)static_cast<const signed char*>(td->theta)[e]
                           : (int)static_cast<const short*>(td->theta)[e];
    int qc = 0;
    if (cb == 8) qc = (int)static_cast<const signed char*>(td->comp)[e];
    else if (cb == 16) qc = (int)static_cast<const short*>(td->comp)[e];
    const float g = td->grad[e];
    const int d = quantize_increment(g, k.scale);
    const long long T = (long long)qt * (1LL << k.sh_t) + (long long)qc * (1LL << k.sh_c) -
                        (long long)d * (1LL << k.sh_d);
    const long long P = rne_shift64(T, k.r_t);
    const long long Pc = P > k.qmax_t ? k.qmax_t : (P < -k.qmax_t ? -k.qmax_t : P);
    const unsigned long long aP = (unsigned long long)(P < 0 ? -P : P);
    amax_t = max(amax_t, (unsigned int)aP);
    n_sat_t += (P != Pc);
    if (tb == 8) static_cast<signed char*>(td->theta)[e] = (signed char)Pc;
    else static_cast<short*>(td->theta)[e] = (short)Pc;
    if (cb) {
      const long long R = T - Pc * (1LL << k.r_t);
      const long long Rq = rne_shift64(R, k.r_c);
      const long long Rc = Rq > k.qmax_c ? k.qmax_c : (Rq < -k.qmax_c ? -k.qmax_c : Rq);
      unsigned long long aR = (unsigned long long)(Rq < 0 ? -Rq : Rq);
      if (aR > 0x7fffffffULL) aR = 0x7fffffffULL;
      amax_c = max(amax_c, (unsigned int)aR);
      n_sat_c += (Rq != Rc);
      if (cb == 8) static_cast<signed char*>(td->comp)[e] = (signed char)Rc;
      else static_cast<short*>(td->comp)[e] = (short)Rc;
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

// Sign-extended element i of a pack of BITS-wide integers.
template <int BITS, int BYTES>
__device__ __forceinline__ int unpack_elem(const Pack<BYTES>& r, int i) {
  if constexpr (BITS == 8) {
    const unsigned int w = pack_word(r, i >> 2);
    return (int)(signed char)(w >> (8 * (i & 3)));
  } else {
    const unsigned int w = pack_word(r, i >> 1);
    return (i & 1) ? ((int)w >> 16) : (int)(short)(w & 0xffffu);
  }
}

template <int BITS, int V>
__device__ __forceinline__ Pack<V * BITS / 8> pack_elems(const int (&x)[V]) {
  Pack<V * BITS / 8> r;
  if constexpr (BITS == 8) {
#pragma unroll
    for (int w = 0; w < V / 4; ++w) {
      const unsigned int lo = __byte_perm((unsigned)x[4 * w], (unsigned)x[4 * w + 1], 0x0040);
      const unsigned int hi = __byte_perm((unsigned)x[4 * w + 2], (unsigned)x[4 * w + 3], 0x0040);
      set_pack_word(r, w, __byte_perm(lo, hi, 0x5410));
    }
  } else {
#pragma unroll
    for (int w = 0; w < V / 2; ++w)
      set_pack_word(r, w, __byte_perm((unsigned)x[2 * w], (unsigned)x[2 * w + 1], 0x5410));
  }
  return r;
}

// ----------------------------------------------------------------------------------------
// Steady state (no exponent change, s >= 1 or plain mode): one vector of V elements in
// 32-bit arithmetic.  T = qt*2^s + u with u = qc - d; rounding T by s bits to nearest-even
// only needs u, the parity of the truncated quotient and qt.  Returns false, having stored
// nothing, if any element saturates theta or has a non-finite gradient: the caller then
// runs the vector through update_general.

template <int TB, int CB, int V>
__device__ __forceinline__ bool update_vector(const Pack<V * TB / 8>& pt,
                                              const Pack<(CB ? V * CB / 8 : 8)>& pc,
                                              const Pack<V * 4>& pg, float scale, int s, int qmax_t,
                                              Pack<V * TB / 8>& ot, Pack<(CB ? V * CB / 8 : 8)>& oc,
                                              unsigned int& amax_t, unsigned int& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  int nt[V], nc[V];
  const int hm1 = HAS_COMP ? ((1 << (s - 1)) - 1) : 0;
  int mxP = -0x7fffffff, mnP = 0x7fffffff, mxR = 0, mnR = 0;
  float nf = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const int qt = unpack_elem<TB>(pt, i);
    const float g = __uint_as_float(pack_word(pg, i));
    const int d = quantize_increment(g, scale);
    nf = fmaf(g, 0.0f, nf);             // stays 0 unless some g is Inf or NaN
    int P, r0;
    if constexpr (HAS_COMP) {
      const int u = unpack_elem<(CB ? CB : 8)>(pc, i) - d;
      const int par = (qt + (u >> s)) & 1;
      const int w = (u + hm1 + par) >> s;
      P = qt + w;
      r0 = u - w * (1 << s);
      mxR = max(mxR, r0);
      mnR = min(mnR, r0);
    } else {
      P = qt - d;
      r0 = 0;
    }
    nt[i] = P;
    nc[i] = r0;
    mxP = max(mxP, P);
    mnP = min(mnP, P);
  }
  if ((mxP > qmax_t) | (mnP < -qmax_t) | (nf != nf)) return false;
  amax_t = max(amax_t, (unsigned int)max(mxP, -mnP));
  if constexpr (HAS_COMP) amax_c = max(amax_c, (unsigned int)max(mxR, -mnR));
  ot = pack_elems<TB, V>(nt);
  if constexpr (HAS_COMP) oc = pack_elems<CB, V>(nc);
  return true;
}

// All vectors of one tile that belong to this consumer thread.
template <int TB, int CB>
__device__ __forceinline__ void consume_tile(const TileDesc* td, const unsigned char* stage,
                                             int ctid, WarpSlots* slots, unsigned int& amax_t,
                                             unsigned int& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int V = (TB == 8) ? 16 : 8;              // 16 bytes of theta per vector
  constexpr int TBYTES = V * TB / 8;
  constexpr int CBYTES = HAS_COMP ? V * CB / 8 : 8;
  const StepCoef& k = td->coef;
  const bool steady = (k.delta == 0) && (!HAS_COMP || k.s >= 1);
  const int n_vec = td->n_bulk / V;
  if (steady) {
    const float scale = k.scale;
    const int s = k.s, qmax_t = k.qmax_t;
    unsigned char* theta_g = static_cast<unsigned char*>(td->theta);
    unsigned char* comp_g = static_cast<unsigned char*>(td->comp);
    for (int v = ctid; v < n_vec; v += kConsumers) {
      const Pack<TBYTES> pt = load_pack<TBYTES>(stage + kStageThetaOff + v * TBYTES);
      Pack<CBYTES> pc;
      if constexpr (HAS_COMP) pc = load_pack<CBYTES>(stage + kStageCompOff + v * CBYTES);
      const Pack<V * 4> pg = load_pack<V * 4>(stage + kStageGradOff + v * (V * 4));
      Pack<TBYTES> ot;
      Pack<CBYTES> oc;
      if (update_vector<TB, CB, V>(pt, pc, pg, scale, s, qmax_t, ot, oc, amax_t, amax_c)) {
        store_pack<TBYTES>(theta_g + (size_t)v * TBYTES, ot);
        if constexpr (HAS_COMP) store_pack<CBYTES>(comp_g + (size_t)v * CBYTES, oc);
      } else {
        update_general(td, v * V, V, slots);
      }
    }
  } else {
    for (int v = ctid; v < n_vec; v += kConsumers) update_general(td, v * V, V, slots);
  }
  // ragged tail (fewer than 16 elements) that the bulk copies did not bring
  const int e = td->n_bulk + ctid;
  if (e < td->count) update_general(td, e, 1, slots);
}

// Next exponent from the max scan: the tight fit puts the largest mantissa in
// (QMAX/2, QMAX].  With L = bit length of amax and QMAX = 2^(b-1)-1, the change is
// L-(b-1), plus one more when amax still exceeds QMAX*2^change.
__device__ __forceinline__ int next_exponent(unsigned int amax, int bits, int e_out, int amax_mode) {
  if (!amax_mode || amax == 0u) return e_out;
  const int L = 32 - __clz(amax);
  int change = L - (bits - 1);
  if (change >= 1) {
    const unsigned long long cap = (unsigned long long)((1 << (bits - 1)) - 1) << change;
    if ((unsigned long long)amax > cap) ++change;
  }
  change = max(-kMaxDelta, min(kMaxDelta, change));
  return max(kExpMin, min(kExpMax, e_out + change));
}

struct __align__(128) BlockShared {
  unsigned long long full[kStages];    // producer -> consumers: the tile's bytes have landed
  unsigned long long empty[kStages];   // consumers -> producer: the stage may be refilled
  TileDesc desc[kStages];
  WarpSlots slots[kConsumerWarps];
  int abort_flag;   // set by the first thread whose bounded wait ran out
  int is_last;
  int never;        // stays 0: abort flag for waits that must not be cut short
};

constexpr size_t kSharedBytes = (size_t)kStages * kStageBytes + sizeof(BlockShared) + 128;

// Publish a consumer warp's scans of tensor t and clear them.
__device__ __forceinline__ void flush_scans(const StepParams& p, int t, WarpSlots* slots, int lane,
                                            unsigned int& amax_t, unsigned int& amax_c) {
  const unsigned int full = 0xffffffffu;
  unsigned int at = __reduce_max_sync(full, amax_t);
  unsigned int ac = __reduce_max_sync(full, amax_c);
  amax_t = 0u;
  amax_c = 0u;
  if (lane == 0 && t >= 0) {
    at = max(at, slots->amax_t);
    ac = max(ac, slots->amax_c);
    if (at) atomicMax(&p.ws.amax_acc[t], at);
    if (ac) atomicMax(&p.ws.amax_acc[p.n_tensors + t], ac);
    if (slots->n_sat_t) atomicAdd(&p.ws.counters[t], (unsigned long long)slots->n_sat_t);
    if (slots->n_sat_c) atomicAdd(&p.ws.counters[p.n_tensors + t], (unsigned long long)slots->n_sat_c);
    if (slots->n_nonfinite)
      atomicAdd(&p.ws.counters[2 * p.n_tensors + t], (unsigned long long)slots->n_nonfinite);
    slots->amax_t = slots->amax_c = slots->n_sat_t = slots->n_sat_c = slots->n_nonfinite = 0u;
  }
  __syncwarp();
}

__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
  BlockShared* sh = reinterpret_cast<BlockShared*>(base + (size_t)kStages * kStageBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this block's contiguous run of tiles
  const long long g = gridDim.x, b = blockIdx.x;
  const int tile0 = (int)(b * p.n_chunks / g);
  const int n_my = (int)((b + 1) * p.n_chunks / g) - tile0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sh->full[s], 1u);
      mbar_init(&sh->empty[s], (unsigned)kConsumerWarps);
    }
    sh->abort_flag = 0;
    sh->is_last = 0;
    sh->never = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kConsumerWarps * (int)(sizeof(WarpSlots) / 4))
    reinterpret_cast<unsigned int*>(sh->slots)[threadIdx.x] = 0u;
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int cur = -1;
      TensorInfo ti{};
      StepCoef coef{};
      const float* grad = nullptr;
      int issued = 0;
      for (int i = 0; i < n_my; ++i) {
        const int stage = i % kStages, use = i / kStages;
        if (use > 0 && !mbar_wait(&sh->empty[stage], (unsigned)(use - 1) & 1u, &sh->abort_flag)) {
          sh->abort_flag = 1;
          atomicCAS(p.ws.error, 0u, (unsigned)kErrEmptyWait);
          break;
        }
        const ChunkRef cr = p.ws.chunks[tile0 + i];
        if (cr.tensor != cur) {
          cur = cr.tensor;
          ti = p.ws.info[cur];
          const int e_in = p.ws.exp_cur[cur], e_out = p.ws.exp_next[cur];
          grad = p.inline_args ? a.grads[cur] : p.ws.grad_ptr[cur];
          const float lr = p.inline_args ? a.lrs[cur] : p.ws.lr[cur];
          coef = make_coef(ti, e_in, e_out, lr);
        }
        const long long first = (long long)cr.index * kChunk;
        const long long left = ti.numel - first;
        const int count = left < (long long)kChunk ? (int)left : kChunk;
        const int n_bulk = count & ~15;
        const int tbytes = ti.theta_bits >> 3, cbytes = ti.comp_bits >> 3;
        TileDesc& td = sh->desc[stage];
        td.coef = coef;
        td.theta = static_cast<unsigned char*>(ti.theta) + first * tbytes;
        td.comp = ti.comp ? static_cast<unsigned char*>(ti.comp) + first * cbytes : nullptr;
        td.grad = grad + first;
        td.tensor = cur;
        td.count = count;
        td.n_bulk = n_bulk;
        td.theta_bits = ti.theta_bits;
        td.comp_bits = ti.comp_bits;
        unsigned char* st = base + (size_t)stage * kStageBytes;
        if (n_bulk > 0) {
          mbar_arrive_expect_tx(&sh->full[stage], (unsigned)(n_bulk * (tbytes + cbytes + 4)));
          bulk_load(st + kStageThetaOff, td.theta, (unsigned)(n_bulk * tbytes), &sh->full[stage]);
          if (cbytes) bulk_load(st + kStageCompOff, td.comp, (unsigned)(n_bulk * cbytes), &sh->full[stage]);
          bulk_load(st + kStageGradOff, td.grad, (unsigned)(n_bulk * 4), &sh->full[stage]);
        } else {
          mbar_arrive(&sh->full[stage]);
        }
        issued = i + 1;
      }
      // Before the block may exit, every copy it started must have landed (normally the
      // consumers have long since seen them; this only matters after a give-up).
      for (int i = max(0, issued - kStages); i < issued; ++i)
        mbar_wait(&sh->full[i % kStages], (unsigned)(i / kStages) & 1u, &sh->never);
    }
  } else {
    // ------------------------------------------------------------------ consumers
    const int ctid = threadIdx.x;
    WarpSlots* slots = &sh->slots[warp];
    unsigned int amax_t = 0u, amax_c = 0u;
    int cur = -1;
    for (int i = 0; i < n_my; ++i) {
      const int stage = i % kStages, use = i / kStages;
      if (!mbar_wait(&sh->full[stage], (unsigned)use & 1u, &sh->abort_flag)) {
        if (lane == 0) {
          sh->abort_flag = 1;
          atomicCAS(p.ws.error, 0u, (unsigned)kErrFullWait);
        }
        break;
      }
      const TileDesc* td = &sh->desc[stage];
      const int t = td->tensor;
      if (t != cur) {
        flush_scans(p, cur, slots, lane, amax_t, amax_c);
        cur = t;
      }
      const unsigned char* st = base + (size_t)stage * kStageBytes;
      const int tb = td->theta_bits, cb = td->comp_bits;
      if (tb == 8) {
        if (cb == 8) consume_tile<8, 8>(td, st, ctid, slots, amax_t, amax_c);
        else if (cb == 16) consume_tile<8, 16>(td, st, ctid, slots, amax_t, amax_c);
        else consume_tile<8, 0>(td, st, ctid, slots, amax_t, amax_c);
      } else {
        if (cb == 8) consume_tile<16, 8>(td, st, ctid, slots, amax_t, amax_c);
        else if (cb == 16) consume_tile<16, 16>(td, st, ctid, slots, amax_t, amax_c);
        else consume_tile<16, 0>(td, st, ctid, slots, amax_t, amax_c);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[stage]);
    }
    flush_scans(p, cur, slots, lane, amax_t, amax_c);
  }

  // ---------------------------------------------------------------------- block done
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int done = atomicAdd(p.ws.ticket, 1u);
    sh->is_last = (done == gridDim.x - 1u);
  }
  __syncthreads();
  if (!sh->is_last) return;

  // Last block to finish: every other block has published its scans and has long since
  // read the exponents, so they can be rotated here.  No block ever waits for another.
  __threadfence();
  for (int i = threadIdx.x; i < p.n_tensors; i += kBlockThreads) {
    const unsigned int at = __ldcg(&p.ws.amax_acc[i]);
    const unsigned int ac = __ldcg(&p.ws.amax_acc[p.n_tensors + i]);
    const int eo = p.ws.exp_next[i];
    p.ws.exp_cur[i] = eo;
    p.ws.exp_next[i] = next_exponent(at, p.ws.info[i].theta_bits, eo, p.amax_mode);
    p.ws.amax_last[i] = at;
    p.ws.amax_last[p.n_tensors + i] = ac;
    p.ws.amax_acc[i] = 0u;
    p.ws.amax_acc[p.n_tensors + i] = 0u;
  }
  if (threadIdx.x == 0) *p.ws.ticket = 0u;
}

// Per-step arguments of long lists: written to the workspace from kernel parameters.
__global__ void ksgd_upload_args_kernel(const __grid_constant__ UploadBatch b, int first, int count,
                                        const float** grad_ptr, float* lr) {
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    grad_ptr[first + i] = b.grads[i];
    lr[first + i] = b.lrs[i];
  }
}

// Caller-chosen exponents for the coming step, limited to kMaxDelta around the current one.
__global__ void ksgd_set_exponents_kernel(const __grid_constant__ ExponentBatch b, int first,
                                          int count, const int* exp_cur, int* exp_next) {
  for (int i = threadIdx.x; i < count; i += blockDim.x) {
    const int cur = exp_cur[first + i];
    int e = max(kExpMin, min(kExpMax, b.exp_next[i]));
    e = max(cur - kMaxDelta, min(cur + kMaxDelta, e));
    exp_next[first + i] = e;
  }
}

}  // namespace ksgd
