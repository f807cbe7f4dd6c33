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
// The persistent grid, the paged shared-memory ring, the scan publishing and the state that
// steps hand to one another are those of kahan_sgd_ring.cuh; this file adds what is specific
// to the plain optimizer: three arrays per tile (gradient, theta, c), the arithmetic of an
// element, two max scans and one exponent (two in strict mode) per tensor.
#pragma once

#include "kahan_sgd_ring.cuh"

namespace ksgd {

constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kBlockThreads = kConsumers + 32;   // + one producer warp

struct TensorInfo {
  void* theta;
  void* comp;
  long long numel;
  int theta_bits;
  int comp_bits;
  int s;       // grid distance: exp_comp = exp_theta - s  (0 in plain mode)
  int pad;
};

// What a step leaves behind for one tensor: everything the next step needs to know about it,
// in one 32-byte record (one load).
struct __align__(32) TensorState {
  int exp_theta;          // exponent of theta's mantissas as this step wrote them
  int exp_comp;           // strict mode: the same for the compensation's own exponent
  unsigned int amax[2];   // this step's max scans of theta and c (blocks add to them while the step runs)
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

struct StepParams {
  Workspace ws;
  int n_tensors;
  int n_chunks;
  int amax_mode;     // 1: exponents follow the max scan, 0: fixed
  int inline_args;   // 1: grads/lrs are in the InlineArgs parameter
  int state_in_l2;       // 1: theta and c of the whole list fit in L2 and stay there from step to step
  const int* exp_grad_dev;   // fixed-point gradients: device array of their exponents (as a scan on the
                             // device left them), or nullptr: the exponents come with the per-step arguments
  int advance;           // 1: this launch ends a step (the phase word moves on); 0: more launches of the
                         //    same step follow (the host-buffer entry point updates groups of tensors in turn)
  // The launch covers tiles [tile_begin, tile_begin + tile_count), which are all the tiles
  // of tensors [tensor_begin, tensor_begin + tensor_count): the whole list for an ordinary
  // step, one group of tensors when the host-buffer entry point pipelines its copies.
  int tile_begin, tile_count, tensor_begin, tensor_count;
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
constexpr int kFlagStream = 32;      // the list does not stay in L2: results are stored with the streaming hint
constexpr int kFlagThetaPageShift = 8;   // 5 bits each: first ring page of theta, c, g
constexpr int kFlagCompPageShift = 13;
constexpr int kFlagGradPageShift = 18;

// Max scans and counters of one tile, gathered in shared memory: the consumer warps add to
// it, the producer publishes it when it takes the tile's stage back.  (Two maxima, then three
// counts: the order the ring expects.)
struct TileScan {
  unsigned int amax_t, amax_c, n_sat_t, n_sat_c, n_nonfinite, pad[3];
};

// ----------------------------------------------------------------------------------------
// Arithmetic

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
// 2^24.  Statements 2-4 of Algorithm 1 for a vector whose increments d (on the output
// compensation grid, as always) the caller has formed already; k.pow2dc = 2^-delta.  Shared
// by the plain optimizer, the momentum optimizer and ADAM.
//
// Finer grid (delta < 0, a = -delta): the stored mantissas scale up exactly,
//   base = M + qt*2^a (both even, so exact even beyond 2^24),  u = qc*2^a - d,
//   Pb = fma(u, 2^-s, base) = M + P,  w = Pb - base,  r0 = fma(w, -2^s, u) = Rq  (no second rounding).
// Coarser grid (delta > 0, a = delta, s' = s + a): theta's mantissa is split with two integer
// operations per packed word, qt = A*2^a + B with 0 <= B < 2^a (on the sign-flipped lanes the
// split is a logical shift and a mask), so that
//   T = A*2^s' + v,  v = B*2^s + qc - d*2^a   (exact when |d|*2^a <= 4e6)
//   Pb = fma(v, 2^-s', M + A) = M + P,  w = Pb - (M + A),  R = fma(w, -2^s', v),
//   Rm = fma(R, 2^-a, M) = M + Rq   (the second rounding of the coarser grid, ties on Rq's parity).
// In both cases |Rq| <= 2^(s-1) whenever P needs no clamp, so c never clamps on this path.
// yM[i] = M + d_i.  The caller guarantees |d| <= regrid_d_limit(k) (and no NaN); the function
// returns false (nothing stored: the vector goes to the general path) when some |P| exceeds
// QMAX.  A coarser change needs a <= TB - 1 (the producer checks).
struct RegridCoef {
  float pow2dc;     // 2^-delta
  float inv2s;      // 2^-s
  float pow2s_neg;  // -2^s
};

__device__ __forceinline__ float regrid_d_limit(const RegridCoef& k) {
  return k.pow2dc > 1.0f ? 4000000.0f : __fmul_rn(4000000.0f, k.pow2dc);   // coarser: |d| * 2^a stays exact
}

template <int TB, int CB, int V>
__device__ __forceinline__ bool regrid_core(const Pack<V * TB / 8>& pt, const Pack<(CB ? V * CB / 8 : 8)>& pc,
                                            const float (&yM)[V], const RegridCoef& k, Pack<V * TB / 8>& ot,
                                            Pack<(CB ? V * CB / 8 : 8)>& oc, float& amax_t, float& amax_c) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int CBS = CB ? CB : 8;
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
  float Pm[V], rm[V], ra[2];
  float hiP = kMagic, loP = kMagic, aR = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    float qc = 0.0f;
    if constexpr (HAS_COMP) qc = __fadd_rn(magic_signed<CBS>(pc, i), -kMagic);
    float P, r;
    if (finer) {
      const float qt = __fadd_rn(magic_signed<TB>(pt, i), -kMagic);
      const float base = __fmaf_rn(qt, up, kMagic);
      const float u = __fmaf_rn(qc, up, __fadd_rn(kMagic, -yM[i]));
      P = __fmaf_rn(u, inv2sp, base);
      const float w = __fadd_rn(P, -base);
      r = __fmaf_rn(w, pow2sp_neg, u);
      rm[i] = __fadd_rn(r, kMagic);
    } else {
      const float base = __fadd_rn(magic_elem<TB>(pA, i), -biasA);       // M + A
      const float B = __fadd_rn(magic_elem<TB>(pB, i), -kMagic);
      const float d = __fadd_rn(yM[i], -kMagic);
      const float v = __fmaf_rn(d, -up, __fmaf_rn(B, pow2s, qc));
      P = __fmaf_rn(v, inv2sp, base);
      const float w = __fadd_rn(P, -base);
      const float R = __fmaf_rn(w, pow2sp_neg, v);
      rm[i] = __fmaf_rn(R, down, kMagic);
      r = __fadd_rn(rm[i], -kMagic);
    }
    Pm[i] = P;
    ra[i & 1] = fabsf(r);
    if (i & 1) {
      hiP = max3(hiP, Pm[i - 1], P);
      loP = min3(loP, Pm[i - 1], P);
      if constexpr (HAS_COMP) aR = max3(aR, ra[0], ra[1]);
    }
  }
  const float aP = fmaxf(__fadd_rn(hiP, -kMagic), __fadd_rn(kMagic, -loP));
  constexpr float qmax_t = (float)((1 << (TB - 1)) - 1);
  if (aP > qmax_t) return false;
  amax_t = fmaxf(amax_t, aP);
  if constexpr (HAS_COMP) amax_c = fmaxf(amax_c, aR);
  ot = pack_magic<TB, V>(Pm);
  if constexpr (HAS_COMP) oc = pack_magic<CB, V>(rm);
  return true;
}

// The plain optimizer's increment for such a vector: d = rne(g * scale), as in update_vector.
template <int TB, int CB, int V, int GB>
__device__ __forceinline__ bool update_vector_regrid(const Pack<V * TB / 8>& pt, const Pack<(CB ? V * CB / 8 : 8)>& pc,
                                                     const Pack<V * GB / 8>& pg, const SteadyCoef& k,
                                                     Pack<V * TB / 8>& ot, Pack<(CB ? V * CB / 8 : 8)>& oc,
                                                     float& amax_t, float& amax_c) {
  constexpr int GBS = GB == 32 ? 8 : GB;
  const RegridCoef rk{k.pow2dc, k.inv2s, k.pow2s_neg};
  float yM[V], xa[2];
  float aX = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    float g;
    if constexpr (GB == 32) g = __uint_as_float(pack_word(pg, i));
    else g = __fadd_rn(magic_signed<GBS>(pg, i), -kMagic);
    const float x = __fmul_rn(g, k.scale);              // the one binary32 multiply
    yM[i] = __fadd_rn(x, kMagic);                       // M + d
    xa[i & 1] = fabsf(x);
    if (i & 1) aX = max3_nan(aX, xa[0], xa[1]);         // NaN if any product is
  }
  if (!(aX <= regrid_d_limit(rk))) return false;        // also Inf and NaN products
  return regrid_core<TB, CB, V>(pt, pc, yM, rk, ot, oc, amax_t, amax_c);
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
  const bool stream = (h.flags & kFlagStream) != 0;
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
    if (stream) {
      store_pack_streaming<TBYTES>(h.theta + (size_t)v * TBYTES, ot);
      if constexpr (HAS_COMP) store_pack_streaming<CBYTES>(h.comp + (size_t)v * CBYTES, oc);
    } else {
      store_pack<TBYTES>(h.theta + (size_t)v * TBYTES, ot);
      if constexpr (HAS_COMP) store_pack<CBYTES>(h.comp + (size_t)v * CBYTES, oc);
    }
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
  m.e_out = r1.x ? r1.x - kOvrBias : next_exponent((unsigned)r0.z, m.ti.theta_bits, m.e_in, p.amax_mode);   // r0.z, r0.w: amax[0], amax[1]
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
                                                const TensorInfo* ti) {
  TensorMeta m;
  m.ti = ti ? *ti : p.ws.info[t];
  m.grad = p.inline_args ? a.grads[t] : p.ws.grad_ptr[t];
  m.lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];
  m.eg = 0;
  step_exponents(p, t, ph, strict, m);
  return m;
}

__device__ __forceinline__ TensorMeta load_meta(const StepParams& p, const QGradArgs& a, int t, int ph, bool strict,
                                                const TensorInfo* ti) {
  TensorMeta m;
  m.ti = ti ? *ti : p.ws.info[t];
  m.grad = p.inline_args ? a.grads[t] : static_cast<const void*>(p.ws.grad_ptr[t]);
  m.lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];
  if (p.exp_grad_dev) m.eg = max(kExpMin, min(kExpMax, __ldcg(p.exp_grad_dev + t)));
  else m.eg = p.inline_args ? (int)a.exp_grad[t] : p.ws.exp_grad[t];
  step_exponents(p, t, ph, strict, m);
  return m;
}

// The plain optimizer as a policy of the ring (kahan_sgd_ring.cuh).  GB = 32: binary32
// gradients; 8 / 16: fixed-point gradients (one or two bytes per parameter instead of four on
// the gradient stream).  STRICT: every statement of Algorithm 1 rounds into the stored format
// and the compensation has its own exponent (comp_bits != 0 for every tensor).
template <int GB, bool STRICT>
struct PlainPolicy {
  static constexpr int kStreams = 3;          // gradient, theta, c
  static constexpr int kConsumerWarps = ksgd::kConsumerWarps;
  static constexpr int kAmax = 2, kCounts = 3;
  static constexpr int kLongStepTiles = 16;   // tiles per block from which the ring limits its tiles in flight
  static constexpr bool kGradEvictFirstBeyondL2 = true;
  using Params = StepParams;
  using Info = TensorInfo;
  using State = TensorState;
  using TileDesc = ksgd::TileDesc;
  using TileScan = ksgd::TileScan;
  using Meta = TensorMeta;

  template <typename Args>
  static __device__ __forceinline__ Meta load_meta(const Params& p, const Args& a, int t, int ph, const Info* ti) {
    return ksgd::load_meta(p, a, t, ph, STRICT, ti);
  }
  static __device__ __forceinline__ void record(const Params& p, int t, int ph, const Meta& m) {
    record_exponents(p, t, ph, STRICT, m);
  }
  static __device__ __forceinline__ void streams(const Meta& m, const unsigned char* (&base)[kStreams],
                                                 int (&bytes)[kStreams]) {
    base[0] = static_cast<const unsigned char*>(m.grad);
    bytes[0] = GB / 8;
    base[1] = static_cast<const unsigned char*>(m.ti.theta);
    bytes[1] = m.ti.theta_bits >> 3;
    base[2] = static_cast<const unsigned char*>(m.ti.comp);
    bytes[2] = m.ti.comp_bits >> 3;
  }
  static __device__ __forceinline__ void fill_desc(TileDesc& td, const Params& p, const Meta& meta, int tensor,
                                                   int count, int n_bulk, const int (&page)[kStreams],
                                                   const unsigned char* const (&gptr)[kStreams]) {
    const TensorInfo& ti = meta.ti;
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
    td.scale = scale_hot;
    td.pow2s_neg = -pow2_float(coef.s);
    td.inv2s = pow2_float(-coef.s);
    td.pow2dc = pow2_float(-coef.delta_c);
    td.theta = const_cast<unsigned char*>(gptr[1]);
    td.comp = const_cast<unsigned char*>(gptr[2]);
    td.tensor = tensor;
    td.n_bulk = n_bulk;
    td.count = count;
    td.flags = ((ti.theta_bits == 16 ? 3 : 0) + (ti.comp_bits >> 3)) |
           ((coef.delta == 0 && scale_ok && (!STRICT || coef.s >= 0)) ? kFlagSteady : 0) |
           // a coarser grid splits theta's mantissa at bit delta: that needs delta <= theta_bits - 1
           ((!STRICT && coef.delta != 0 && scale_ok && coef.delta <= ti.theta_bits - 1) ? kFlagRegrid : 0) |
           (p.state_in_l2 ? 0 : kFlagStream) |
           (page[1] << kFlagThetaPageShift) |
           (page[2] << kFlagCompPageShift) | (page[0] << kFlagGradPageShift);
    td.coef = coef;
    td.grad = gptr[0];
  }
  // One consumer thread's share of a tile: the exact-fp32 paths per format, the scans of its
  // warp added to the tile's slot.
  static __device__ __forceinline__ void consume(const TileDesc* td, TileScan* scan, unsigned char* smem, int ctid,
                                                 int lane) {
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
  }
};

constexpr size_t kSharedBytes = ring_shared_bytes<PlainPolicy<32, false>>();   // the same for every plain variant

__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  ring_step<PlainPolicy<32, false>>(p, a);
}

template <int GB>
__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_step_qgrad_kernel(const __grid_constant__ StepParams p, const __grid_constant__ QGradArgs a) {
  ring_step<PlainPolicy<GB, false>>(p, a);
}

__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_strict_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  ring_step<PlainPolicy<32, true>>(p, a);
}

template <int GB>
__global__ void __launch_bounds__(kBlockThreads, 1)
ksgd_strict_step_qgrad_kernel(const __grid_constant__ StepParams p, const __grid_constant__ QGradArgs a) {
  ring_step<PlainPolicy<GB, true>>(p, a);
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
