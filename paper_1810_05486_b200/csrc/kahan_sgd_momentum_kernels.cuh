// Device code of the momentum optimizer with the lazy update (Section 4 of
// arXiv 1810.05486: Algorithm 1 "implemented in the optimizers", momentum mu = 0.9 kept
// in INT8 or INT16).  Per element
//     v <- mu*v + eta*g          velocity, a third dynamic fixed-point tensor
//     theta <- theta - v         through Algorithm 1, with v in the place of eta*g
// and three max scans per tensor (|P|, |Rq|, |V|) that steer the exponents of theta and of
// the velocity independently.
//
// The persistent grid, the paged shared-memory ring, the scan publishing and the state that
// steps hand to one another are those of kahan_sgd_ring.cuh; this file is the policy: four
// arrays per tile (gradient, theta, c, v), the arithmetic of an element, three scans and two
// exponents per tensor.  HBM traffic: 2*m/8 + 2*n/8 + 2*b/8 + 4 bytes per parameter.
#pragma once

#include "kahan_sgd_kernels.cuh"

namespace ksgd {
namespace mom {

struct TensorInfo {
  void* theta;
  void* comp;
  void* mom;
  long long numel;
  int theta_bits;
  int comp_bits;
  int mom_bits;
  int s;       // grid distance: exp_comp = exp_theta - s
};

// What a step leaves behind for one tensor (see kahan_sgd_ring.cuh): one 32-byte record.
struct __align__(32) TensorState {
  int exp_theta;          // exponents as this step wrote them
  int exp_mom;
  unsigned int amax[3];   // this step's max scans: |P|, |Rq|, |V|
  int ovr_theta;          // exponents the NEXT step must write instead of those the scans give
  int ovr_mom;            //   (value + kOvrBias, 0 = none; set at init)
  int pad;
};

struct Workspace {
  unsigned int* phase;             // [0] phase of the coming step; [1] entry tickets of the running step
  TensorState* state;              // [3][slab]
  int slab;
  unsigned long long* counters;    // [4n] sat_theta | sat_comp | sat_mom | nonfinite
  unsigned int* error;             // [1]
  TensorInfo* info;                // [n]
  ChunkRef* chunks;                // [n_chunks]
  const float** grad_ptr;          // [n] per-step arguments for lists longer than kInlineArgs
  float* lr;                       // [n]
  float* mu;                       // [n]
};

struct StepParams {
  Workspace ws;
  int n_tensors;
  int tile_begin, tile_count;      // all tiles of the list
  int amax_mode;
  int state_in_l2;
  int inline_args;                 // 1: grads/lrs/mus are in the StepArgs parameter
  int advance;                     // 1 (every launch is a whole step)
};

struct StepArgs {                  // per-step arguments, passed as a kernel parameter
  const float* grads[kInlineArgs];
  float lrs[kInlineArgs];
  float mus[kInlineArgs];
};

// Twelve consumer warps (three per scheduler, plus the producer's) leave 128 registers per
// thread: a vector of eight elements with three mantissa arrays then stays in registers.
constexpr int kWarps = 12;                     // consumer warps; one more warp produces
constexpr int kThreads = 32 * kWarps;
constexpr int kBlock = kThreads + 32;

// What a tile's tensor needs for this step (general path reads all of it).
struct Coef {
  float scale_v;   // lr * 2^-ev_out: gradient -> velocity LSBs of the output grid
  float mu_s;      // mu * 2^(ev_in - ev_out)
  int k;           // ev_out - ec_out: velocity LSB -> compensation LSBs (a shift, either way)
  int s;
  int delta;       // e_out - e_in (theta)
  int delta_v;     // ev_out - ev_in
  int sh_t, sh_c, sh_d, r_t, r_c;
  int qmax_t, qmax_c, qmax_v;
};

struct __align__(16) TileDesc {
  // steady path: four 16-byte loads
  float scale_v, mu_s, pow2k, pow2s_neg;
  float inv2s, qmax_t, qmax_v, d_limit;   // d_limit: bound on |V| that keeps |V * 2^k| <= 4e6
  void* theta;
  void* comp;
  void* mom;
  int n_bulk;
  int flags;
  // the rest
  int tensor;
  int count;
  Coef coef;
  const float* grad;
};
constexpr int kFormatMask = 7;       // bit 0: theta 16, bit 1: comp 16, bit 2: mom 16
constexpr int kSteady = 8;
constexpr int kRegrid = 16;      // theta's exponent changes: the exact-fp32 re-gridding path applies
constexpr int kThetaPageShift = 8, kCompPageShift = 13, kGradPageShift = 18, kMomPageShift = 23;

// Three maxima, then four counts: the order the ring expects.
struct TileScan {
  unsigned int amax_t, amax_c, amax_v, n_sat_t, n_sat_c, n_sat_v, n_nonfinite, pad;
};

__device__ __forceinline__ Coef make_coef(const TensorInfo& ti, int e_in, int e_out, int ev_in, int ev_out,
                                          float lr, float mu) {
  Coef k;
  const int delta = e_out - e_in;
  k.s = ti.s;
  k.delta = delta;
  k.delta_v = ev_out - ev_in;
  k.sh_t = ti.s + max(0, -delta);
  k.sh_c = max(0, -delta);
  k.sh_d = max(0, delta);
  k.r_t = ti.s + max(0, delta);
  k.r_c = max(0, delta);
  k.qmax_t = (1 << (ti.theta_bits - 1)) - 1;
  k.qmax_c = (1 << (ti.comp_bits - 1)) - 1;
  k.qmax_v = (1 << (ti.mom_bits - 1)) - 1;
  k.k = ev_out - (e_out - ti.s);
  k.scale_v = __fmul_rn(lr, pow2_float(-ev_out));
  k.mu_s = __fmul_rn(mu, pow2_float(ev_in - ev_out));
  return k;
}

__device__ __forceinline__ int load_q(const void* p, int bits, int e) {
  return bits == 8 ? (int)static_cast<const signed char*>(p)[e] : (int)static_cast<const short*>(p)[e];
}
__device__ __forceinline__ void store_q(void* p, int bits, int e, long long v) {
  if (bits == 8) static_cast<signed char*>(p)[e] = (signed char)v;
  else static_cast<short*>(p)[e] = (short)v;
}
__device__ __forceinline__ long long clamp_ll(long long x, long long q) {
  return x > q ? q : (x < -q ? -q : x);
}

// Elements [first, first+n) with 64-bit integers, in place on arrays in the ring or in
// global memory: exponent changes of theta or of the velocity, vectors that left the
// steady path, ragged tails.  Out of line, one copy for all formats.
__device__ __noinline__ void update_general(const Coef* coef, int tb, int cb, int vb, void* theta, void* comp,
                                            void* momv, const float* grad, int first, int n,
                                            TileScan* scan) {
  const Coef k = *coef;
  unsigned int amax_t = 0, amax_c = 0, amax_v = 0, n_sat_t = 0, n_sat_c = 0, n_sat_v = 0, n_nf = 0;
#pragma unroll 1
  for (int e = first; e < first + n; ++e) {
    const int qt = load_q(theta, tb, e), qc = load_q(comp, cb, e), qv = load_q(momv, vb, e);
    const float g = grad[e];
    // velocity: y = fma(mu_s, Qv, fl32(g * scale_v)), V = rne(y)
    const float y = __fmaf_rn(k.mu_s, (float)qv, __fmul_rn(g, k.scale_v));
    int V = __float2int_rn(y);                       // saturates, NaN -> 0
    V = max(min(V, kDLimit), -kDLimit);
    const long long Vc = clamp_ll(V, k.qmax_v);
    amax_v = max(amax_v, (unsigned int)(V < 0 ? -V : V));
    n_sat_v += (Vc != V);
    store_q(momv, vb, e, Vc);
    // the stored velocity on the compensation grid
    long long d;
    if (k.k >= 0) d = k.k > 40 ? (Vc > 0 ? kDLimit : (Vc < 0 ? -kDLimit : 0)) : clamp_ll(Vc * (1LL << k.k), kDLimit);
    else d = -k.k > 40 ? 0 : rne_shift64(Vc, -k.k);
    // Algorithm 1, statements 1-4
    const long long T = (long long)qt * (1LL << k.sh_t) + (long long)qc * (1LL << k.sh_c) - d * (1LL << k.sh_d);
    const long long P = rne_shift64(T, k.r_t);
    const long long Pc = clamp_ll(P, k.qmax_t);
    amax_t = max(amax_t, (unsigned int)(unsigned long long)(P < 0 ? -P : P));
    n_sat_t += (P != Pc);
    store_q(theta, tb, e, Pc);
    const long long R = T - Pc * (1LL << k.r_t);
    const long long Rq = rne_shift64(R, k.r_c);
    const long long Rc = clamp_ll(Rq, k.qmax_c);
    unsigned long long aR = (unsigned long long)(Rq < 0 ? -Rq : Rq);
    if (aR > 0x7fffffffULL) aR = 0x7fffffffULL;
    amax_c = max(amax_c, (unsigned int)aR);
    n_sat_c += (Rq != Rc);
    store_q(comp, cb, e, Rc);
    n_nf += ((__float_as_uint(g) & 0x7f800000u) == 0x7f800000u);
  }
  if (amax_t) atomicMax(&scan->amax_t, amax_t);
  if (amax_c) atomicMax(&scan->amax_c, amax_c);
  if (amax_v) atomicMax(&scan->amax_v, amax_v);
  if (n_sat_t) atomicAdd(&scan->n_sat_t, n_sat_t);
  if (n_sat_c) atomicAdd(&scan->n_sat_c, n_sat_c);
  if (n_sat_v) atomicAdd(&scan->n_sat_v, n_sat_v);
  if (n_nf) atomicAdd(&scan->n_nonfinite, n_nf);
}

struct SteadyCoef {
  float scale_v, mu_s, pow2k, pow2s_neg, inv2s, qmax_t, qmax_v, d_limit;
};

// Steady state (no exponent change of theta; the velocity's exponent may change, because
// mu_s and scale_v already carry both of its exponents): eight elements on the FP32 pipe
// used as an exact integer unit (see update_vector of the plain step for the technique).
// With M = 1.5 * 2^23:
//   y  = fma(mu_s, Qv, fl32(g*scale_v))      the velocity, as defined (two roundings)
//   Vm = y + M = M + rne(y) = M + V          |y| <= 4e6
//   dm = fma(V, 2^k, M) = M + d              exact product for k >= 0, rne for k < 0
//   u  = Qc - d,  Pm = fma(u, 2^-s, M + Qt), w = Pm - (M + Qt), r0 = fma(w, -2^s, u)
// theta', c' and v' are the low bits of Pm, r0 + M and Vm.  Returns false, nothing stored,
// if a value could leave the exact range or a clamp is needed.
template <int TB, int CB, int VB>
__device__ __forceinline__ bool update_vector(const Pack<TB>& pt, const Pack<CB>& pc, const Pack<VB>& pv,
                                              const Pack<32>& pg, const SteadyCoef& k, Pack<TB>& ot, Pack<CB>& oc,
                                              Pack<VB>& ov, float& amax_t, float& amax_c, float& amax_v) {
  constexpr int V = 8;
  // the scans take two elements per instruction
  float Pm[V], rm[V], Vm[V], va[2], ra[2];
  float hiP = kMagic, loP = kMagic, aR = 0.0f, aV = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const float qtM = magic_signed<TB>(pt, i);                                    // M + Qt
    const float qc = __fadd_rn(magic_signed<CB>(pc, i), -kMagic);                 // Qc
    const float qv = __fadd_rn(magic_signed<VB>(pv, i), -kMagic);                 // Qv
    const float g = __uint_as_float(pack_word(pg, i));
    const float y = __fmaf_rn(k.mu_s, qv, __fmul_rn(g, k.scale_v));
    const float vm = __fadd_rn(y, kMagic);              // M + rne(y)
    const float v = __fadd_rn(vm, -kMagic);             // Inf or NaN if y is
    const float d = __fadd_rn(__fmaf_rn(v, k.pow2k, kMagic), -kMagic);
    const float u = __fadd_rn(qc, -d);
    const float P = __fmaf_rn(u, k.inv2s, qtM);
    const float w = __fadd_rn(P, -qtM);
    const float r0 = __fmaf_rn(w, k.pow2s_neg, u);
    Pm[i] = P;
    rm[i] = __fadd_rn(r0, kMagic);
    Vm[i] = vm;
    va[i & 1] = fabsf(v);
    ra[i & 1] = fabsf(r0);
    if (i & 1) {
      aV = max3_nan(aV, va[0], va[1]);                  // NaN if any y is
      hiP = max3(hiP, Pm[i - 1], P);
      loP = min3(loP, Pm[i - 1], P);
      aR = max3(aR, ra[0], ra[1]);
    }
  }
  const float aP = fmaxf(__fadd_rn(hiP, -kMagic), __fadd_rn(kMagic, -loP));
  // |y| > 4e6 (where y + M stops being exact) shows as |V| far beyond QMAX_v, so the velocity
  // bound covers it; a NaN fails the same comparison
  if (!(aV <= k.qmax_v) | !(aV <= k.d_limit) | (aP > k.qmax_t)) return false;
  amax_t = fmaxf(amax_t, aP);
  amax_c = fmaxf(amax_c, aR);
  amax_v = fmaxf(amax_v, aV);
  ot = pack_magic<TB, V>(Pm);
  oc = pack_magic<CB, V>(rm);
  ov = pack_magic<VB, V>(Vm);
  return true;
}

// All vectors of one tile that belong to this consumer thread (8 consecutive elements per
// vector; with V = 8 a vector of B-bit mantissas is B bytes).  Returns true if the general
// path wrote into the ring.
template <int TB, int CB, int VB>
__device__ __forceinline__ bool consume_tile(const TileDesc* td, unsigned char* ring, int ctid, TileScan* scan,
                                             float& amax_t, float& amax_c, float& amax_v) {
  constexpr int V = 8;
  const uint4* q = reinterpret_cast<const uint4*>(td);
  const uint4 q0 = q[0], q1 = q[1], q2 = q[2], q3 = q[3];
  SteadyCoef k;
  k.scale_v = __uint_as_float(q0.x);
  k.mu_s = __uint_as_float(q0.y);
  k.pow2k = __uint_as_float(q0.z);
  k.pow2s_neg = __uint_as_float(q0.w);
  k.inv2s = __uint_as_float(q1.x);
  k.qmax_t = __uint_as_float(q1.y);
  k.qmax_v = __uint_as_float(q1.z);
  k.d_limit = __uint_as_float(q1.w);
  unsigned char* theta_g = reinterpret_cast<unsigned char*>(((unsigned long long)q2.y << 32) | q2.x);
  unsigned char* comp_g = reinterpret_cast<unsigned char*>(((unsigned long long)q2.w << 32) | q2.z);
  unsigned char* mom_g = reinterpret_cast<unsigned char*>(((unsigned long long)q3.y << 32) | q3.x);
  const int n_bulk = (int)q3.z, flags = (int)q3.w;
  unsigned char* theta_s = ring + ((flags >> kThetaPageShift) & 31) * kPageBytes;
  unsigned char* comp_s = ring + ((flags >> kCompPageShift) & 31) * kPageBytes;
  unsigned char* mom_s = ring + ((flags >> kMomPageShift) & 31) * kPageBytes;
  const float* grad_s = reinterpret_cast<const float*>(ring + ((flags >> kGradPageShift) & 31) * kPageBytes);
  const bool steady = (flags & kSteady) != 0;
  bool wrote_ring = false;
  const int n_vec = n_bulk / V;
  for (int v = ctid; v < n_vec; v += kThreads) {
    Pack<TB> ot;
    Pack<CB> oc;
    Pack<VB> ov;
    bool done = false;
    if (steady) {
      const Pack<TB> pt = load_pack<TB>(theta_s + v * TB);
      const Pack<CB> pc = load_pack<CB>(comp_s + v * CB);
      const Pack<VB> pv = load_pack<VB>(mom_s + v * VB);
      const Pack<32> pg = load_pack<32>(grad_s + v * V);
      done = update_vector<TB, CB, VB>(pt, pc, pv, pg, k, ot, oc, ov, amax_t, amax_c, amax_v);
    }
    if (!done) {
      update_general(&td->coef, TB, CB, VB, theta_s, comp_s, mom_s, grad_s, v * V, V, scan);
      ot = load_pack<TB>(theta_s + v * TB);
      oc = load_pack<CB>(comp_s + v * CB);
      ov = load_pack<VB>(mom_s + v * VB);
      wrote_ring = true;
    }
    store_pack<TB>(theta_g + (size_t)v * TB, ot);
    store_pack<CB>(comp_g + (size_t)v * CB, oc);
    store_pack<VB>(mom_g + (size_t)v * VB, ov);
  }
  // ragged tail (fewer than 16 elements) that the bulk copies did not bring
  const int e = n_bulk + ctid;
  if (e < td->count) update_general(&td->coef, TB, CB, VB, theta_g, comp_g, mom_g, td->grad, e, 1, scan);
  return wrote_ring;
}

// A vector of a tensor whose theta changes its exponent in this step: the velocity as in
// update_vector, then statements 2-4 of Algorithm 1 through regrid_core (kahan_sgd_kernels.cuh).
template <int TB, int CB, int VB>
__device__ __forceinline__ bool update_vector_regrid(const Pack<TB>& pt, const Pack<CB>& pc, const Pack<VB>& pv,
                                                     const Pack<32>& pg, const SteadyCoef& k, const RegridCoef& rk,
                                                     Pack<TB>& ot, Pack<CB>& oc, Pack<VB>& ov, float& amax_t,
                                                     float& amax_c, float& amax_v) {
  constexpr int V = 8;
  float yM[V], Vm[V], va[2], da[2];
  float aV = 0.0f, aD = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const float qv = __fadd_rn(magic_signed<VB>(pv, i), -kMagic);
    const float g = __uint_as_float(pack_word(pg, i));
    const float y = __fmaf_rn(k.mu_s, qv, __fmul_rn(g, k.scale_v));
    const float vm = __fadd_rn(y, kMagic);
    const float v = __fadd_rn(vm, -kMagic);
    yM[i] = __fmaf_rn(v, k.pow2k, kMagic);              // M + d
    Vm[i] = vm;
    va[i & 1] = fabsf(v);
    da[i & 1] = fabsf(__fadd_rn(yM[i], -kMagic));
    if (i & 1) {
      aV = max3_nan(aV, va[0], va[1]);
      aD = max3(aD, da[0], da[1]);
    }
  }
  if (!(aV <= k.qmax_v) | !(aV <= k.d_limit) | !(aD <= regrid_d_limit(rk))) return false;
  float at = amax_t, ac = amax_c;
  if (!regrid_core<TB, CB, V>(pt, pc, yM, rk, ot, oc, at, ac)) return false;
  amax_t = at;
  amax_c = ac;
  amax_v = fmaxf(amax_v, aV);
  ov = pack_magic<VB, V>(Vm);
  return true;
}

template <int TB, int CB, int VB>
__device__ __forceinline__ bool regrid_tile_format(const TileDesc* td, unsigned char* ring, int ctid, TileScan* scan,
                                                   float& amax_t, float& amax_c, float& amax_v) {
  constexpr int V = 8;
  const uint4* q = reinterpret_cast<const uint4*>(td);
  const uint4 q0 = q[0], q1 = q[1], q2 = q[2], q3 = q[3];
  SteadyCoef k;
  k.scale_v = __uint_as_float(q0.x);
  k.mu_s = __uint_as_float(q0.y);
  k.pow2k = __uint_as_float(q0.z);
  k.pow2s_neg = __uint_as_float(q0.w);
  k.inv2s = __uint_as_float(q1.x);
  k.qmax_t = __uint_as_float(q1.y);
  k.qmax_v = __uint_as_float(q1.z);
  k.d_limit = __uint_as_float(q1.w);
  const RegridCoef rk{pow2_float(-td->coef.delta), k.inv2s, k.pow2s_neg};
  unsigned char* theta_g = reinterpret_cast<unsigned char*>(((unsigned long long)q2.y << 32) | q2.x);
  unsigned char* comp_g = reinterpret_cast<unsigned char*>(((unsigned long long)q2.w << 32) | q2.z);
  unsigned char* mom_g = reinterpret_cast<unsigned char*>(((unsigned long long)q3.y << 32) | q3.x);
  const int n_bulk = (int)q3.z, flags = (int)q3.w;
  unsigned char* theta_s = ring + ((flags >> kThetaPageShift) & 31) * kPageBytes;
  unsigned char* comp_s = ring + ((flags >> kCompPageShift) & 31) * kPageBytes;
  unsigned char* mom_s = ring + ((flags >> kMomPageShift) & 31) * kPageBytes;
  const float* grad_s = reinterpret_cast<const float*>(ring + ((flags >> kGradPageShift) & 31) * kPageBytes);
  bool wrote_ring = false;
  const int n_vec = n_bulk / V;
  for (int v = ctid; v < n_vec; v += kThreads) {
    Pack<TB> ot;
    Pack<CB> oc;
    Pack<VB> ov;
    const Pack<TB> pt = load_pack<TB>(theta_s + v * TB);
    const Pack<CB> pc = load_pack<CB>(comp_s + v * CB);
    const Pack<VB> pv = load_pack<VB>(mom_s + v * VB);
    const Pack<32> pg = load_pack<32>(grad_s + v * V);
    if (!update_vector_regrid<TB, CB, VB>(pt, pc, pv, pg, k, rk, ot, oc, ov, amax_t, amax_c, amax_v)) {
      update_general(&td->coef, TB, CB, VB, theta_s, comp_s, mom_s, grad_s, v * V, V, scan);
      ot = load_pack<TB>(theta_s + v * TB);
      oc = load_pack<CB>(comp_s + v * CB);
      ov = load_pack<VB>(mom_s + v * VB);
      wrote_ring = true;
    }
    store_pack<TB>(theta_g + (size_t)v * TB, ot);
    store_pack<CB>(comp_g + (size_t)v * CB, oc);
    store_pack<VB>(mom_g + (size_t)v * VB, ov);
  }
  const int e = n_bulk + ctid;
  if (e < td->count) update_general(&td->coef, TB, CB, VB, theta_g, comp_g, mom_g, td->grad, e, 1, scan);
  return wrote_ring;
}

__device__ __forceinline__ void add_warp_scans(TileScan* scan, int lane, float amax_t, float amax_c, float amax_v) {
  // the exact-fp32 paths' scans are exact integers below 2^23 held in floats
  const unsigned int full = 0xffffffffu;
  const unsigned int at = __reduce_max_sync(full, (unsigned int)amax_t);
  const unsigned int ac = __reduce_max_sync(full, (unsigned int)amax_c);
  const unsigned int av = __reduce_max_sync(full, (unsigned int)amax_v);
  if (lane == 0) {
    if (at) atomicMax(&scan->amax_t, at);
    if (ac) atomicMax(&scan->amax_c, ac);
    if (av) atomicMax(&scan->amax_v, av);
  }
}

// A whole tile of a tensor whose theta changes its exponent, for one consumer thread.  Out of
// line, called once per such tile with next to nothing live around the call, so that its
// registers cost the tiles whose exponent does not change nothing.
__device__ __noinline__ void regrid_tile(const TileDesc* td, TileScan* scan, unsigned char* ring) {
  const int ctid = threadIdx.x;
  float amax_t = 0.0f, amax_c = 0.0f, amax_v = 0.0f;
  bool wrote_ring;
  switch (td->flags & kFormatMask) {
    case 0: wrote_ring = regrid_tile_format<8, 8, 8>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 1: wrote_ring = regrid_tile_format<16, 8, 8>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 2: wrote_ring = regrid_tile_format<8, 16, 8>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 3: wrote_ring = regrid_tile_format<16, 16, 8>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 4: wrote_ring = regrid_tile_format<8, 8, 16>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 5: wrote_ring = regrid_tile_format<16, 8, 16>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    case 6: wrote_ring = regrid_tile_format<8, 16, 16>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
    default: wrote_ring = regrid_tile_format<16, 16, 16>(td, ring, ctid, scan, amax_t, amax_c, amax_v); break;
  }
  add_warp_scans(scan, threadIdx.x & 31, amax_t, amax_c, amax_v);
  if (wrote_ring) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Exponent of the velocity for the next step.  The velocity's maximum moves with every
// gradient, so it keeps its exponent while its largest mantissa stays in (QMAX/4, QMAX] and
// otherwise takes the tight fit (coarser at once, finer only after a fourfold drop).
__host__ __device__ __forceinline__ int next_exponent_velocity(unsigned int amax, int bits, int ev_out, int amax_mode) {
  const unsigned int q = (1u << (bits - 1)) - 1u;
  if (amax <= q && 4ull * amax > q) return ev_out;
  return next_exponent(amax, bits, ev_out, amax_mode);
}

// What the producer knows about a tile's tensor.
struct TensorMeta {
  TensorInfo ti;
  const float* grad;
  float lr, mu;
  int e_in, e_out, ev_in, ev_out;
};

struct Policy {
  static constexpr int kStreams = 4;          // gradient, theta, c, v
  static constexpr int kConsumerWarps = kWarps;
  static constexpr int kAmax = 3, kCounts = 4;
  // no limit on tiles in flight: with 7 to 12 pages per tile the ring holds little more than two
  // tiles anyway, and the limit measured equal (momentum) or 0.5 % slower (ADAM) in long steps
  static constexpr int kLongStepTiles = 1 << 30;
  static constexpr bool kGradEvictFirstBeyondL2 = false;
  using Params = StepParams;
  using Info = TensorInfo;
  using State = TensorState;
  using TileDesc = mom::TileDesc;
  using TileScan = mom::TileScan;
  using Meta = TensorMeta;

  // The exponents the tensor reads and writes in the step of phase ph, derived from the record
  // the preceding step left (one 32-byte load), and the per-step arguments.
  static __device__ __forceinline__ Meta load_meta(const Params& p, const StepArgs& a, int t, int ph, const Info* ti) {
    Meta m;
    m.ti = ti ? *ti : p.ws.info[t];
    m.grad = p.inline_args ? a.grads[t] : p.ws.grad_ptr[t];
    m.lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];
    m.mu = p.inline_args ? a.mus[t] : p.ws.mu[t];
    const int prev = ph == 0 ? 2 : ph - 1;
    const int4* rec = reinterpret_cast<const int4*>(&p.ws.state[(size_t)prev * p.ws.slab + t]);
    const int4 r0 = __ldcg(rec), r1 = __ldcg(rec + 1);     // exp_theta exp_mom amax[0] amax[1] | amax[2] ovr_theta ovr_mom -
    m.e_in = r0.x;
    m.ev_in = r0.y;
    m.e_out = r1.y ? r1.y - kOvrBias : next_exponent((unsigned)r0.z, m.ti.theta_bits, m.e_in, p.amax_mode);
    m.ev_out = r1.z ? r1.z - kOvrBias : next_exponent_velocity((unsigned)r1.x, m.ti.mom_bits, m.ev_in, p.amax_mode);
    return m;
  }
  static __device__ __forceinline__ void record(const Params& p, int t, int ph, const Meta& m) {
    const int next = ph == 2 ? 0 : ph + 1;
    TensorState* now = &p.ws.state[(size_t)ph * p.ws.slab + t];
    now->exp_theta = m.e_out;
    now->exp_mom = m.ev_out;
    int4* nx = reinterpret_cast<int4*>(&p.ws.state[(size_t)next * p.ws.slab + t]);
    nx[0] = make_int4(0, 0, 0, 0);
    nx[1] = make_int4(0, 0, 0, 0);
  }
  static __device__ __forceinline__ void streams(const Meta& m, const unsigned char* (&base)[kStreams],
                                                 int (&bytes)[kStreams]) {
    base[0] = reinterpret_cast<const unsigned char*>(m.grad);
    bytes[0] = 4;
    base[1] = static_cast<const unsigned char*>(m.ti.theta);
    bytes[1] = m.ti.theta_bits >> 3;
    base[2] = static_cast<const unsigned char*>(m.ti.comp);
    bytes[2] = m.ti.comp_bits >> 3;
    base[3] = static_cast<const unsigned char*>(m.ti.mom);
    bytes[3] = m.ti.mom_bits >> 3;
  }
  static __device__ __forceinline__ void fill_desc(TileDesc& td, const Params&, const Meta& meta, int tensor, int count,
                                                   int n_bulk, const int (&page)[kStreams],
                                                   const unsigned char* const (&gptr)[kStreams]) {
    const TensorInfo& ti = meta.ti;
    const Coef coef = make_coef(ti, meta.e_in, meta.e_out, meta.ev_in, meta.ev_out, meta.lr, meta.mu);
    // velocity LSB -> compensation LSBs as a float factor; beyond +-30 the steady path
    // is never exact (k large) or the increment is always zero (k very negative)
    const int kk = max(-40, min(30, coef.k));
    td.scale_v = coef.scale_v;
    td.mu_s = coef.mu_s;
    td.pow2k = pow2_float(kk);
    td.pow2s_neg = -pow2_float(coef.s);
    td.inv2s = pow2_float(-coef.s);
    td.qmax_t = (float)coef.qmax_t;
    td.qmax_v = (float)coef.qmax_v;
    td.d_limit = coef.k > 22 ? 0.5f : (coef.k > 0 ? 4000000.0f * pow2_float(-coef.k) : 4000000.0f);
    td.theta = const_cast<unsigned char*>(gptr[1]);
    td.comp = const_cast<unsigned char*>(gptr[2]);
    td.mom = const_cast<unsigned char*>(gptr[3]);
    td.n_bulk = n_bulk;
    td.flags = ((ti.theta_bits == 16 ? 1 : 0) | (ti.comp_bits == 16 ? 2 : 0) | (ti.mom_bits == 16 ? 4 : 0)) |
               (coef.delta == 0 ? kSteady : 0) |
               // a coarser grid splits theta's mantissa at bit delta: that needs delta <= theta_bits - 1
               ((coef.delta != 0 && coef.delta <= ti.theta_bits - 1) ? kRegrid : 0) | (page[1] << kThetaPageShift) |
               (page[2] << kCompPageShift) | (page[0] << kGradPageShift) | (page[3] << kMomPageShift);
    td.tensor = tensor;
    td.count = count;
    td.coef = coef;
    td.grad = reinterpret_cast<const float*>(gptr[0]);
  }
  static __device__ __forceinline__ void consume(const TileDesc* td, TileScan* scan, unsigned char* smem, int ctid,
                                                 int lane) {
    if (td->flags & kRegrid) {
      regrid_tile(td, scan, smem);
      return;
    }
    float amax_t = 0.0f, amax_c = 0.0f, amax_v = 0.0f;
    bool wrote_ring;
    switch (td->flags & kFormatMask) {
      case 0: wrote_ring = consume_tile<8, 8, 8>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 1: wrote_ring = consume_tile<16, 8, 8>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 2: wrote_ring = consume_tile<8, 16, 8>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 3: wrote_ring = consume_tile<16, 16, 8>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 4: wrote_ring = consume_tile<8, 8, 16>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 5: wrote_ring = consume_tile<16, 8, 16>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      case 6: wrote_ring = consume_tile<8, 16, 16>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
      default: wrote_ring = consume_tile<16, 16, 16>(td, smem, ctid, scan, amax_t, amax_c, amax_v); break;
    }
    add_warp_scans(scan, lane, amax_t, amax_c, amax_v);
    // if the general path wrote into the ring, order those writes before the bulk copy
    // that refills the pages
    if (wrote_ring) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
};

constexpr size_t kSharedBytes = ring_shared_bytes<Policy>();

__global__ void __launch_bounds__(kBlock, 1)
ksgd_momentum_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ StepArgs a) {
  ring_step<Policy>(p, a);
}

}  // namespace mom
}  // namespace ksgd
