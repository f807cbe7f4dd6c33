// Device code of the lazy update (SGD with Kahan summation, Algorithm 1 of
// arXiv 1810.05486) in dynamic fixed-point, for sm_100a.
//
// One launch of ksgd_step_kernel performs, for a ragged list of tensors:
//   - Algorithm 1, statement 1: the fp32 gradient increment is rounded onto the
//     compensation grid (one binary32 multiply + round-to-nearest-even);
//   - statements 2-4: T = theta + c - d is formed exactly in integers, rounded onto
//     theta's grid (theta'), and what the rounding lost is stored back as c';
//   - the per-tensor max scans (warp reduce -> block reduce -> one atomicMax per
//     block) that dynamic fixed-point needs to choose the next exponent (Section 5);
//   - in the last block to finish, the exponent choice itself for every tensor.
// The pass is bound by HBM traffic: 2*m/8 + 2*n/8 + 4 bytes per parameter.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace ksgd {

constexpr int kThreads = 256;        // threads per block
constexpr int kChunk = 8192;         // elements of one tensor handled by one block
constexpr int kInlineArgs = 256;     // lists up to this long pass grads/lrs as kernel parameters
constexpr int kUploadBatch = 1024;   // tensors per launch of the argument-upload kernel
constexpr int kDLimit = 1 << 30;     // clamp of the quantized increment, in compensation LSBs
constexpr int kMaxDelta = 8;         // largest exponent change per step
constexpr int kExpMin = -64, kExpMax = 64;

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
  int index;   // chunk number inside that tensor: elements [index*kChunk, ...)
};

// Device-side view of the caller's workspace.
struct Workspace {
  int* exp_cur;                    // [n] exponent of the stored mantissas
  int* exp_next;                   // [n] exponent the coming step writes
  unsigned int* amax_last;         // [2n] max scans of the last finished step (theta | comp)
  unsigned long long* counters;    // [3n] cumulative: sat_theta | sat_comp | nonfinite
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

// Everything a block needs to know about its tensor for this step.
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

// Per-thread reduction state.
struct Scan {
  unsigned int amax_t = 0;
  unsigned int amax_c = 0;
  unsigned int n_sat_t = 0;
  unsigned int n_sat_c = 0;
  unsigned int n_nonfinite = 0;
};

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

// Algorithm 1 for one element with 64-bit intermediates; handles every exponent change,
// saturation and non-finite gradients.  HAS_COMP = false is Eq. 1 (plain low-precision SGD).
template <bool HAS_COMP>
__device__ __forceinline__ void update_general(int qt, int qc, float g, const StepCoef& k,
                                               int& qt_new, int& qc_new, Scan& sc) {
  const int d = quantize_increment(g, k.scale);
  long long T = (long long)qt * (1LL << k.sh_t) - (long long)d * (1LL << k.sh_d);
  if (HAS_COMP) T += (long long)qc * (1LL << k.sh_c);
  const long long P = rne_shift64(T, k.r_t);
  const long long Pc = P > k.qmax_t ? k.qmax_t : (P < -k.qmax_t ? -k.qmax_t : P);
  qt_new = (int)Pc;
  const unsigned long long aP = (unsigned long long)(P < 0 ? -P : P);
  sc.amax_t = max(sc.amax_t, (unsigned int)aP);
  sc.n_sat_t += (P != Pc);
  if (HAS_COMP) {
    const long long R = T - Pc * (1LL << k.r_t);
    const long long Rq = rne_shift64(R, k.r_c);
    const long long Rc = Rq > k.qmax_c ? k.qmax_c : (Rq < -k.qmax_c ? -k.qmax_c : Rq);
    qc_new = (int)Rc;
    unsigned long long aR = (unsigned long long)(Rq < 0 ? -Rq : Rq);
    if (aR > 0x7fffffffULL) aR = 0x7fffffffULL;
    sc.amax_c = max(sc.amax_c, (unsigned int)aR);
    sc.n_sat_c += (Rq != Rc);
  } else {
    qc_new = 0;
  }
  const unsigned int gb = __float_as_uint(g) & 0x7f800000u;
  sc.n_nonfinite += (gb == 0x7f800000u);
}

// ----------------------------------------------------------------------------------------
// 16-byte vector access helpers.  V elements of B bits each (V*B/8 is 8, 16 or 32 bytes).

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
__device__ __forceinline__ Pack<BYTES> load_pack_stream(const void* p) {  // read-once data
  Pack<BYTES> r;
  if constexpr (BYTES == 8) {
    r.v = __ldcs(reinterpret_cast<const uint2*>(p));
  } else if constexpr (BYTES == 16) {
    r.v = __ldcs(reinterpret_cast<const uint4*>(p));
  } else {
#pragma unroll
    for (int i = 0; i < BYTES / 16; ++i) r.v[i] = __ldcs(reinterpret_cast<const uint4*>(p) + i);
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
// One vector of V elements: fast 32-bit path for the steady state (no exponent change,
// s >= 1 or plain mode), falling back to update_general for the whole vector when any
// element saturates theta or has a non-finite gradient.

template <int TB, int CB, int V>
__device__ __forceinline__ void update_vector(const Pack<V * TB / 8>& pt,
                                              const Pack<(CB ? V * CB / 8 : 8)>& pc,
                                              const Pack<V * 4>& pg, const StepCoef& k,
                                              bool steady, Pack<V * TB / 8>& ot,
                                              Pack<(CB ? V * CB / 8 : 8)>& oc, Scan& sc) {
  constexpr bool HAS_COMP = CB != 0;
  int qt[V], qc[V], nt[V], nc[V];
  float g[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    qt[i] = unpack_elem<TB>(pt, i);
    qc[i] = HAS_COMP ? unpack_elem<(CB ? CB : 8)>(pc, i) : 0;
    g[i] = __uint_as_float(pack_word(pg, i));
  }

  bool redo = !steady;
  if (steady) {
    // T = qt*2^s + u with u = qc - d.  Rounding T by s bits to nearest-even only needs
    // u, the parity of the truncated quotient and qt itself, all within 32 bits.
    const int s = k.s;
    const int hm1 = HAS_COMP ? ((1 << (s - 1)) - 1) : 0;
    int mxP = INT_MIN, mnP = INT_MAX, mxR = 0, mnR = 0;
    float nf = 0.0f;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const int d = quantize_increment(g[i], k.scale);
      nf = fmaf(g[i], 0.0f, nf);          // stays 0 unless some g is Inf or NaN
      const int u = qc[i] - d;
      int P, r0;
      if (HAS_COMP) {
        const int par = (qt[i] + (u >> s)) & 1;
        const int w = (u + hm1 + par) >> s;
        P = qt[i] + w;
        r0 = u - (w << s);
      } else {
        P = qt[i] + u;
        r0 = 0;
      }
      nt[i] = P;
      nc[i] = r0;
      mxP = max(mxP, P);
      mnP = min(mnP, P);
      if (HAS_COMP) {
        mxR = max(mxR, r0);
        mnR = min(mnR, r0);
      }
    }
    redo = (mxP > k.qmax_t) | (mnP < -k.qmax_t) | (nf != nf);
    if (!redo) {
      sc.amax_t = max(sc.amax_t, (unsigned int)max(mxP, -mnP));
      if (HAS_COMP) sc.amax_c = max(sc.amax_c, (unsigned int)max(mxR, -mnR));
    }
  }
  if (redo) {
#pragma unroll
    for (int i = 0; i < V; ++i) update_general<HAS_COMP>(qt[i], qc[i], g[i], k, nt[i], nc[i], sc);
  }
  ot = pack_elems<TB, V>(nt);
  if constexpr (HAS_COMP) oc = pack_elems<CB, V>(nc);
}

template <int TB, int CB>
__device__ __forceinline__ void process_chunk(void* theta_v, void* comp_v, const float* grad,
                                              int count, const StepCoef& k, Scan& sc) {
  constexpr bool HAS_COMP = CB != 0;
  constexpr int V = (TB == 8) ? 16 : 8;              // one 16-byte load of theta per vector
  constexpr int TBYTES = V * TB / 8;
  constexpr int CBYTES = HAS_COMP ? V * CB / 8 : 8;
  constexpr int ITERS = kChunk / (kThreads * V);
  using ThetaT = typename std::conditional<TB == 8, signed char, short>::type;
  using CompT = typename std::conditional<CB == 16, short, signed char>::type;
  ThetaT* theta = static_cast<ThetaT*>(theta_v);
  CompT* comp = static_cast<CompT*>(comp_v);
  const bool steady = (k.delta == 0) && (!HAS_COMP || k.s >= 1);

  if (count == kChunk) {
    Pack<TBYTES> pt[ITERS];
    Pack<CBYTES> pc[ITERS];
    Pack<V * 4> pg[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int e = (it * kThreads + threadIdx.x) * V;
      pt[it] = load_pack<TBYTES>(theta + e);
      if constexpr (HAS_COMP) pc[it] = load_pack<CBYTES>(comp + e);
      pg[it] = load_pack_stream<V * 4>(grad + e);
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int e = (it * kThreads + threadIdx.x) * V;
      Pack<TBYTES> ot;
      Pack<CBYTES> oc;
      update_vector<TB, CB, V>(pt[it], pc[it], pg[it], k, steady, ot, oc, sc);
      store_pack<TBYTES>(theta + e, ot);
      if constexpr (HAS_COMP) store_pack<CBYTES>(comp + e, oc);
    }
  } else {
    const int n_vec = count / V;
    for (int v = threadIdx.x; v < n_vec; v += kThreads) {
      const int e = v * V;
      Pack<TBYTES> pt = load_pack<TBYTES>(theta + e), ot;
      Pack<CBYTES> pc, oc;
      if constexpr (HAS_COMP) pc = load_pack<CBYTES>(comp + e);
      Pack<V * 4> pg = load_pack_stream<V * 4>(grad + e);
      update_vector<TB, CB, V>(pt, pc, pg, k, steady, ot, oc, sc);
      store_pack<TBYTES>(theta + e, ot);
      if constexpr (HAS_COMP) store_pack<CBYTES>(comp + e, oc);
    }
    // ragged tail: fewer than V elements, one per thread
    const int e = n_vec * V + threadIdx.x;
    if (threadIdx.x < V && e < count) {
      int nt, nc;
      update_general<HAS_COMP>((int)theta[e], HAS_COMP ? (int)comp[e] : 0, grad[e], k, nt, nc, sc);
      theta[e] = (ThetaT)nt;
      if constexpr (HAS_COMP) comp[e] = (CompT)nc;
    }
  }
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

__global__ void __launch_bounds__(kThreads)
ksgd_step_kernel(const __grid_constant__ StepParams p, const __grid_constant__ InlineArgs a) {
  __shared__ unsigned int red[5][kThreads / 32];
  __shared__ int is_last;

  const ChunkRef cr = p.ws.chunks[blockIdx.x];
  const int t = cr.tensor;
  const TensorInfo ti = p.ws.info[t];
  const int e_in = p.ws.exp_cur[t];
  const int e_out = p.ws.exp_next[t];
  const float* grad = p.inline_args ? a.grads[t] : p.ws.grad_ptr[t];
  const float lr = p.inline_args ? a.lrs[t] : p.ws.lr[t];

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

  const long long base = (long long)cr.index * kChunk;
  const long long left = ti.numel - base;
  const int count = left < (long long)kChunk ? (int)left : kChunk;
  const float* g = grad + base;

  Scan sc;
  if (ti.theta_bits == 8) {
    signed char* th = static_cast<signed char*>(ti.theta) + base;
    if (ti.comp_bits == 8) process_chunk<8, 8>(th, static_cast<signed char*>(ti.comp) + base, g, count, k, sc);
    else if (ti.comp_bits == 16) process_chunk<8, 16>(th, static_cast<short*>(ti.comp) + base, g, count, k, sc);
    else process_chunk<8, 0>(th, nullptr, g, count, k, sc);
  } else {
    short* th = static_cast<short*>(ti.theta) + base;
    if (ti.comp_bits == 8) process_chunk<16, 8>(th, static_cast<signed char*>(ti.comp) + base, g, count, k, sc);
    else if (ti.comp_bits == 16) process_chunk<16, 16>(th, static_cast<short*>(ti.comp) + base, g, count, k, sc);
    else process_chunk<16, 0>(th, nullptr, g, count, k, sc);
  }

  // block-level reduction of the scans, then one atomic per quantity per block
  const unsigned int full = 0xffffffffu;
  const unsigned int wa_t = __reduce_max_sync(full, sc.amax_t);
  const unsigned int wa_c = __reduce_max_sync(full, sc.amax_c);
  const unsigned int rare = sc.n_sat_t | sc.n_sat_c | sc.n_nonfinite;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { red[0][warp] = wa_t; red[1][warp] = wa_c; }
  const int any_rare = __syncthreads_or(rare != 0u);
  if (any_rare) {
    const unsigned int w0 = __reduce_add_sync(full, sc.n_sat_t);
    const unsigned int w1 = __reduce_add_sync(full, sc.n_sat_c);
    const unsigned int w2 = __reduce_add_sync(full, sc.n_nonfinite);
    if (lane == 0) { red[2][warp] = w0; red[3][warp] = w1; red[4][warp] = w2; }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    unsigned int at = 0, ac = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) { at = max(at, red[0][w]); ac = max(ac, red[1][w]); }
    if (at) atomicMax(&p.ws.amax_acc[t], at);
    if (ac) atomicMax(&p.ws.amax_acc[p.n_tensors + t], ac);
    if (any_rare) {
      unsigned int c0 = 0, c1 = 0, c2 = 0;
#pragma unroll
      for (int w = 0; w < kThreads / 32; ++w) { c0 += red[2][w]; c1 += red[3][w]; c2 += red[4][w]; }
      if (c0) atomicAdd(&p.ws.counters[t], (unsigned long long)c0);
      if (c1) atomicAdd(&p.ws.counters[p.n_tensors + t], (unsigned long long)c1);
      if (c2) atomicAdd(&p.ws.counters[2 * p.n_tensors + t], (unsigned long long)c2);
    }
    __threadfence();
    const unsigned int done = atomicAdd(p.ws.ticket, 1u);
    is_last = (done == gridDim.x - 1u);
  }
  __syncthreads();
  if (!is_last) return;

  // Last block to finish: every other block has published its scans and has long since
  // read the exponents, so they can be rotated here.  No block ever waits for another.
  __threadfence();
  for (int i = threadIdx.x; i < p.n_tensors; i += kThreads) {
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
