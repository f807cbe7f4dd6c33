// fp32 <-> dynamic fixed-point conversion kernels (Section 1 of arXiv 1810.05486: uniform
// linear quantization with one shared exponent per tensor; Section 5: the exponent comes
// from a scan of the maximum).  Used when a model enters or leaves the fixed-point format,
// and once per step and gradient tensor when the gradients are fixed-point tensors too.
//
// Import is two passes over the source, both bound by HBM traffic: a max scan (16-byte
// loads) whose last block picks the exponent on the device and leaves it in device memory,
// and the quantization, which reads that exponent from device memory (no host round trip
// in between) and writes theta and c; a warp works on 512 consecutive elements at a time with
// 16-byte accesses per lane to the binary32 array and to 8-bit mantissa arrays (the packed
// words are transposed among four lanes for that), 8-byte ones to 16-bit arrays; what is left
// over, and arrays that do not start on 16-byte boundaries, take narrower paths.  All scalings
// are by powers of two and every intermediate is exactly representable in binary32, so the
// only roundings are the ones the definition names.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace ksgd {
namespace convert {

constexpr int kThreads = 256;
constexpr int kExpLo = -64, kExpHi = 64;

// Device scratch of the scan: the running maximum (bit pattern of a non-negative float,
// ordered like the values) and the count of blocks that have finished.  Both are zero
// between calls: the caller clears them once, the last block of every scan clears them again.
struct ScanScratch {
  unsigned int amax_bits;
  unsigned int done;
};

// Smallest exponent in [-64, 64] whose b-bit grid holds amax (0 for an all-zero tensor).
__host__ __device__ inline int fit_exponent(float amax, int bits) {
  if (!(amax > 0.0f)) return 0;
  const double q = (double)((1 << (bits - 1)) - 1);
  int e = kExpLo;
  while (e < kExpHi && (double)amax > ldexp(q, e)) ++e;
  return e;
}

__device__ __forceinline__ unsigned int finite_abs_bits(float x) {
  const unsigned int b = __float_as_uint(x) & 0x7fffffffu;
  return b < 0x7f800000u ? b : 0u;
}

// max |x| over the finite elements; the last block to finish turns it into the exponent and
// stores it at *exp_out (device memory).  x 16-byte aligned: float4 loads; else scalar.
// (Ordinary loads: a source that fits the L2 is then still there for the quantization.)
__global__ void __launch_bounds__(kThreads) absmax_fit_kernel(const float* __restrict__ x, long long n, int bits,
                                                              ScanScratch* scratch, int* exp_out) {
  unsigned int m = 0u;
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  if ((reinterpret_cast<uintptr_t>(x) & 15u) == 0u) {
    const long long n4 = n >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    long long i = tid;
    for (; i + 3 * stride < n4; i += 4 * stride) {      // four loads in flight per thread
      const float4 a = __ldg(x4 + i), b = __ldg(x4 + i + stride), c = __ldg(x4 + i + 2 * stride),
                   d = __ldg(x4 + i + 3 * stride);
      m = max(m, max(max(finite_abs_bits(a.x), finite_abs_bits(a.y)), max(finite_abs_bits(a.z), finite_abs_bits(a.w))));
      m = max(m, max(max(finite_abs_bits(b.x), finite_abs_bits(b.y)), max(finite_abs_bits(b.z), finite_abs_bits(b.w))));
      m = max(m, max(max(finite_abs_bits(c.x), finite_abs_bits(c.y)), max(finite_abs_bits(c.z), finite_abs_bits(c.w))));
      m = max(m, max(max(finite_abs_bits(d.x), finite_abs_bits(d.y)), max(finite_abs_bits(d.z), finite_abs_bits(d.w))));
    }
    for (; i < n4; i += stride) {
      const float4 a = __ldg(x4 + i);
      m = max(m, max(max(finite_abs_bits(a.x), finite_abs_bits(a.y)), max(finite_abs_bits(a.z), finite_abs_bits(a.w))));
    }
    for (long long j = (n4 << 2) + tid; j < n; j += stride) m = max(m, finite_abs_bits(x[j]));
  } else {
    for (long long j = tid; j < n; j += stride) m = max(m, finite_abs_bits(x[j]));
  }
  __shared__ unsigned int warp_max[kThreads / 32];
  __shared__ int is_last;
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int b = 0u;
    for (int w = 0; w < kThreads / 32; ++w) b = max(b, warp_max[w]);
    if (b) atomicMax(&scratch->amax_bits, b);
    __threadfence();
    is_last = atomicAdd(&scratch->done, 1u) == gridDim.x - 1u;
    if (is_last) {
      __threadfence();
      const unsigned int all = __ldcg(&scratch->amax_bits);
      *exp_out = fit_exponent(__uint_as_float(all), bits);
      scratch->amax_bits = 0u;
      scratch->done = 0u;
    }
  }
}

// One element in binary32, every step exact except the two roundings of the definition:
//   Q_theta = clamp(rne(x / 2^e)),  Q_c = clamp(rne((x - Q_theta*2^e) / 2^(e-s))).
// x / 2^e is an exact scaling (a result below the normal range is far below half a unit and
// rounds to 0 either way).  Clamping to +-(QMAX + 1/4) first and rounding then gives the same
// integer as rounding first and clamping to +-QMAX (everything from QMAX + 1/4 on rounds to
// QMAX), and keeps the value where adding M = 1.5 * 2^23 rounds it to the nearest integer,
// ties to even; the integer is then the low bits of M's bit pattern (no conversion
// instruction).  x/2^e - Q_theta is a difference of two floats that either lie within a
// factor of two of each other or has a result of fewer bits than x/2^e, so it is exact
// whenever the result can still matter (beyond 2^24 it only has to be large).
// NaN -> 0, +-Inf -> +-QMAX with nothing left for c.
// qt and qc come back as the bit patterns of M + Q: the low 8 or 16 bits are the mantissa in
// two's complement (M's own low bits are zero), which is all the packing below takes.
template <int TB, int CB>
__device__ __forceinline__ void quantize_one(float x, float inv2e, float pow2s, int& qt, int& qc) {
  constexpr float kM = 12582912.0f;
  constexpr int kMBits = 0x4B400000;
  constexpr float bound_t = (float)((1 << (TB - 1)) - 1) + 0.25f;
  constexpr float bound_c = (float)((1 << ((CB ? CB : 8) - 1)) - 1) + 0.25f;
  const float xs = __fmul_rn(x, inv2e);
  const float tm = __fadd_rn(fminf(fmaxf(xs, -bound_t), bound_t), kM);   // NaN -> a finite bound, fixed below
  qt = x != x ? kMBits : __float_as_int(tm);
  qc = kMBits;
  if constexpr (CB != 0) {
    const float t = __fadd_rn(tm, -kM);
    const float r = __fmul_rn(__fadd_rn(xs, -t), pow2s);
    const float rm = __fadd_rn(fminf(fmaxf(r, -bound_c), bound_c), kM);
    qc = !(fabsf(x) < __int_as_float(0x7f800000)) ? kMBits : __float_as_int(rm);   // NaN or Inf: nothing left for c
  }
}

// The mantissas of four such bit patterns packed into one (8-bit) or two (16-bit) words by
// byte selection.
__device__ __forceinline__ unsigned int pack4x8(const int (&q)[4]) {
  const unsigned int lo = __byte_perm((unsigned int)q[0], (unsigned int)q[1], 0x0040);
  const unsigned int hi = __byte_perm((unsigned int)q[2], (unsigned int)q[3], 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}
__device__ __forceinline__ uint2 pack4x16(const int (&q)[4]) {
  return make_uint2(__byte_perm((unsigned int)q[0], (unsigned int)q[1], 0x5410),
                    __byte_perm((unsigned int)q[2], (unsigned int)q[3], 0x5410));
}

// 4 x 4 transposition of 32-bit words inside every group of four neighbouring lanes: word k
// of lane 4q + a becomes word a of lane 4q + k.  Two exchanges (with the lane two away, then
// with the neighbour), four shuffles.  It turns "lane l holds the words of groups l, l + 32,
// l + 64, l + 96" (how coalesced 16-byte accesses to the binary32 array hand them out) into
// "lane l holds four neighbouring words" (one 16-byte access to an 8-bit array) and back, so
// that an 8-bit array is read and written 16 bytes per lane too instead of 4.
__device__ __forceinline__ void quad_transpose(unsigned int (&a)[4], int lane) {
  const unsigned int full = 0xffffffffu;
  const bool up2 = (lane & 2) != 0, up1 = (lane & 1) != 0;
  unsigned int s0 = up2 ? a[0] : a[2], s1 = up2 ? a[1] : a[3];
  s0 = __shfl_xor_sync(full, s0, 2);
  s1 = __shfl_xor_sync(full, s1, 2);
  if (up2) { a[0] = s0; a[1] = s1; } else { a[2] = s0; a[3] = s1; }
  unsigned int t0 = up1 ? a[0] : a[1], t1 = up1 ? a[2] : a[3];
  t0 = __shfl_xor_sync(full, t0, 1);
  t1 = __shfl_xor_sync(full, t1, 1);
  if (up1) { a[0] = t0; a[2] = t1; } else { a[1] = t0; a[3] = t1; }
}

// A warp's piece of the arrays in the main loops below: 512 consecutive elements, i.e. 128
// groups of four; lane l works on groups l, l + 32, l + 64 and l + 96 of the piece.
constexpr int kPiece = 512;

// Byte offset, inside a piece of an 8-bit array, of the 16 bytes lane l holds after the
// transposition: groups 32 * (l % 4) + 4 * (l / 4) ... + 3.
__device__ __forceinline__ int piece_offset8(int lane) { return 128 * (lane & 3) + 16 * (lane >> 2); }

// (streaming stores: the mantissas are not read again soon, and must not push the source of an
// import out of L2 before the quantization has read it)
template <int BITS>
__device__ __forceinline__ void store_piece(void* base, long long piece, int lane, const int (&q)[4][4]) {
  if constexpr (BITS == 8) {
    unsigned int w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = pack4x8(q[j]);
    quad_transpose(w, lane);
    __stcs(reinterpret_cast<uint4*>(static_cast<char*>(base) + piece * kPiece + piece_offset8(lane)),
           make_uint4(w[0], w[1], w[2], w[3]));
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      __stcs(reinterpret_cast<uint2*>(base) + piece * (kPiece / 4) + 32 * j + lane, pack4x16(q[j]));
  }
}

template <int BITS>
__device__ __forceinline__ void store4(void* base, long long i4, const int (&q)[4]) {
  if constexpr (BITS == 8) __stcs(reinterpret_cast<unsigned int*>(base) + i4, pack4x8(q));
  else __stcs(reinterpret_cast<uint2*>(base) + i4, pack4x16(q));
}

template <int BITS>
__device__ __forceinline__ void store1(void* base, long long i, int q) {
  if constexpr (BITS == 8) static_cast<signed char*>(base)[i] = (signed char)q;
  else static_cast<short*>(base)[i] = (short)q;
}

// exp_dev != nullptr: the exponent is read from device memory (left there by the scan);
// otherwise e_fixed applies.  Four consecutive elements per thread and access when the three
// arrays are aligned for it (16 bytes for x; 4 or 8 for theta and c), one otherwise.
template <int TB, int CB>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const float* __restrict__ x, void* theta, void* comp,
                                                            long long n, const int* exp_dev, int e_fixed, int s) {
  const int e = exp_dev ? __ldcg(exp_dev) : e_fixed;
  const float inv2e = __int_as_float((127 - e) << 23);      // |e| <= 64: a normal power of two
  const float pow2s = __int_as_float((127 + s) << 23);
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const bool vec = ((reinterpret_cast<uintptr_t>(x) & 15u) | (reinterpret_cast<uintptr_t>(theta) & (TB / 2 - 1)) |
                    (CB ? (reinterpret_cast<uintptr_t>(comp) & ((CB ? CB : 8) / 2 - 1)) : 0)) == 0u;
  long long done = 0;
  // Main loop, when every array starts on a 16-byte boundary: a warp takes pieces of 512
  // elements; four coalesced 16-byte loads per lane, 16-byte stores to 8-bit arrays (after a
  // transposition among four lanes), 8-byte stores to 16-bit arrays.
  constexpr int CBS = CB ? CB : 8;
  const bool pieces = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(theta) |
                        (CB ? reinterpret_cast<uintptr_t>(comp) : 0)) & 15u) == 0u;
  if (pieces) {
    const int lane = threadIdx.x & 31;
    const long long n_pieces = n / kPiece;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    for (long long pc = tid >> 5; pc < n_pieces; pc += stride >> 5) {
      float4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = __ldcs(x4 + pc * (kPiece / 4) + 32 * j + lane);   // last use of the source
      int qt[4][4], qc[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        quantize_one<TB, CB>(v[j].x, inv2e, pow2s, qt[j][0], qc[j][0]);
        quantize_one<TB, CB>(v[j].y, inv2e, pow2s, qt[j][1], qc[j][1]);
        quantize_one<TB, CB>(v[j].z, inv2e, pow2s, qt[j][2], qc[j][2]);
        quantize_one<TB, CB>(v[j].w, inv2e, pow2s, qt[j][3], qc[j][3]);
      }
      store_piece<TB>(theta, pc, lane, qt);
      if constexpr (CB != 0) store_piece<CBS>(comp, pc, lane, qc);
    }
    done = n_pieces * kPiece;
  }
  if (vec) {
    const long long n4 = n >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(x);
#pragma unroll 2
    for (long long i = (done >> 2) + tid; i < n4; i += stride) {
      const float4 v = __ldcs(x4 + i);       // last use of the source: let it leave the caches first
      int qt[4], qc[4];
      quantize_one<TB, CB>(v.x, inv2e, pow2s, qt[0], qc[0]);
      quantize_one<TB, CB>(v.y, inv2e, pow2s, qt[1], qc[1]);
      quantize_one<TB, CB>(v.z, inv2e, pow2s, qt[2], qc[2]);
      quantize_one<TB, CB>(v.w, inv2e, pow2s, qt[3], qc[3]);
      store4<TB>(theta, i, qt);
      if constexpr (CB != 0) store4<(CB ? CB : 8)>(comp, i, qc);
    }
    done = n4 << 2;
  }
  for (long long j = done + tid; j < n; j += stride) {
    int qt, qc;
    quantize_one<TB, CB>(x[j], inv2e, pow2s, qt, qc);
    store1<TB>(theta, j, qt);
    if constexpr (CB != 0) store1<(CB ? CB : 8)>(comp, j, qc);
  }
}

// Four mantissas as floats: an integer dot product with a one-hot selector sign-extends a
// mantissa and adds it to the bit pattern of M = 1.5 * 2^23 (for |q| < 2^22 integer addition
// on the bits is addition of the values); subtracting M leaves q.  No conversion instruction.
template <int BITS>
__device__ __forceinline__ void load4(const void* base, long long i4, float (&q)[4]) {
  constexpr float kM = 12582912.0f;
  constexpr int kMBits = 0x4B400000;
  if constexpr (BITS == 8) {
    const int w = (int)reinterpret_cast<const unsigned int*>(base)[i4];
#pragma unroll
    for (int j = 0; j < 4; ++j) q[j] = __fadd_rn(__int_as_float(__dp4a(w, 1 << (8 * j), kMBits)), -kM);
  } else {
    const uint2 w = reinterpret_cast<const uint2*>(base)[i4];
    q[0] = __fadd_rn(__int_as_float(__dp2a_lo((int)w.x, 0x0001, kMBits)), -kM);
    q[1] = __fadd_rn(__int_as_float(__dp2a_lo((int)w.x, 0x0100, kMBits)), -kM);
    q[2] = __fadd_rn(__int_as_float(__dp2a_lo((int)w.y, 0x0001, kMBits)), -kM);
    q[3] = __fadd_rn(__int_as_float(__dp2a_lo((int)w.y, 0x0100, kMBits)), -kM);
  }
}

// The same from words already in registers: one word of four 8-bit mantissas, or two words
// of two 16-bit mantissas each.
template <int BITS>
__device__ __forceinline__ void unpack4(unsigned int w0, unsigned int w1, float (&q)[4]) {
  constexpr float kM = 12582912.0f;
  constexpr int kMBits = 0x4B400000;
  if constexpr (BITS == 8) {
#pragma unroll
    for (int j = 0; j < 4; ++j) q[j] = __fadd_rn(__int_as_float(__dp4a((int)w0, 1 << (8 * j), kMBits)), -kM);
  } else {
    q[0] = __fadd_rn(__int_as_float(__dp2a_lo((int)w0, 0x0001, kMBits)), -kM);
    q[1] = __fadd_rn(__int_as_float(__dp2a_lo((int)w0, 0x0100, kMBits)), -kM);
    q[2] = __fadd_rn(__int_as_float(__dp2a_lo((int)w1, 0x0001, kMBits)), -kM);
    q[3] = __fadd_rn(__int_as_float(__dp2a_lo((int)w1, 0x0100, kMBits)), -kM);
  }
}

// A lane's four groups of a piece (groups l, l + 32, l + 64, l + 96) as floats: one 16-byte
// load and a transposition among four lanes for an 8-bit array, four coalesced 8-byte loads
// for a 16-bit one.
template <int BITS>
__device__ __forceinline__ void load_piece(const void* base, long long piece, int lane, float (&q)[4][4]) {
  if constexpr (BITS == 8) {
    const uint4 w = *reinterpret_cast<const uint4*>(static_cast<const char*>(base) + piece * kPiece +
                                                    piece_offset8(lane));
    unsigned int a[4] = {w.x, w.y, w.z, w.w};
    quad_transpose(a, lane);
#pragma unroll
    for (int j = 0; j < 4; ++j) unpack4<8>(a[j], 0u, q[j]);
  } else {
    uint2 w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = reinterpret_cast<const uint2*>(base)[piece * (kPiece / 4) + 32 * j + lane];
#pragma unroll
    for (int j = 0; j < 4; ++j) unpack4<16>(w[j].x, w[j].y, q[j]);
  }
}

template <int BITS>
__device__ __forceinline__ float load1(const void* base, long long i) {
  if constexpr (BITS == 8) return (float)static_cast<const signed char*>(base)[i];
  else return (float)static_cast<const short*>(base)[i];
}

// x = fl32(Q_theta * 2^e + Q_c * 2^(e-s)): the FMA forms Q_theta * 2^s + Q_c exactly and
// rounds once; the scaling by 2^(e-s) that follows is exact (the result is a normal number:
// |e - s| <= 79).
template <int TB, int CB>
__global__ void __launch_bounds__(kThreads) dequantize_kernel(const void* __restrict__ theta,
                                                              const void* __restrict__ comp, float* x, long long n,
                                                              int e, int s) {
  const float pow2s = __int_as_float((127 + s) << 23);
  const float pow2es = __int_as_float((127 + e - s) << 23);
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const bool vec = ((reinterpret_cast<uintptr_t>(x) & 15u) | (reinterpret_cast<uintptr_t>(theta) & (TB / 2 - 1)) |
                    (CB ? (reinterpret_cast<uintptr_t>(comp) & ((CB ? CB : 8) / 2 - 1)) : 0)) == 0u;
  long long done = 0;
  // Main loop, when every array starts on a 16-byte boundary: a warp takes pieces of 512
  // elements, 8-bit arrays are read 16 bytes per lane, the result leaves in four coalesced
  // 16-byte stores per lane.
  constexpr int CBS = CB ? CB : 8;
  const bool pieces = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(theta) |
                        (CB ? reinterpret_cast<uintptr_t>(comp) : 0)) & 15u) == 0u;
  if (pieces) {
    const int lane = threadIdx.x & 31;
    const long long n_pieces = n / kPiece;
    for (long long pc = tid >> 5; pc < n_pieces; pc += stride >> 5) {
      float qt[4][4], qc[4][4] = {};
      load_piece<TB>(theta, pc, lane, qt);
      if constexpr (CB != 0) load_piece<CBS>(comp, pc, lane, qc);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float4 v;
        v.x = __fmul_rn(__fmaf_rn(qt[j][0], pow2s, qc[j][0]), pow2es);
        v.y = __fmul_rn(__fmaf_rn(qt[j][1], pow2s, qc[j][1]), pow2es);
        v.z = __fmul_rn(__fmaf_rn(qt[j][2], pow2s, qc[j][2]), pow2es);
        v.w = __fmul_rn(__fmaf_rn(qt[j][3], pow2s, qc[j][3]), pow2es);
        __stcs(reinterpret_cast<float4*>(x) + pc * (kPiece / 4) + 32 * j + lane, v);
      }
    }
    done = n_pieces * kPiece;
  }
  if (vec) {
    const long long n4 = n >> 2;
#pragma unroll 2
    for (long long i = (done >> 2) + tid; i < n4; i += stride) {
      float qt[4], qc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      load4<TB>(theta, i, qt);
      if constexpr (CB != 0) load4<(CB ? CB : 8)>(comp, i, qc);
      float4 v;
      v.x = __fmul_rn(__fmaf_rn(qt[0], pow2s, qc[0]), pow2es);
      v.y = __fmul_rn(__fmaf_rn(qt[1], pow2s, qc[1]), pow2es);
      v.z = __fmul_rn(__fmaf_rn(qt[2], pow2s, qc[2]), pow2es);
      v.w = __fmul_rn(__fmaf_rn(qt[3], pow2s, qc[3]), pow2es);
      __stcs(reinterpret_cast<float4*>(x) + i, v);
    }
    done = n4 << 2;
  }
  for (long long j = done + tid; j < n; j += stride) {
    float qc = 0.0f;
    if constexpr (CB != 0) qc = load1<(CB ? CB : 8)>(comp, j);
    x[j] = __fmul_rn(__fmaf_rn(load1<TB>(theta, j), pow2s, qc), pow2es);
  }
}

}  // namespace convert
}  // namespace ksgd
