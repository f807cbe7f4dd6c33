// fp32 <-> dynamic fixed-point conversion kernels (Section 1 of arXiv 1810.05486: uniform
// linear quantization with one shared exponent per tensor; Section 5: the exponent comes
// from a scan of the maximum).  Utilities around the update, used when a model enters or
// leaves the fixed-point format, not per step: plain grid-stride kernels, coalesced accesses.  All scalings are by powers of two, so the
// double arithmetic below is exact and the only roundings are the ones the definition names.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace ksgd {
namespace convert {

constexpr int kThreads = 256;

// max |x| over the finite elements, as the bit pattern of a non-negative float (ordered
// like the values), accumulated with atomicMax into *out (cleared by the caller).
__global__ void __launch_bounds__(kThreads) absmax_kernel(const float* __restrict__ x, long long n,
                                                          unsigned int* out) {
  unsigned int m = 0u;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const unsigned int b = __float_as_uint(x[i]) & 0x7fffffffu;
    if (b < 0x7f800000u) m = max(m, b);
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicMax(out, m);
}

__device__ __forceinline__ double clampd(double v, double q) { return fmin(fmax(v, -q), q); }

// One element: Q_theta = clamp(rne(x / 2^e)), Q_c = clamp(rne((x - Q_theta*2^e) / 2^(e-s))).
__device__ __forceinline__ void quantize_one(float xf, int e, int s, double qmax_t, double qmax_c,
                                             bool has_comp, int& qt, int& qc) {
  const double v = (double)xf;
  qc = 0;
  if (v != v) { qt = 0; return; }
  if (isinf(v)) { qt = v > 0 ? (int)qmax_t : -(int)qmax_t; return; }
  const double t = clampd(rint(scalbn(v, -e)), qmax_t);
  qt = (int)t;
  if (has_comp) qc = (int)clampd(rint(scalbn(v - scalbn(t, e), s - e)), qmax_c);
}

template <typename ThetaT, typename CompT, bool HAS_COMP>
__global__ void __launch_bounds__(kThreads) quantize_kernel(const float* __restrict__ x, ThetaT* theta,
                                                            CompT* comp, long long n, int e, int s,
                                                            int theta_bits, int comp_bits) {
  const double qmax_t = (double)((1 << (theta_bits - 1)) - 1);
  const double qmax_c = HAS_COMP ? (double)((1 << (comp_bits - 1)) - 1) : 0.0;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    int qt, qc;
    quantize_one(x[i], e, s, qmax_t, qmax_c, HAS_COMP, qt, qc);
    theta[i] = (ThetaT)qt;
    if (HAS_COMP) comp[i] = (CompT)qc;
  }
}

// x = fl32(Q_theta * 2^e + Q_c * 2^(e-s)): exact in double, one rounding to binary32.
template <typename ThetaT, typename CompT, bool HAS_COMP>
__global__ void __launch_bounds__(kThreads) dequantize_kernel(const ThetaT* __restrict__ theta,
                                                              const CompT* __restrict__ comp, float* x,
                                                              long long n, int e, int s) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    double v = scalbn((double)theta[i], e);
    if (HAS_COMP) v += scalbn((double)comp[i], e - s);
    x[i] = __double2float_rn(v);
  }
}

}  // namespace convert
}  // namespace ksgd
