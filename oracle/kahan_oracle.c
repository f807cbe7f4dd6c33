/*
 * CPU oracle for the lazy update (SGD with Kahan summation, Algorithm 1 of
 * arXiv 1810.05486) in the dynamic fixed-point setting of Section 2 / Fig. 1.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, one-element-at-a-time
 * restatement of the update, used to check the CUDA library and to give a CPU
 * baseline time.  It shares no code with the CUDA library and nothing in the
 * product path may call it.
 *
 * Number system (Section 2, Fig. 1): a tensor is an array of signed integer
 * mantissas with one shared exponent; value = Q * 2^e.  The parameter theta
 * has m-bit mantissas Q_theta at exponent e_theta.  The extra "accumulator"
 * parameter of Algorithm 1 is stored negated, as the compensation c = -acc,
 * with n-bit mantissas Q_c at exponent e_c = e_theta - s, s = n - 1 - k, where
 * k is the number of bits by which the accumulator overlaps the parameter
 * (Section 2: "m + n - 2 - k" magnitude bits in total).  theta + c is the
 * virtually widened parameter.
 *
 * One step for one element (Algorithm 1, statements 1-4, with c = -acc):
 *   stmt 1  acc += eta*g      : the increment is rounded onto the accumulator
 *                               grid,  d = rne(g * eta * 2^-e_c)
 *   stmt 2  theta_u = theta-acc: T = theta + c - d exactly (wide integer on the
 *                               fine grid), theta' = T rounded onto theta's grid
 *   stmt 3  acc += theta_u-theta: c' = T - theta' (what the rounding lost)
 *   stmt 4  theta = theta_u
 *
 * Readings fixed where the paper is silent:
 *   - every rounding is round-to-nearest, ties-to-even (the paper only says
 *     "uniform linear quantization without stochastic computing", Section 1);
 *   - saturation is a symmetric clamp to +-(2^(b-1) - 1);
 *   - the sum acc + eta*g is kept wide until statements 2-3;
 *   - the increment is clamped to +-2^30 accumulator LSBs; NaN gives 0;
 *   - a step reads the mantissas at exponent e_in and writes them at e_out
 *     (|e_out - e_in| <= 8); the increment is rounded on the output grid;
 *   - the next exponent is the tight fit of the step's max |P| (max scan,
 *     Section 5 "Related work" on how dynamic fixed-point picks exponents).
 *
 * Parity pins (tests/test_oracle_pins.py): stall-vs-move (Section 2), the exact
 * accumulation invariant, brute force over all inputs at small bit-widths
 * against exact rational arithmetic, a literal four-statement transcription of
 * Algorithm 1, the m+n-2-k bit-width closed form with the ties-to-even step
 * counts, the plain-SGD reduction (Eq. 1), regrid value preservation, and the
 * exponent-policy property; for the momentum variant (tests/test_oracle_momentum_pins.py):
 * reduction to the plain lazy update at mu = 0, the velocity recursion against exact
 * rationals with explicit binary32 rounding, the geometric fixed point, the exact
 * accumulation invariant and both directions of the velocity-to-compensation grid shift.
 * Accuracy tables of Section 4: parity unpinned
 * (datasets and trained weights are not available).
 * Three rules of the optimizer variants are readings the paper neither states nor
 * contradicts (Section 4 names momentum and ADAM and prints no arithmetic for them;
 * Section 5 only cites max-scan schemes), and nothing outside this file fixes them, so
 * for each of them parity is unpinned against the paper; their tests state the
 * reading's own property:
 *   - ksgd_oracle_next_exponent_velocity: the dead band (the velocity and the ADAM
 *     moments keep their exponent while the largest mantissa lies in (QMAX/4, QMAX]);
 *   - ksgd_oracle_adam_element: a stored second moment <= 0 enters the denominator
 *     as one unit of its grid;
 *   - ksgd_oracle_next_exponent_acc: an empty scan makes the strict accumulator's
 *     grid 8 binades finer.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int64_t P;        /* parameter mantissa before saturation, units of 2^e_out      */
  int64_t Rq;       /* compensation mantissa before saturation, units of 2^ec_out  */
  int64_t T;        /* theta + c - d on the fine grid 2^f, f = min(ec_in, ec_out)  */
  int32_t d;        /* quantized increment, units of 2^ec_out                      */
  int32_t q_theta;  /* stored parameter mantissa  (saturated P)                    */
  int32_t q_comp;   /* stored compensation mantissa (saturated Rq)                 */
  int32_t nonfinite;/* 1 if the gradient was NaN or +-Inf                          */
} ksgd_oracle_elem;

typedef struct {
  uint32_t amax_theta;  /* max |P| over the tensor                                 */
  uint32_t amax_comp;   /* max min(|Rq|, 2^31 - 1) over the tensor                 */
  uint64_t n_sat_theta; /* elements whose parameter mantissa was clamped           */
  uint64_t n_sat_comp;  /* elements whose compensation mantissa was clamped        */
  uint64_t n_nonfinite; /* NaN / Inf gradients                                     */
} ksgd_oracle_stats;

static int64_t pow2_i64(int r) { return (int64_t)1 << r; }

/* floor(a / 2^r) without relying on the shift of a negative number. */
static int64_t floor_div_pow2(int64_t a, int r) {
  int64_t den = pow2_i64(r);
  int64_t q = a / den;            /* truncates toward zero */
  if ((a % den) != 0 && a < 0) q -= 1;
  return q;
}

/* a / 2^r rounded to the nearest integer, ties to the even integer. */
int64_t ksgd_oracle_rne_shift(int64_t a, int32_t r) {
  if (r == 0) return a;
  int64_t q = floor_div_pow2(a, r);
  int64_t rem = a - q * pow2_i64(r);      /* 0 <= rem < 2^r */
  int64_t half = pow2_i64(r - 1);
  if (rem > half) return q + 1;
  if (rem == half && (q % 2 != 0)) return q + 1;
  return q;
}

static int64_t clamp_i64(int64_t x, int64_t lo, int64_t hi) {
  return x < lo ? lo : (x > hi ? hi : x);
}

static int64_t qmax_bits(int bits) { return pow2_i64(bits - 1) - 1; }

/*
 * Statement 1 of Algorithm 1, increment part: eta*g rounded onto the
 * accumulator's output grid.  scale = eta * 2^-ec_out exactly (a power-of-two
 * rescaling of a binary32), x = g*scale is one binary32 multiply, then
 * round-to-nearest-even to an integer, clamped to +-2^30; NaN -> 0.
 */
int32_t ksgd_oracle_increment(float g, float lr, int32_t ec_out) {
  float scale = ldexpf(lr, -ec_out);
  float xv = g * scale;            /* one binary32 multiply (SSE, no contraction) */
  if (isnan(xv)) return 0;
  const float lim = 1073741824.0f; /* 2^30 */
  if (xv >= lim) return (int32_t)1 << 30;
  if (xv <= -lim) return -((int32_t)1 << 30);
  return (int32_t)nearbyintf(xv);  /* default rounding mode: to nearest even */
}

/*
 * One element, any mantissa widths m (parameter) and n (compensation; n = 0 is
 * plain low-precision SGD, Eq. 1) from 2 to 16 bits.  s is the distance between
 * the two grids (ignored, taken as 0, when n = 0).
 */
void ksgd_oracle_element(int32_t q_theta, int32_t q_comp, float g, float lr,
                         int32_t m, int32_t n, int32_t s, int32_t e_in,
                         int32_t e_out, ksgd_oracle_elem* out) {
  if (n == 0) { s = 0; q_comp = 0; }
  int32_t ec_in = e_in - s;
  int32_t ec_out = e_out - s;
  int32_t f = ec_in < ec_out ? ec_in : ec_out;

  int32_t d = ksgd_oracle_increment(g, lr, ec_out);

  /* statements 1-2: theta + c - d, exact, in units of 2^f */
  int64_t T = (int64_t)q_theta * pow2_i64(e_in - f) +
              (int64_t)q_comp * pow2_i64(ec_in - f) -
              (int64_t)d * pow2_i64(ec_out - f);

  /* statement 2/4: round onto the parameter's output grid and saturate */
  int64_t P = ksgd_oracle_rne_shift(T, e_out - f);
  int64_t q_theta_new = clamp_i64(P, -qmax_bits(m), qmax_bits(m));

  /* statement 3: what the parameter could not take stays in the compensation */
  int64_t R = T - q_theta_new * pow2_i64(e_out - f);
  int64_t Rq = 0, q_comp_new = 0;
  if (n != 0) {
    Rq = ksgd_oracle_rne_shift(R, ec_out - f);
    q_comp_new = clamp_i64(Rq, -qmax_bits(n), qmax_bits(n));
  }

  out->P = P;
  out->Rq = Rq;
  out->T = T;
  out->d = d;
  out->q_theta = (int32_t)q_theta_new;
  out->q_comp = (int32_t)q_comp_new;
  out->nonfinite = isfinite(g) ? 0 : 1;
}

static int32_t load_mantissa(const void* p, int64_t i, int bits) {
  return bits <= 8 ? (int32_t)((const int8_t*)p)[i] : (int32_t)((const int16_t*)p)[i];
}

static void store_mantissa(void* p, int64_t i, int bits, int32_t v) {
  if (bits <= 8) ((int8_t*)p)[i] = (int8_t)v; else ((int16_t*)p)[i] = (int16_t)v;
}

/*
 * One step over one tensor, in place.  Mantissas of up to 8 bits live in int8
 * arrays, wider ones in int16 arrays.  comp may be NULL iff comp_bits == 0.
 * n_threads > 1 splits the elements statically over OpenMP threads; max and
 * integer sums are exact, so the result does not depend on n_threads.
 * Returns 0, or -1 on an argument the format does not allow.
 */
int ksgd_oracle_step_tensor(void* theta, void* comp, const float* grad,
                            int64_t numel, int32_t theta_bits, int32_t comp_bits,
                            int32_t overlap_k, int32_t e_in, int32_t e_out,
                            float lr, ksgd_oracle_stats* stats, int32_t n_threads) {
  if (!theta || !grad || !stats || numel <= 0) return -1;
  if (theta_bits < 2 || theta_bits > 16) return -1;
  if (comp_bits != 0 && (comp_bits < 2 || comp_bits > 16)) return -1;
  if (comp_bits != 0 && (!comp || overlap_k < 0 || overlap_k > comp_bits - 1)) return -1;
  if (e_out - e_in > 8 || e_in - e_out > 8) return -1;
  int32_t s = comp_bits == 0 ? 0 : comp_bits - 1 - overlap_k;

  uint32_t amax_theta = 0, amax_comp = 0;
  uint64_t n_sat_theta = 0, n_sat_comp = 0, n_nonfinite = 0;
  if (n_threads < 1) n_threads = 1;

#pragma omp parallel for schedule(static) num_threads(n_threads) \
    reduction(max : amax_theta, amax_comp) reduction(+ : n_sat_theta, n_sat_comp, n_nonfinite)
  for (int64_t i = 0; i < numel; ++i) {
    ksgd_oracle_elem r;
    int32_t qt = load_mantissa(theta, i, theta_bits);
    int32_t qc = comp_bits ? load_mantissa(comp, i, comp_bits) : 0;
    ksgd_oracle_element(qt, qc, grad[i], lr, theta_bits, comp_bits, s, e_in, e_out, &r);
    store_mantissa(theta, i, theta_bits, r.q_theta);
    if (comp_bits) store_mantissa(comp, i, comp_bits, r.q_comp);

    int64_t aP = r.P < 0 ? -r.P : r.P;
    int64_t aR = r.Rq < 0 ? -r.Rq : r.Rq;
    if (aR > 2147483647LL) aR = 2147483647LL;
    if ((uint32_t)aP > amax_theta) amax_theta = (uint32_t)aP;
    if ((uint32_t)aR > amax_comp) amax_comp = (uint32_t)aR;
    n_sat_theta += (r.P != r.q_theta);
    n_sat_comp += (comp_bits != 0 && r.Rq != r.q_comp);
    n_nonfinite += (uint64_t)r.nonfinite;
  }
  stats->amax_theta = amax_theta;
  stats->amax_comp = amax_comp;
  stats->n_sat_theta = n_sat_theta;
  stats->n_sat_comp = n_sat_comp;
  stats->n_nonfinite = n_nonfinite;
  return 0;
}

/*
 * Exponent for the next step from the max scan of this one (dynamic
 * fixed-point: the shared exponent follows the tensor's maximum).  amax_theta
 * is max |P| in units of 2^e_out.  Tight fit: the largest mantissa of the
 * rescaled tensor lands in (QMAX/2, QMAX].  The move is limited to 8 binades
 * per step and the exponent to [-64, 64].  amax_mode == 0 keeps e_out.
 */
int32_t ksgd_oracle_next_exponent(uint32_t amax_theta, int32_t theta_bits,
                                  int32_t e_out, int32_t amax_mode) {
  if (!amax_mode || amax_theta == 0) return e_out;
  int64_t A = (int64_t)amax_theta;
  int64_t Q = qmax_bits(theta_bits);
  int32_t delta = 0;
  if (A > Q) {
    int32_t j = 1;
    while (A > Q * pow2_i64(j)) ++j;
    delta = j;
  } else {
    int32_t r = 0;
    while (A * pow2_i64(r + 1) <= Q) ++r;
    delta = -r;
  }
  if (delta > 8) delta = 8;
  if (delta < -8) delta = -8;
  int32_t e_next = e_out + delta;
  if (e_next > 64) e_next = 64;
  if (e_next < -64) e_next = -64;
  return e_next;
}

/* ------------------------------------------------------------------------------------
 * Momentum optimizer with the lazy update (Section 4: "the lazy update described in
 * Algorithm 1 was implemented in the optimizers"; momentum mu = 0.9 in INT8, INT16 for
 * AlexNet).  The paper gives no formulas; the reading taken is the classical form
 *     v <- mu*v + eta*g ,   theta <- theta - v
 * with v a third dynamic fixed-point tensor (b-bit mantissas Q_v, own exponent e_v that
 * follows its own max scan) and Algorithm 1 applied with v in the place of eta*g:
 *   mu_s = fl32(mu * 2^(ev_in - ev_out))                 exact power-of-two rescaling
 *   bq   = fl32(g * fl32(eta * 2^-ev_out))               one binary32 multiply
 *   y    = fma32(mu_s, Q_v, bq)                           one rounding
 *   V    = clamp(rne(y), +-2^30), NaN -> 0 ;  Q_v' = clamp(V, +-(2^(b-1)-1))
 *   d    = Q_v' * 2^k (clamped to +-2^30) if k >= 0 else rne(Q_v' / 2^-k),
 *          k = ev_out - ec_out: the stored velocity expressed on the compensation grid
 *   then statements 1-4 of Algorithm 1 with this d.
 */
typedef struct {
  ksgd_oracle_elem upd;  /* the parameter update (d = increment taken from the velocity)   */
  int64_t V;             /* velocity mantissa before saturation, units of 2^ev_out          */
  int32_t q_mom;         /* stored velocity mantissa                                        */
} ksgd_oracle_mom_elem;

static int32_t velocity_mantissa(int32_t q_mom, float g, float lr, float mu, int32_t ev_in,
                                 int32_t ev_out) {
  float mu_s = ldexpf(mu, ev_in - ev_out);
  float scale_v = ldexpf(lr, -ev_out);
  float bq = g * scale_v;
  float y = fmaf(mu_s, (float)q_mom, bq);
  if (isnan(y)) return 0;
  const float lim = 1073741824.0f;
  if (y >= lim) return (int32_t)1 << 30;
  if (y <= -lim) return -((int32_t)1 << 30);
  return (int32_t)nearbyintf(y);
}

void ksgd_oracle_momentum_element(int32_t q_theta, int32_t q_comp, int32_t q_mom, float g, float lr,
                                  float mu, int32_t m, int32_t n, int32_t s, int32_t b,
                                  int32_t e_in, int32_t e_out, int32_t ev_in, int32_t ev_out,
                                  ksgd_oracle_mom_elem* out) {
  if (n == 0) { s = 0; q_comp = 0; }
  int64_t V = velocity_mantissa(q_mom, g, lr, mu, ev_in, ev_out);
  int64_t q_mom_new = clamp_i64(V, -qmax_bits(b), qmax_bits(b));

  int32_t ec_in = e_in - s, ec_out = e_out - s;
  int32_t f = ec_in < ec_out ? ec_in : ec_out;
  int32_t k = ev_out - ec_out;
  int64_t d;
  if (k >= 0) {
    /* |Q_v'| < 2^15, so any k >= 16 with Q_v' != 0 is beyond the clamp */
    d = k > 40 ? (q_mom_new > 0 ? pow2_i64(30) : (q_mom_new < 0 ? -pow2_i64(30) : 0))
               : clamp_i64(q_mom_new * pow2_i64(k), -pow2_i64(30), pow2_i64(30));
  } else {
    d = -k > 40 ? 0 : ksgd_oracle_rne_shift(q_mom_new, -k);
  }

  int64_t T = (int64_t)q_theta * pow2_i64(e_in - f) + (int64_t)q_comp * pow2_i64(ec_in - f) -
              d * pow2_i64(ec_out - f);
  int64_t P = ksgd_oracle_rne_shift(T, e_out - f);
  int64_t q_theta_new = clamp_i64(P, -qmax_bits(m), qmax_bits(m));
  int64_t R = T - q_theta_new * pow2_i64(e_out - f);
  int64_t Rq = 0, q_comp_new = 0;
  if (n != 0) {
    Rq = ksgd_oracle_rne_shift(R, ec_out - f);
    q_comp_new = clamp_i64(Rq, -qmax_bits(n), qmax_bits(n));
  }
  out->upd.P = P;
  out->upd.Rq = Rq;
  out->upd.T = T;
  out->upd.d = (int32_t)d;
  out->upd.q_theta = (int32_t)q_theta_new;
  out->upd.q_comp = (int32_t)q_comp_new;
  out->upd.nonfinite = isfinite(g) ? 0 : 1;
  out->V = V;
  out->q_mom = (int32_t)q_mom_new;
}

typedef struct {
  ksgd_oracle_stats upd;
  uint32_t amax_mom;    /* max |V| over the tensor                     */
  uint64_t n_sat_mom;   /* elements whose velocity mantissa was clamped */
} ksgd_oracle_mom_stats;

int ksgd_oracle_momentum_step_tensor(void* theta, void* comp, void* mom, const float* grad,
                                     int64_t numel, int32_t theta_bits, int32_t comp_bits,
                                     int32_t overlap_k, int32_t mom_bits, int32_t e_in,
                                     int32_t e_out, int32_t ev_in, int32_t ev_out, float lr, float mu,
                                     ksgd_oracle_mom_stats* stats, int32_t n_threads) {
  if (!theta || !mom || !grad || !stats || numel <= 0) return -1;
  if (theta_bits < 2 || theta_bits > 16 || mom_bits < 2 || mom_bits > 16) return -1;
  if (comp_bits != 0 && (comp_bits < 2 || comp_bits > 16)) return -1;
  if (comp_bits != 0 && (!comp || overlap_k < 0 || overlap_k > comp_bits - 1)) return -1;
  if (e_out - e_in > 8 || e_in - e_out > 8 || ev_out - ev_in > 8 || ev_in - ev_out > 8) return -1;
  int32_t s = comp_bits == 0 ? 0 : comp_bits - 1 - overlap_k;
  uint32_t amax_theta = 0, amax_comp = 0, amax_mom = 0;
  uint64_t n_sat_theta = 0, n_sat_comp = 0, n_nonfinite = 0, n_sat_mom = 0;
  if (n_threads < 1) n_threads = 1;
#pragma omp parallel for schedule(static) num_threads(n_threads) \
    reduction(max : amax_theta, amax_comp, amax_mom) \
    reduction(+ : n_sat_theta, n_sat_comp, n_nonfinite, n_sat_mom)
  for (int64_t i = 0; i < numel; ++i) {
    ksgd_oracle_mom_elem r;
    int32_t qt = load_mantissa(theta, i, theta_bits);
    int32_t qc = comp_bits ? load_mantissa(comp, i, comp_bits) : 0;
    int32_t qv = load_mantissa(mom, i, mom_bits);
    ksgd_oracle_momentum_element(qt, qc, qv, grad[i], lr, mu, theta_bits, comp_bits, s, mom_bits,
                                 e_in, e_out, ev_in, ev_out, &r);
    store_mantissa(theta, i, theta_bits, r.upd.q_theta);
    if (comp_bits) store_mantissa(comp, i, comp_bits, r.upd.q_comp);
    store_mantissa(mom, i, mom_bits, r.q_mom);
    int64_t aP = r.upd.P < 0 ? -r.upd.P : r.upd.P;
    int64_t aR = r.upd.Rq < 0 ? -r.upd.Rq : r.upd.Rq;
    int64_t aV = r.V < 0 ? -r.V : r.V;
    if (aR > 2147483647LL) aR = 2147483647LL;
    if ((uint32_t)aP > amax_theta) amax_theta = (uint32_t)aP;
    if ((uint32_t)aR > amax_comp) amax_comp = (uint32_t)aR;
    if ((uint32_t)aV > amax_mom) amax_mom = (uint32_t)aV;
    n_sat_theta += (r.upd.P != r.upd.q_theta);
    n_sat_comp += (comp_bits != 0 && r.upd.Rq != r.upd.q_comp);
    n_sat_mom += (r.V != r.q_mom);
    n_nonfinite += (uint64_t)r.upd.nonfinite;
  }
  stats->upd.amax_theta = amax_theta;
  stats->upd.amax_comp = amax_comp;
  stats->upd.n_sat_theta = n_sat_theta;
  stats->upd.n_sat_comp = n_sat_comp;
  stats->upd.n_nonfinite = n_nonfinite;
  stats->amax_mom = amax_mom;
  stats->n_sat_mom = n_sat_mom;
  return 0;
}

/*
 * Exponent of the velocity for the next step.  The velocity's maximum moves with every
 * gradient, so the tight fit used for theta would change the exponent back and forth from
 * step to step; the velocity therefore keeps its exponent while its largest mantissa stays
 * in (QMAX/4, QMAX]: coarser at once when amax > QMAX (as for theta), finer only when
 * 4*amax <= QMAX, and then by the tight fit.  Same limits (8 binades per step, [-64, 64]).
 */
int32_t ksgd_oracle_next_exponent_velocity(uint32_t amax_mom, int32_t mom_bits, int32_t ev_out,
                                           int32_t amax_mode) {
  if (!amax_mode || amax_mom == 0) return ev_out;
  int64_t A = (int64_t)amax_mom;
  int64_t Q = qmax_bits(mom_bits);
  if (A <= Q && 4 * A > Q) return ev_out;
  return ksgd_oracle_next_exponent(amax_mom, mom_bits, ev_out, amax_mode);
}

/* ------------------------------------------------------------------------------------
 * ADAM with the lazy update (Section 4: ADAM, beta1 = 0.9, beta2 = 0.999, needs INT16 for
 * its moments "because of beta2").  The paper gives no formulas; the reading taken is the
 * usual ADAM with the bias correction folded into the step size by the caller
 * (lr_t = eta * sqrt(1 - beta2^t) / (1 - beta1^t)):
 *     m <- beta1*m + (1-beta1)*g ,  v <- beta2*v + (1-beta2)*g^2 ,
 *     theta <- theta - lr_t * m / (sqrt(v) + eps)      (the subtraction through Algorithm 1)
 * with m and v two more dynamic fixed-point tensors (16-bit mantissas, own exponents).
 * Every floating-point operation is one correctly rounded binary32 operation:
 *   c1 = fl(1 - beta1), c2 = fl(1 - beta2)
 *   ym = fma(fl(beta1 * 2^(em_in-em_out)), Q_m, fl(g * fl(c1 * 2^-em_out)))    M = rne(ym)
 *   yv = fma(fl(beta2 * 2^(ev_in-ev_out)), Q_v, fl(fl(g*g) * fl(c2 * 2^-ev_out)))  V = rne(yv)
 *   (both clamped to +-2^30, NaN -> 0, then to +-(2^15 - 1) for storage)
 *   mr = Q_m' * 2^em_out, vr = max(Q_v', 1) * 2^ev_out  exact
 *   q  = fl(mr / fl(sqrt(vr) + eps))
 *   d  = clamp(rne(fl(q * fl(lr_t * 2^-ec_out))), +-2^30), NaN -> 0
 *   then statements 1-4 of Algorithm 1 with this d.
 * The floor of one unit on the second-moment mantissa: a second moment below the resolution
 * of its 16-bit grid would otherwise leave eps alone in the denominator and turn any
 * non-zero first moment into a step of m/eps (1e8 m with the usual eps); a value that the
 * grid cannot tell from zero is taken as one unit instead, which bounds the step by
 * |m| / sqrt(2^ev_out).
 */
typedef struct {
  ksgd_oracle_elem upd;
  int64_t M, V;          /* moment mantissas before saturation */
  int32_t q_m, q_v;      /* stored moment mantissas            */
} ksgd_oracle_adam_elem;

static int32_t rne_clamped(float y) {
  if (isnan(y)) return 0;
  const float lim = 1073741824.0f;
  if (y >= lim) return (int32_t)1 << 30;
  if (y <= -lim) return -((int32_t)1 << 30);
  return (int32_t)nearbyintf(y);
}

void ksgd_oracle_adam_element(int32_t q_theta, int32_t q_comp, int32_t q_m, int32_t q_v, float g, float lr,
                              float beta1, float beta2, float eps, int32_t m, int32_t n, int32_t s,
                              int32_t e_in, int32_t e_out, int32_t em_in, int32_t em_out,
                              int32_t ev_in, int32_t ev_out, ksgd_oracle_adam_elem* out) {
  if (n == 0) { s = 0; q_comp = 0; }
  float c1 = 1.0f - beta1, c2 = 1.0f - beta2;
  float ym = fmaf(ldexpf(beta1, em_in - em_out), (float)q_m, g * ldexpf(c1, -em_out));
  float g2 = g * g;
  float yv = fmaf(ldexpf(beta2, ev_in - ev_out), (float)q_v, g2 * ldexpf(c2, -ev_out));
  int64_t M = rne_clamped(ym), V = rne_clamped(yv);
  int64_t qm_new = clamp_i64(M, -32767, 32767), qv_new = clamp_i64(V, -32767, 32767);

  int32_t ec_in = e_in - s, ec_out = e_out - s;
  int32_t f = ec_in < ec_out ? ec_in : ec_out;
  float mr = ldexpf((float)qm_new, em_out);
  float vr = ldexpf((float)(qv_new > 1 ? qv_new : 1), ev_out);
  float root = sqrtf(vr);
  float den = root + eps;
  float q = mr / den;
  float x = q * ldexpf(lr, -ec_out);
  int64_t d = rne_clamped(x);

  int64_t T = (int64_t)q_theta * pow2_i64(e_in - f) + (int64_t)q_comp * pow2_i64(ec_in - f) -
              d * pow2_i64(ec_out - f);
  int64_t P = ksgd_oracle_rne_shift(T, e_out - f);
  int64_t q_theta_new = clamp_i64(P, -qmax_bits(m), qmax_bits(m));
  int64_t R = T - q_theta_new * pow2_i64(e_out - f);
  int64_t Rq = 0, q_comp_new = 0;
  if (n != 0) {
    Rq = ksgd_oracle_rne_shift(R, ec_out - f);
    q_comp_new = clamp_i64(Rq, -qmax_bits(n), qmax_bits(n));
  }
  out->upd.P = P; out->upd.Rq = Rq; out->upd.T = T; out->upd.d = (int32_t)d;
  out->upd.q_theta = (int32_t)q_theta_new; out->upd.q_comp = (int32_t)q_comp_new;
  out->upd.nonfinite = isfinite(g) ? 0 : 1;
  out->M = M; out->V = V; out->q_m = (int32_t)qm_new; out->q_v = (int32_t)qv_new;
}

typedef struct {
  ksgd_oracle_stats upd;
  uint32_t amax_m, amax_v;
  uint64_t n_sat_m, n_sat_v;
} ksgd_oracle_adam_stats;

int ksgd_oracle_adam_step_tensor(void* theta, void* comp, int16_t* mom1, int16_t* mom2, const float* grad,
                                 int64_t numel, int32_t theta_bits, int32_t comp_bits, int32_t overlap_k,
                                 int32_t e_in, int32_t e_out, int32_t em_in, int32_t em_out, int32_t ev_in,
                                 int32_t ev_out, float lr, float beta1, float beta2, float eps,
                                 ksgd_oracle_adam_stats* stats, int32_t n_threads) {
  if (!theta || !mom1 || !mom2 || !grad || !stats || numel <= 0) return -1;
  if (theta_bits < 2 || theta_bits > 16) return -1;
  if (comp_bits != 0 && (comp_bits < 2 || comp_bits > 16)) return -1;
  if (comp_bits != 0 && (!comp || overlap_k < 0 || overlap_k > comp_bits - 1)) return -1;
  int32_t s = comp_bits == 0 ? 0 : comp_bits - 1 - overlap_k;
  uint32_t amax_theta = 0, amax_comp = 0, amax_m = 0, amax_v = 0;
  uint64_t n_sat_theta = 0, n_sat_comp = 0, n_nonfinite = 0, n_sat_m = 0, n_sat_v = 0;
  if (n_threads < 1) n_threads = 1;
#pragma omp parallel for schedule(static) num_threads(n_threads) \
    reduction(max : amax_theta, amax_comp, amax_m, amax_v) \
    reduction(+ : n_sat_theta, n_sat_comp, n_nonfinite, n_sat_m, n_sat_v)
  for (int64_t i = 0; i < numel; ++i) {
    ksgd_oracle_adam_elem r;
    int32_t qt = load_mantissa(theta, i, theta_bits);
    int32_t qc = comp_bits ? load_mantissa(comp, i, comp_bits) : 0;
    ksgd_oracle_adam_element(qt, qc, mom1[i], mom2[i], grad[i], lr, beta1, beta2, eps, theta_bits,
                             comp_bits, s, e_in, e_out, em_in, em_out, ev_in, ev_out, &r);
    store_mantissa(theta, i, theta_bits, r.upd.q_theta);
    if (comp_bits) store_mantissa(comp, i, comp_bits, r.upd.q_comp);
    mom1[i] = (int16_t)r.q_m;
    mom2[i] = (int16_t)r.q_v;
    int64_t aP = r.upd.P < 0 ? -r.upd.P : r.upd.P, aR = r.upd.Rq < 0 ? -r.upd.Rq : r.upd.Rq;
    int64_t aM = r.M < 0 ? -r.M : r.M, aV = r.V < 0 ? -r.V : r.V;
    if (aR > 2147483647LL) aR = 2147483647LL;
    if ((uint32_t)aP > amax_theta) amax_theta = (uint32_t)aP;
    if ((uint32_t)aR > amax_comp) amax_comp = (uint32_t)aR;
    if ((uint32_t)aM > amax_m) amax_m = (uint32_t)aM;
    if ((uint32_t)aV > amax_v) amax_v = (uint32_t)aV;
    n_sat_theta += (r.upd.P != r.upd.q_theta);
    n_sat_comp += (comp_bits != 0 && r.upd.Rq != r.upd.q_comp);
    n_sat_m += (r.M != r.q_m);
    n_sat_v += (r.V != r.q_v);
    n_nonfinite += (uint64_t)r.upd.nonfinite;
  }
  stats->upd.amax_theta = amax_theta; stats->upd.amax_comp = amax_comp;
  stats->upd.n_sat_theta = n_sat_theta; stats->upd.n_sat_comp = n_sat_comp;
  stats->upd.n_nonfinite = n_nonfinite;
  stats->amax_m = amax_m; stats->amax_v = amax_v; stats->n_sat_m = n_sat_m; stats->n_sat_v = n_sat_v;
  return 0;
}

/* ------------------------------------------------------------------------------------
 * Strict Algorithm 1: every statement rounds into the stored format, and the accumulator
 * is a dynamic fixed-point tensor of its own -- n-bit mantissas with an exponent that
 * follows the accumulator's maximum, not theta's exponent (Section 2: acc is an n-bit
 * tensor below theta, Figure 1; Section 5: exponents from a scan of the maximum).  The
 * overlap k is then not a parameter but a result, k = n - 1 - (e - e_acc).
 * As everywhere here the tensor stored is c = -acc.  With f the smallest of the four
 * exponents (theta's and c's, each read at *_in and written at *_out):
 *   d   = clamp(rne(fl(g * fl(lr * 2^-ec_out))), +-2^30)              the increment on c's grid
 *   C1  = rne((Q_c * 2^(ec_in-f) - d * 2^(ec_out-f)) / 2^(ec_out-f))  statement 1: acc += eta g
 *   Qc1 = clamp(C1, +-QMAX_n)                                         ... stored in n bits
 *   T   = Q_theta * 2^(e_in-f) + Qc1 * 2^(ec_out-f)                   statement 2: theta - acc
 *   P   = rne(T / 2^(e_out-f)),  Q_theta' = clamp(P, +-QMAX_m)        ... stored in m bits
 *   C2  = rne((T - Q_theta' * 2^(e_out-f)) / 2^(ec_out-f))            statement 3: acc += theta_u - theta
 *   Q_c' = clamp(C2, +-QMAX_n)                                        ... stored in n bits
 * Scans: max |P| for theta, max(|C1|, |C2|) for c (so that an increment too large for the
 * accumulator raises its exponent), each capped at 2^31 - 1.
 * Exponents must satisfy  -8 <= e - ec <= 36  at both ends of the step (the sums then fit
 * in 64 bits); the policy keeps them there.
 */
typedef struct {
  int64_t C1, T, P, C2;
  int32_t d, q_comp_mid, q_theta, q_comp, nonfinite;
} ksgd_oracle_strict_elem;

static int64_t rne_div_pow2(int64_t a, int r) { return r == 0 ? a : ksgd_oracle_rne_shift(a, r); }

void ksgd_oracle_strict_element(int32_t q_theta, int32_t q_comp, float g, float lr, int32_t m, int32_t n,
                                int32_t e_in, int32_t e_out, int32_t ec_in, int32_t ec_out,
                                ksgd_oracle_strict_elem* out) {
  int32_t f = e_in;
  if (e_out < f) f = e_out;
  if (ec_in < f) f = ec_in;
  if (ec_out < f) f = ec_out;
  int64_t d = ksgd_oracle_increment(g, lr, ec_out);
  int64_t C1 = rne_div_pow2((int64_t)q_comp * pow2_i64(ec_in - f) - d * pow2_i64(ec_out - f), ec_out - f);
  int64_t Qc1 = clamp_i64(C1, -qmax_bits(n), qmax_bits(n));
  int64_t T = (int64_t)q_theta * pow2_i64(e_in - f) + Qc1 * pow2_i64(ec_out - f);
  int64_t P = rne_div_pow2(T, e_out - f);
  int64_t Qt = clamp_i64(P, -qmax_bits(m), qmax_bits(m));
  int64_t C2 = rne_div_pow2(T - Qt * pow2_i64(e_out - f), ec_out - f);
  int64_t Qc2 = clamp_i64(C2, -qmax_bits(n), qmax_bits(n));
  out->C1 = C1; out->T = T; out->P = P; out->C2 = C2; out->d = (int32_t)d;
  out->q_comp_mid = (int32_t)Qc1; out->q_theta = (int32_t)Qt; out->q_comp = (int32_t)Qc2;
  out->nonfinite = isfinite(g) ? 0 : 1;
}

static int strict_window_ok(int32_t e, int32_t ec) { return e - ec >= -8 && e - ec <= 36; }

int ksgd_oracle_strict_step_tensor(void* theta, void* comp, const float* grad, int64_t numel,
                                   int32_t theta_bits, int32_t comp_bits, int32_t e_in, int32_t e_out,
                                   int32_t ec_in, int32_t ec_out, float lr, ksgd_oracle_stats* stats,
                                   int32_t n_threads) {
  if (!theta || !comp || !grad || !stats || numel <= 0) return -1;
  if (theta_bits < 2 || theta_bits > 16 || comp_bits < 2 || comp_bits > 16) return -1;
  if (!strict_window_ok(e_in, ec_in) || !strict_window_ok(e_out, ec_out)) return -1;
  /* outside this the 64-bit sums of the element could overflow; the exponent rule below
   * never asks for more (its own fit moves at most 8, theta's window at most 8 more) */
  if (ec_out - ec_in > 16 || ec_in - ec_out > 16 || e_out - e_in > 8 || e_in - e_out > 8) return -1;
  uint32_t amax_theta = 0, amax_comp = 0;
  uint64_t n_sat_theta = 0, n_sat_comp = 0, n_nonfinite = 0;
  if (n_threads < 1) n_threads = 1;
#pragma omp parallel for schedule(static) num_threads(n_threads) \
    reduction(max : amax_theta, amax_comp) reduction(+ : n_sat_theta, n_sat_comp, n_nonfinite)
  for (int64_t i = 0; i < numel; ++i) {
    ksgd_oracle_strict_elem r;
    ksgd_oracle_strict_element(load_mantissa(theta, i, theta_bits), load_mantissa(comp, i, comp_bits), grad[i],
                               lr, theta_bits, comp_bits, e_in, e_out, ec_in, ec_out, &r);
    store_mantissa(theta, i, theta_bits, r.q_theta);
    store_mantissa(comp, i, comp_bits, r.q_comp);
    int64_t aP = r.P < 0 ? -r.P : r.P, a1 = r.C1 < 0 ? -r.C1 : r.C1, a2 = r.C2 < 0 ? -r.C2 : r.C2;
    int64_t aC = a1 > a2 ? a1 : a2;
    if (aP > 2147483647LL) aP = 2147483647LL;
    if (aC > 2147483647LL) aC = 2147483647LL;
    if ((uint32_t)aP > amax_theta) amax_theta = (uint32_t)aP;
    if ((uint32_t)aC > amax_comp) amax_comp = (uint32_t)aC;
    n_sat_theta += (r.P != r.q_theta);
    n_sat_comp += (uint64_t)(r.C1 != r.q_comp_mid) + (uint64_t)(r.C2 != r.q_comp);
    n_nonfinite += (uint64_t)r.nonfinite;
  }
  stats->amax_theta = amax_theta; stats->amax_comp = amax_comp;
  stats->n_sat_theta = n_sat_theta; stats->n_sat_comp = n_sat_comp; stats->n_nonfinite = n_nonfinite;
  return 0;
}

/* The accumulator's next exponent: the tight fit of its own maximum (same rule as for
 * theta), then moved into the window [e_next - 36, e_next + 8] around theta's next exponent
 * and into [-64, 64].  A scan of zero says that every increment rounded to nothing on the
 * present grid (or that there was none): the grid then becomes 8 binades finer, so that an
 * empty accumulator finds the scale of the increments instead of swallowing them for ever. */
int32_t ksgd_oracle_next_exponent_acc(uint32_t amax_comp, int32_t comp_bits, int32_t ec_out, int32_t e_next,
                                      int32_t amax_mode) {
  int32_t ec = ksgd_oracle_next_exponent(amax_comp, comp_bits, ec_out, amax_mode);
  if (amax_mode && amax_comp == 0) ec = ec_out - 8;
  if (ec < e_next - 36) ec = e_next - 36;
  if (ec > e_next + 8) ec = e_next + 8;
  if (ec > 64) ec = 64;
  if (ec < -64) ec = -64;
  return ec;
}

/* ------------------------------------------------------------------------------------
 * fp32 <-> dynamic fixed-point (Section 1: uniform linear quantization with one shared
 * exponent per tensor; Section 5: the exponent comes from a scan of the maximum).
 *
 * Exponent: the smallest e in [-64, 64] with max|x| <= QMAX_m * 2^e over the finite x
 * (e = 0 for an all-zero or all-non-finite tensor).
 * Import: Q_theta = clamp(rne(x / 2^e), +-QMAX_m); with a compensation tensor the part
 * theta cannot hold goes there, Q_c = clamp(rne((x - Q_theta*2^e) / 2^(e-s)), +-QMAX_n),
 * so that theta + c carries m+n-2-k bits of x.  NaN -> 0, +-Inf -> +-QMAX_m (c = 0).
 * Export: x = fl32(Q_theta * 2^e + Q_c * 2^(e-s)), computed exactly and rounded once.
 * All scalings are by powers of two, so double arithmetic is exact here.
 */
int32_t ksgd_oracle_fit_exponent(const float* x, int64_t numel, int32_t bits) {
  double amax = 0.0;
  for (int64_t i = 0; i < numel; ++i)
    if (isfinite(x[i]) && fabs((double)x[i]) > amax) amax = fabs((double)x[i]);
  if (amax == 0.0) return 0;
  double Q = (double)qmax_bits(bits);
  int32_t e = -64;
  while (e < 64 && amax > ldexp(Q, e)) ++e;
  return e;
}

void ksgd_oracle_quantize(const float* x, void* theta, void* comp, int64_t numel, int32_t theta_bits,
                          int32_t comp_bits, int32_t overlap_k, int32_t e) {
  int32_t s = comp_bits ? comp_bits - 1 - overlap_k : 0;
  double Qt = (double)qmax_bits(theta_bits);
  for (int64_t i = 0; i < numel; ++i) {
    double v = (double)x[i];
    int64_t qt, qc = 0;
    if (isnan(v)) {
      qt = 0;
    } else if (isinf(v)) {
      qt = v > 0 ? (int64_t)Qt : -(int64_t)Qt;
    } else {
      double t = nearbyint(ldexp(v, -e));          /* exact scaling, ties to even */
      if (t > Qt) t = Qt;
      if (t < -Qt) t = -Qt;
      qt = (int64_t)t;
      if (comp_bits) {
        double Qc = (double)qmax_bits(comp_bits);
        double r = nearbyint(ldexp(v - ldexp((double)qt, e), -(e - s)));
        if (r > Qc) r = Qc;
        if (r < -Qc) r = -Qc;
        qc = (int64_t)r;
      }
    }
    store_mantissa(theta, i, theta_bits, (int32_t)qt);
    if (comp_bits) store_mantissa(comp, i, comp_bits, (int32_t)qc);
  }
}

void ksgd_oracle_dequantize(const void* theta, const void* comp, float* x, int64_t numel,
                            int32_t theta_bits, int32_t comp_bits, int32_t overlap_k, int32_t e) {
  int32_t s = comp_bits ? comp_bits - 1 - overlap_k : 0;
  for (int64_t i = 0; i < numel; ++i) {
    double v = ldexp((double)load_mantissa(theta, i, theta_bits), e);
    if (comp_bits) v += ldexp((double)load_mantissa(comp, i, comp_bits), e - s);
    x[i] = (float)v;                                /* one rounding to binary32 */
  }
}

int32_t ksgd_oracle_max_threads(void) {
#ifdef _OPENMP
  return (int32_t)omp_get_max_threads();
#else
  return 1;
#endif
}
