// CPU oracle for the INT8 State Space Duality (SSD) layer of SSDi8.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
// the layer computes, written from the paper.  It shares no code with the CUDA
// library and must never be linked, imported or called by it; only the tests,
// the smoke check and the CPU-baseline leg of the benchmark use it.
//
// Levels
//   L0  naive recurrence of the discretised SSM (Eq. "h' = Ah + Bx, y = Ch"
//       of Section 3.2 with the zero-order-hold step dt):
//         h_t = exp(dt_t A) h_{t-1} + dt_t B_t x_t^T ,  y_t = C_t h_t + D x_t
//   L1  chunked (dual) form of Algorithm 2 in fp64, no internal quantisation
//   L2  SSDi8: Algorithm 2 with the INT8 path of Section 4.2 (Eq. 1, 3, 4); inter-chunk states
//       either fp32 or, as in the paper, persistent INT8 with a fixed-point decay (Eq. 7)
//   L3  single-token recurrent step (L0 restated per token, state in place)
//
// Precision.  Everything is fp64 with exact integer products, except the
// values that DECIDE an integer code (a re-quantisation).  Those are formed in
// IEEE binary32 by the operation sequence written next to each of them
// (fmul/fadd/fdiv/fmaf, round-to-nearest-even, no contraction, no fast math),
// so that the int8 tensors and int32 accumulators are well-defined bit for bit.
// The exponential inside those values is exp32() below, a fixed sequence of
// binary32 operations, pinned against libm's exp by the tests.
//
// Two forms of the internal re-quantisations.  The "plain" functions (orc_*_plain,
// orc_ssdi8_fwd_plain) are the definitions written out: fp64, libm exp, one exponential per
// element, no blocking of any kind; they are what a reader checks against Algorithm 2 and
// Eq. 1, 3, 4 by eye.  The other stage functions (orc_chunk_state, orc_state_passing,
// orc_chunk_scan) restate the operation-by-operation binary32 arithmetic that the library's
// header fixes for every value that decides an integer code, so that a second implementation
// can be compared bit for bit; their factorisation of the decay into 16-token sub-blocks is
// part of that interface, not of the method.  The tests tie the two together: every code of the
// binary32 form equals the plain form's code or is its neighbour with the fp64 value next to
// the rounding boundary between them.
//
// Pins (tests/test_oracle_*.py): L1 == L0 for every chunk size (duality and
// chunk invariance), closed form for constant inputs, A -> 0 reduces to masked
// linear attention (numpy matmul), dt = 0 gives y = D x, integer GEMM stages
// against numpy int64 matmul, quantiser error bounds and idempotence, exp32
// against libm, L2 within its quantisation error bound of L1, L3 == L0.
//
// Every function here has such a pin; none is left unpinned.  The paper prints
// no worked example (none of its figures survive in the text), so no pin is a
// value the paper prints: all of them are the mathematics listed above.
//
// Build: g++ -O2 -fopenmp -ffp-contract=off -shared -fPIC (see oracle/build.py)

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

typedef int64_t i64;

struct Dims {
  int32_t batch, seqlen, nheads, headdim, dstate, ngroups, chunk;
};

// ---- binary32 building blocks (never contracted: compiled with -ffp-contract=off)
inline float fmul(float a, float b) { return a * b; }
inline float fsub(float a, float b) { return a - b; }
inline float fdiv(float a, float b) { return a / b; }

inline float f_from_bits(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }
inline uint32_t bits_from_f(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

// round half to even, then saturate to [-127, 127] ("nearest quantised level",
// Eq. 1; 2^(b-1)-1 levels on each side, so -128 is never produced)
inline int8_t rne_clamp(float v) {
  float r = std::nearbyintf(v);  // default rounding mode: to nearest, ties to even
  if (!(r >= -127.0f)) r = -127.0f;  // also catches NaN
  if (r > 127.0f) r = 127.0f;
  return (int8_t)(int)r;
}

// exp32: binary32 exponential used wherever an exponential feeds a rounding
// decision.  Cody-Waite reduction x = n ln2 + r, degree-7 Taylor polynomial in
// r by Horner with fused multiply-adds, scaling by 2^n through the exponent
// field.  Arguments below -80 give exactly 0; arguments above +80 are clamped
// (the method only ever passes x <= 0 because dt > 0 and A < 0).
inline float exp32(float x) {
  if (!(x >= -80.0f)) return 0.0f;
  if (x > 80.0f) x = 80.0f;
  const float LOG2E = f_from_bits(0x3FB8AA3Bu);    // 1.44269502
  const float LN2_HI = f_from_bits(0x3F317200u);   // 0.693145752 (low mantissa bits zero)
  const float LN2_LO = f_from_bits(0x35BFBE8Eu);   // 1.42860677e-6
  float n = std::nearbyintf(fmul(x, LOG2E));
  float r = std::fmaf(n, -LN2_HI, x);
  r = std::fmaf(n, -LN2_LO, r);
  float p = f_from_bits(0x39500D01u);               // 1/5040
  p = std::fmaf(p, r, f_from_bits(0x3AB60B61u));    // 1/720
  p = std::fmaf(p, r, f_from_bits(0x3C088889u));    // 1/120
  p = std::fmaf(p, r, f_from_bits(0x3D2AAAABu));    // 1/24
  p = std::fmaf(p, r, f_from_bits(0x3E2AAAABu));    // 1/6
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  uint32_t u = bits_from_f(p) + ((uint32_t)((int32_t)n) << 23);
  return f_from_bits(u);
}

// round(a b) saturated, a b being the exact product (48 significant bits: exact in binary64)
inline int8_t rne_clamp_exact_product(float a, float b) {
  double r = std::nearbyint((double)a * (double)b);
  if (!(r >= -127.0)) r = -127.0;
  if (r > 127.0) r = 127.0;
  return (int8_t)(int)r;
}

inline int sub_block(int Q) { return Q < 16 ? Q : 16; }

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------
// exp32 over an array (exposed so the tests can pin it against libm)
void orc_exp32(const float* x, float* out, i64 n) {
  for (i64 i = 0; i < n; ++i) out[i] = exp32(x[i]);
}

// ---------------------------------------------------------------------------
// Eq. 1: uniform symmetric quantiser.  View in[R][Ch][I], one step size per Ch.
//   alpha = absmax / 127 (1 if the channel is all zero), q = round(v / alpha),
//   quotient formed in binary32 by true division, ties to even, saturated.
// mode 0: static (alpha given)   mode 1: calibrate (alpha written, then quantise)
// mode 2: observe (alpha = max(alpha, absmax/127); out may be NULL)
void orc_quantize(const float* in, i64 R, i64 Ch, i64 I, float* scale, int mode, int8_t* out) {
  if (mode == 1 || mode == 2) {
    for (i64 ch = 0; ch < Ch; ++ch) {
      float m = 0.0f;
      for (i64 r = 0; r < R; ++r)
        for (i64 i = 0; i < I; ++i) {
          float a = std::fabs(in[(r * Ch + ch) * I + i]);
          if (a > m) m = a;
        }
      float alpha = (m == 0.0f) ? 1.0f : fdiv(m, 127.0f);
      if (mode == 2) {
        // an all-zero observation leaves the running step size unchanged
        if (m != 0.0f && alpha > scale[ch]) scale[ch] = alpha;
      } else {
        scale[ch] = alpha;
      }
    }
  }
  if (!out) return;
#pragma omp parallel for
  for (i64 r = 0; r < R; ++r)
    for (i64 ch = 0; ch < Ch; ++ch) {
      float alpha = scale[ch];
      for (i64 i = 0; i < I; ++i) {
        i64 k = (r * Ch + ch) * I + i;
        out[k] = rne_clamp(fdiv(in[k], alpha));
      }
    }
}

// ---------------------------------------------------------------------------
// L0: naive recurrence in fp64 on real-valued inputs.
// x [b,L,H,P], B,C [b,L,G,N], dt [b,L,H], A [H], D [H] or NULL, corr [H*P] or
// NULL, init [b,H,P,N] or NULL  ->  y [b,L,H,P], final [b,H,P,N] (may be NULL)
void orc_ssd_recurrence(const Dims* d, const double* x, const double* B, const double* C,
                        const double* dt, const double* A, const double* D, const double* corr,
                        const double* init, double* y, double* final_state) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups;
  const int hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<double> S((size_t)P * N, 0.0);
      if (init)
        for (int k = 0; k < P * N; ++k) S[k] = init[((i64)b * H + h) * P * N + k];
      for (int t = 0; t < L; ++t) {
        const double dtt = dt[((i64)b * L + t) * H + h];
        const double a = std::exp(dtt * A[h]);
        const double* xt = x + (((i64)b * L + t) * H + h) * P;
        const double* Bt = B + (((i64)b * L + t) * G + g) * N;
        const double* Ct = C + (((i64)b * L + t) * G + g) * N;
        double* yt = y + (((i64)b * L + t) * H + h) * P;
        for (int p = 0; p < P; ++p) {
          double acc = 0.0;
          for (int n = 0; n < N; ++n) {
            double s = a * S[(size_t)p * N + n] + dtt * xt[p] * Bt[n];
            S[(size_t)p * N + n] = s;
            acc += Ct[n] * s;
          }
          double v = acc;
          if (D) v += D[h] * xt[p];
          if (corr) v += corr[h * P + p];
          yt[p] = v;
        }
      }
      if (final_state)
        for (int k = 0; k < P * N; ++k) final_state[((i64)b * H + h) * P * N + k] = S[k];
    }
}

// ---------------------------------------------------------------------------
// L1: Algorithm 2 (SSD layer, chunked) in fp64 with no internal quantisation.
// Module by module, in the paper's order and names.  Two readings are fixed
// here and pinned by L1 == L0: ChunkScan1 multiplies by exp(dA_cs) only (the
// dt factor printed in LUT_scan1 does not belong there: dt already entered the
// state through LUT_state), and chunk k reads the state at the END of chunk
// k-1.  In LUT_scan2 the dt carries the column (source token) index and the
// causal mask keeps j <= i.
void orc_ssd_chunked(const Dims* d, const double* x, const double* B, const double* C,
                     const double* dt, const double* A, const double* D, const double* corr,
                     const double* init, double* y, double* final_state) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk;
  const int c = L / Q, hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<double> S((size_t)P * N, 0.0), loc((size_t)P * N), cs(Q), CB((size_t)Q * Q);
      if (init)
        for (int k = 0; k < P * N; ++k) S[k] = init[((i64)b * H + h) * P * N + k];
      for (int k = 0; k < c; ++k) {
        const i64 t0 = (i64)b * L + (i64)k * Q;
        // Module 1: ChunkCumsum
        double acc = 0.0;
        for (int i = 0; i < Q; ++i) {
          acc += dt[(t0 + i) * H + h] * A[h];
          cs[i] = acc;
        }
        // Module 4: ChunkBMM  CB[i][j] = sum_n C[i][n] B[j][n]
        for (int i = 0; i < Q; ++i)
          for (int j = 0; j <= i; ++j) {
            double s = 0.0;
            for (int n = 0; n < N; ++n)
              s += C[((t0 + i) * G + g) * N + n] * B[((t0 + j) * G + g) * N + n];
            CB[(size_t)i * Q + j] = s;
          }
        // Module 5 + 6 + final sum, using the state that entered this chunk
        for (int i = 0; i < Q; ++i) {
          const double* Ci = C + ((t0 + i) * G + g) * N;
          double* yi = y + ((t0 + i) * H + h) * P;
          const double dec = std::exp(cs[i]);
          for (int p = 0; p < P; ++p) {
            double off = 0.0;
            for (int n = 0; n < N; ++n) off += Ci[n] * S[(size_t)p * N + n];
            double diag = 0.0;
            for (int j = 0; j <= i; ++j) {
              const double lut = dt[(t0 + j) * H + h] * std::exp(cs[i] - cs[j]);
              diag += CB[(size_t)i * Q + j] * lut * x[((t0 + j) * H + h) * P + p];
            }
            double v = off * dec + diag;
            if (D) v += D[h] * x[((t0 + i) * H + h) * P + p];
            if (corr) v += corr[h * P + p];
            yi[p] = v;
          }
        }
        // Module 2: ChunkState with LUT_state moved onto X (Eq. 3: the product
        // is unchanged because LUT_state runs along the contracted axis l)
        for (int k2 = 0; k2 < P * N; ++k2) loc[k2] = 0.0;
        for (int i = 0; i < Q; ++i) {
          const double lut = dt[(t0 + i) * H + h] * std::exp(cs[Q - 1] - cs[i]);
          for (int p = 0; p < P; ++p) {
            const double xs = lut * x[((t0 + i) * H + h) * P + p];
            for (int n = 0; n < N; ++n)
              loc[(size_t)p * N + n] += xs * B[((t0 + i) * G + g) * N + n];
          }
        }
        // Module 3: StatePassing  State_k = loc_k + Decay_pass_k * State_{k-1}
        const double gam = std::exp(cs[Q - 1]);
        for (int k2 = 0; k2 < P * N; ++k2) S[k2] = loc[k2] + gam * S[k2];
      }
      if (final_state)
        for (int k2 = 0; k2 < P * N; ++k2) final_state[((i64)b * H + h) * P * N + k2] = S[k2];
    }
}

// ---------------------------------------------------------------------------
// Algorithm 2 module 1, first line: dt = softplus(dt_raw + dt_bias).
// Plain definition: log(1 + exp(v)) with libm in binary64, rounded to binary32 once; v = dt_raw + bias is
// the sum of two binary32 tensors as a binary32 tensor (the reading taken: the bias is added in the
// tensors' own precision, as a framework would, before the softplus is evaluated).
void orc_softplus_dt_plain(const float* dt_raw, const float* bias, i64 rows, i64 H, float* out) {
  for (i64 r = 0; r < rows; ++r)
    for (i64 h = 0; h < H; ++h) {
      const float v32 = bias ? dt_raw[r * H + h] + bias[h] : dt_raw[r * H + h];
      const double v = (double)v32;
      out[r * H + h] = (float)(std::fmax(v, 0.0) + std::log1p(std::exp(-std::fabs(v))));
    }
}

// The library's operation-by-operation softplus (binary64, every operation a single correctly rounded
// add, multiply, divide or fused multiply-add), so that dt is defined bit for bit:
//   v  = (double) fadd(dt_raw, bias)            (binary32 sum, then widened)
//   a  = |v|;  u = exp(-a):  n = rint(-a LOG2E), r = fma(n, -LN2_HI, -a), r = fma(n, -LN2_LO, r),
//        degree-13 Taylor polynomial in r (Horner, fma), scaled by 2^n; u = 0 for a > 700
//   lp = log(1 + u) = 2 atanh(s), s = u / (2 + u): 2 s (1 + z/3 + z^2/5 + ... + z^13/27), z = s s (Horner, fma)
//   dt = (float)(max(v, 0) + lp)
inline double softplus64(double v) {
  const double a = std::fabs(v);
  double u = 0.0;
  if (a <= 700.0) {
    const double LOG2E = 0x1.71547652b82fep+0, LN2_HI = 0x1.62e42fee00000p-1, LN2_LO = 0x1.a39ef35793c76p-33;
    const double n = std::nearbyint(-a * LOG2E);
    double r = std::fma(n, -LN2_HI, -a);
    r = std::fma(n, -LN2_LO, r);
    double p = 1.0 / 6227020800.0;                    // 1/13!
    const double inv_fact[13] = {1.0 / 479001600.0, 1.0 / 39916800.0, 1.0 / 3628800.0, 1.0 / 362880.0,
                                 1.0 / 40320.0, 1.0 / 5040.0, 1.0 / 720.0, 1.0 / 120.0, 1.0 / 24.0,
                                 1.0 / 6.0, 0.5, 1.0, 1.0};
    for (int k = 0; k < 13; ++k) p = std::fma(p, r, inv_fact[k]);
    uint64_t bits;
    std::memcpy(&bits, &p, 8);
    bits += (uint64_t)((int64_t)n) << 52;             // p 2^n: n >= -1010, p in [0.7, 1.42], so the result is normal
    std::memcpy(&u, &bits, 8);
  }
  const double s = u / (2.0 + u), z = s * s;
  double q = 1.0 / 27.0;
  for (int k = 12; k >= 0; --k) q = std::fma(q, z, 1.0 / (double)(2 * k + 1));
  const double lp = 2.0 * s * q;
  return (v > 0.0 ? v : 0.0) + lp;
}

void orc_softplus_dt(const float* dt_raw, const float* bias, i64 rows, i64 H, float* out) {
  for (i64 r = 0; r < rows; ++r)
    for (i64 h = 0; h < H; ++h) {
      const float v32 = bias ? dt_raw[r * H + h] + bias[h] : dt_raw[r * H + h];
      out[r * H + h] = (float)softplus64((double)v32);
    }
}

// ---------------------------------------------------------------------------
// L2 stage: ChunkCumsum (Algorithm 2, module 1).  dt is already positive
// (post-softplus).  The running sum is carried in fp64 in token order (each
// product dt*A of two binary32 numbers is exact in fp64) and stored as
// binary32: cs[b,h,k,i].
void orc_chunk_cumsum(const Dims* d, const float* dt, const float* A, float* cs) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, Q = d->chunk, c = L / Q;
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int k = 0; k < c; ++k) {
        double acc = 0.0;
        for (int i = 0; i < Q; ++i) {
          acc += (double)dt[((i64)b * L + (i64)k * Q + i) * H + h] * (double)A[h];
          cs[(((i64)b * H + h) * c + k) * Q + i] = (float)acc;
        }
      }
}

// ---------------------------------------------------------------------------
// L2 stage: ChunkBMM on the group axis (Section 4.2, "Quantization of ChunkBMM
// and ChunkScan2"): acc_cb[b,k,g,i,j] = sum_n Cq[i,n] Bq[j,n] exactly, then one
// INT32 -> INT8 step  CBq = round(acc_cb * r_cb),  r_cb = fdiv(fmul(s_C,s_B), s_cb).
// All Q x Q entries are written; only j <= i is consumed downstream.
void orc_chunk_bmm(const Dims* d, const int8_t* Cq, const int8_t* Bq, const float* s_C,
                   const float* s_B, const float* s_cb, int32_t* acc_cb, int8_t* CBq) {
  const int b_ = d->batch, L = d->seqlen, N = d->dstate, G = d->ngroups, Q = d->chunk, c = L / Q;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int k = 0; k < c; ++k)
      for (int g = 0; g < G; ++g) {
        const float r_cb = s_cb ? fdiv(fmul(s_C[g], s_B[g]), s_cb[g]) : 0.0f;
        const i64 t0 = (i64)b * L + (i64)k * Q;
        for (int i = 0; i < Q; ++i)
          for (int j = 0; j < Q; ++j) {
            int32_t s = 0;
            for (int n = 0; n < N; ++n)
              s += (int32_t)Cq[((t0 + i) * G + g) * N + n] * (int32_t)Bq[((t0 + j) * G + g) * N + n];
            const i64 o = ((((i64)b * c + k) * G + g) * Q + i) * Q + j;
            if (acc_cb) acc_cb[o] = s;
            if (CBq) CBq[o] = rne_clamp(fmul((float)s, r_cb));
          }
      }
}

// ---------------------------------------------------------------------------
// L2 stage: ChunkState with the sparse-aware reformulation (Eq. 3) and the
// INT32 rescale (Eq. 4, here to fp32 because the inter-chunk states are fp32):
//   LUT_state[i] = fmul(dt_i, exp32(fsub(cs_last, cs_i)))
//   Xs_q[i,p]    = round(fmul(fmul(float(xq[i,p]), r_x[h,p]), LUT_state[i])),
//                  r_x = fdiv(s_x, s_xs)                       (per-(H,P) scale)
//   acc_st[p,n]  = sum_i Xs_q[i,p] Bq[i,n]                     (exact)
//   loc[p,n]     = fmul(float(acc_st), fmul(s_xs[h,p], s_B[g]))
void orc_chunk_state(const Dims* d, const int8_t* xq, const int8_t* Bq, const float* s_x,
                     const float* s_xs, const float* s_B, const float* dt, const float* cs,
                     int8_t* Xsq, int32_t* acc_st, float* loc) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<int8_t> xs((size_t)Q * P);
      for (int k = 0; k < c; ++k) {
        const i64 t0 = (i64)b * L + (i64)k * Q;
        const float* csk = cs + (((i64)b * H + h) * c + k) * Q;
        for (int i = 0; i < Q; ++i) {
          const float lut = fmul(dt[(t0 + i) * H + h], exp32(fsub(csk[Q - 1], csk[i])));
          for (int p = 0; p < P; ++p) {
            const float r_x = fdiv(s_x[h * P + p], s_xs[h * P + p]);
            const i64 o = ((t0 + i) * H + h) * P + p;
            const int8_t q = rne_clamp(fmul(fmul((float)xq[o], r_x), lut));
            xs[(size_t)i * P + p] = q;
            if (Xsq) Xsq[o] = q;
          }
        }
        for (int p = 0; p < P; ++p)
          for (int n = 0; n < N; ++n) {
            int32_t s = 0;
            for (int i = 0; i < Q; ++i)
              s += (int32_t)xs[(size_t)i * P + p] * (int32_t)Bq[((t0 + i) * G + g) * N + n];
            const i64 o = ((((i64)b * c + k) * H + h) * P + p) * N + n;
            if (acc_st) acc_st[o] = s;
            if (loc) loc[o] = fmul((float)s, fmul(s_xs[h * P + p], s_B[g]));
          }
      }
    }
}

// ---------------------------------------------------------------------------
// L2 stage: StatePassing (Eq. 5-6; Algorithm 2 module 3) on fp32 states:
//   Gamma_k = exp32(cs[k, Q-1]);  S_k = fmaf(Gamma_k, S_{k-1}, loc_k);  S_{-1} = init or 0
//   prev[k] = S_{k-1}  (the state chunk k reads),  final = S_{c-1}
//   hq[k]   = round(fmul(prev[k], inv_h)),  inv_h = fdiv(1, s_h[h,p])   (Eq. 4 rescale, per-(H,P))
// gamma may be passed directly (standalone entry point) or derived from cs.
void orc_state_passing(const Dims* d, const float* loc, const float* gamma, const float* init,
                       const float* s_h, float* prev, float* final_state, int8_t* hq) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            Q = d->chunk, c = L / Q;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int p = 0; p < P; ++p) {
        const float inv_h = s_h ? fdiv(1.0f, s_h[h * P + p]) : 0.0f;
        for (int n = 0; n < N; ++n) {
          float S = init ? init[(((i64)b * H + h) * P + p) * N + n] : 0.0f;
          for (int k = 0; k < c; ++k) {
            const i64 o = ((((i64)b * c + k) * H + h) * P + p) * N + n;
            const float l = loc[o];  // read before prev[o] is written: prev may alias loc
            if (hq) hq[o] = rne_clamp(fmul(S, inv_h));
            if (prev) prev[o] = S;
            S = std::fmaf(gamma[((i64)b * H + h) * c + k], S, l);
          }
          if (final_state) final_state[(((i64)b * H + h) * P + p) * N + n] = S;
        }
      }
}

// ---------------------------------------------------------------------------
// L2 stage, the paper's own state format: persistent INT8 states with a fixed-point decay
// (Section 4.2 "Persistent INT8 Representation of Recurrent States", Eq. 4 and Eq. 7).
//   r_st[h,p] = fdiv(fmul(s_xs[h,p], s_B[g]), s_h[h,p])        (Eq. 4: s_x s_b q_max / s_s)
//   locq_k    = round(fmul(float(acc_st_k), r_st))             INT32 -> INT8, per-(H,P) scale s_h
//   Gq_k      = round(fmul(Gamma_k, 128))  in [0, 128]         Q(Decay), S = 2^7
//   Sq_k      = sat(locq_k + ((Gq_k * Sq_{k-1} + 64) >> 7))    Eq. 7: multiply, shift by k = 7 with
//               rounding (floor((v + 64) / 128)), saturate to [-127, 127]
//   Sq_{-1}   = round(fmul(init, fdiv(1, s_h))) or 0;  hq[k] = Sq_{k-1};  final = fmul(float(Sq_{c-1}), s_h)
// All states of all chunks share the one scale s_h[h,p], which is what makes the shift exact.
void orc_state_passing_int8(const Dims* d, const int32_t* acc_st, const float* gamma,
                            const float* init, const float* s_xs, const float* s_B,
                            const float* s_h, int8_t* hq, float* final_state) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int p = 0; p < P; ++p) {
        const float sh = s_h[h * P + p];
        const float r_st = fdiv(fmul(s_xs[h * P + p], s_B[h / hpg]), sh);
        const float inv_h = fdiv(1.0f, sh);
        for (int n = 0; n < N; ++n) {
          int Sq = init ? (int)rne_clamp(fmul(init[(((i64)b * H + h) * P + p) * N + n], inv_h)) : 0;
          for (int k = 0; k < c; ++k) {
            const i64 o = ((((i64)b * c + k) * H + h) * P + p) * N + n;
            hq[o] = (int8_t)Sq;
            const int locq = (int)rne_clamp(fmul((float)acc_st[o], r_st));
            const int Gq = (int)std::nearbyintf(fmul(gamma[((i64)b * H + h) * c + k], 128.0f));
            const int v = Gq * Sq + 64;
            const int shifted = (v >= 0) ? (v / 128) : -((-v + 127) / 128);  // floor(v / 128)
            int Sn = locq + shifted;
            if (Sn > 127) Sn = 127;
            if (Sn < -127) Sn = -127;
            Sq = Sn;
          }
          if (final_state) final_state[(((i64)b * H + h) * P + p) * N + n] = fmul((float)Sq, sh);
        }
      }
}

// Gamma[b,h,k] = exp32(cs[b,h,k,Q-1])   (Decay_pass of Eq. 5)
void orc_chunk_decay(const Dims* d, const float* cs, float* gamma) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, Q = d->chunk, c = L / Q;
  for (i64 u = 0; u < (i64)b_ * H * c; ++u) gamma[u] = exp32(cs[u * Q + Q - 1]);
}

// ---------------------------------------------------------------------------
// L2 stage: ChunkScan1 + ChunkScan2 + output sum (Algorithm 2 modules 5, 6) in the library's
// operation-by-operation binary32 arithmetic (the interface fixed in the library's header, so
// that codes can be compared bit for bit).  This is NOT the definition: the definition is
// orc_chunk_scan_plain further down, and the tests bound the distance between the two.
//  off-diagonal:  acc_off[i,p] = sum_n Cq[i,n] hq[k][p,n]  (exact)
//                 y_off = exp(cs_i) s_C s_h[h,p] acc_off   (decay applied after the product)
//  diagonal: the masked operand CB o LUT_scan2 is re-quantised per output row i
//  so that the product with int8 X is an integer GEMM.  With sub-blocks of
//  SB = min(16, Q) tokens, je = last column of the sub-block of j:
//     same sub-block:  the decay is the running product of the per-token decays
//                      a_m = exp32(fsub(cs_m, cs_{m-1})):  E[i,i] = 1, E[i,j] = fmul(E[i,j+1], a_{j+1});
//                      w = fmul(dt_j, E[i,j]),  f = 1
//     earlier block :  w = fmul(dt_j, exp32(fsub(cs_je, cs_j))),
//                      f = fmul(exp32(fsub(cs_i, cs_pe)), exp32(fsub(cs_pe, cs_je))), pe = last token of the
//                      sub-block before the row's own
//     t[i,j]   = fmul(float(CBq[i,j]), w)          (w f = dt_j exp(cs_i - cs_j); every exponent <= 0)
//     rowmax_i = max over sub-blocks J of fmul(max_{j in J, j<=i} |t[i,j]|, f)
//     inv_i    = rowmax_i >= 1e-30 ? fdiv(127, rowmax_i) : 0
//     Mq[i,j]  = round(t[i,j] * fmul(f, inv_i)), the exact product rounded once (one fused operation)
//     acc_diag[i,p] = sum_{j<=i} Mq[i,j] xq[j,p]    (exact)
//     y_diag   = (s_cb rowmax_i / 127) s_x[h,p] acc_diag
//  y = y_off + y_diag + D s_x xq + corr
// Round to the nearest IEEE binary16 value, ties to even (11 significant bits, subnormal quantum
// 2^-24, overflow to infinity), returned as a double.  Used by the paper's FP16 ChunkScan2 operand.
double orc_round_half(double v) {
  if (v == 0.0 || std::isnan(v) || std::isinf(v)) return v;
  int e;
  (void)std::frexp(std::fabs(v), &e);                  // |v| = m 2^e, m in [0.5, 1)
  const int q = (e - 1 < -14) ? -24 : e - 11;          // exponent of the spacing around |v|
  const double r = std::ldexp(std::nearbyint(std::ldexp(std::fabs(v), -q)), q);
  const double out = (r >= 65520.0) ? INFINITY : r;    // 65520 = the midpoint above the largest half
  return v < 0 ? -out : out;
}

// flags bit 0 (value 1): the paper's own ChunkScan2 operand (Section 4.2; Algorithm 2, module 6):
// no per-row re-quantisation; the masked operand is kept in FP16 with the dequantisation scale of
// CB fused into the look-up table,  M16[i,j] = half(s_cb CBq[i,j] dt_j exp(cs_i - cs_j)), j <= i,
// X enters as the exact FP16 image of its int8 codes, and  y_diag = s_x sum_j M16[i,j] xq[j,p]
// (accumulated here in binary64).  The value that is rounded to FP16 is the binary32 product
// fmul(t[i,j], fmul(f, s_cb)) with t and f of the sub-block factorisation below (f = 1 in the
// row's own sub-block).  rowmax, Mq and acc_diag are not produced in that mode.
void orc_chunk_scan(const Dims* d, const int8_t* xq, const int8_t* Cq, const int8_t* CBq,
                    const int8_t* hq, const float* s_x, const float* s_C, const float* s_cb,
                    const float* s_h, const float* dt, const float* cs, const float* D,
                    const float* corr, int32_t* acc_off, float* rowmax, int8_t* Mq,
                    int32_t* acc_diag, double* y, uint32_t flags, double* M16) {
  const bool fp16_operand = (flags & 1u) != 0;
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
  const int SB = sub_block(Q);
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<float> t(Q), f(Q / SB + 1), a_tok(Q);
      std::vector<int8_t> mq(Q);
      std::vector<double> m16(Q);
      for (int k = 0; k < c; ++k) {
        const i64 t0 = (i64)b * L + (i64)k * Q;
        const float* csk = cs + (((i64)b * H + h) * c + k) * Q;
        const int8_t* cbk = CBq + (((i64)b * c + k) * G + g) * Q * Q;
        const int8_t* hqk = hq + (((i64)b * c + k) * H + h) * P * N;
        a_tok[0] = 1.0f;  // never used: a_m enters only for m >= 1
        for (int m = 1; m < Q; ++m) a_tok[m] = exp32(fsub(csk[m], csk[m - 1]));
        for (int i = 0; i < Q; ++i) {
          const int I = i / SB;
          float rmax = 0.0f;
          for (int J = 0; J <= I; ++J) {
            const int je = J * SB + SB - 1;
            // earlier block: the decay from the block's last token to row i as the product of the row's
            // decay to the end of the block before its own (pe) and the block-to-block decay from there
            // (1 for the block next to the row's own: pe = je)
            const int pe = I * SB - 1;
            f[J] = (J == I) ? 1.0f : fmul(exp32(fsub(csk[i], csk[pe])), exp32(fsub(csk[pe], csk[je])));
            float bmax = 0.0f;
            float E = 1.0f;
            for (int j = (J == I ? i : je); j >= J * SB; --j) {
              float e;
              if (J == I) {
                if (j < i) E = fmul(E, a_tok[j + 1]);
                e = E;
              } else {
                e = exp32(fsub(csk[je], csk[j]));
              }
              const float w = fmul(dt[(t0 + j) * H + h], e);
              t[j] = fmul((float)cbk[(size_t)i * Q + j], w);
              const float a = std::fabs(t[j]);
              if (a > bmax) bmax = a;
            }
            const float m = fmul(bmax, f[J]);
            if (m > rmax) rmax = m;
          }
          if (fp16_operand) {
            // the value that is rounded to FP16 is formed in binary32 in this order (a rounding
            // decision: both sides of a parity test must take it in the same precision)
            for (int j = 0; j <= i; ++j)
              m16[j] = orc_round_half((double)fmul(t[j], (j / SB == I) ? s_cb[g] : fmul(f[j / SB], s_cb[g])));
            if (M16) {  // [b,c,H,Q,Q], zero above the diagonal
              double* o = M16 + ((((i64)b * c + k) * H + h) * Q + i) * Q;
              for (int j = 0; j < Q; ++j) o[j] = (j <= i) ? m16[j] : 0.0;
            }
            const double dec = std::exp((double)csk[i]);
            for (int p = 0; p < P; ++p) {
              int32_t ao = 0;
              for (int n = 0; n < N; ++n)
                ao += (int32_t)Cq[((t0 + i) * G + g) * N + n] * (int32_t)hqk[(size_t)p * N + n];
              double ad = 0.0;
              for (int j = 0; j <= i; ++j) ad += m16[j] * (double)xq[((t0 + j) * H + h) * P + p];
              const i64 o = ((t0 + i) * H + h) * P + p;
              if (acc_off) acc_off[o] = ao;
              double v = dec * (double)s_C[g] * (double)s_h[h * P + p] * (double)ao +
                         (double)s_x[h * P + p] * ad;
              if (D) v += (double)D[h] * (double)s_x[h * P + p] * (double)xq[o];
              if (corr) v += (double)corr[h * P + p];
              y[o] = v;
            }
            continue;
          }
          const float inv = (rmax >= 1e-30f) ? fdiv(127.0f, rmax) : 0.0f;
          for (int j = 0; j < Q; ++j) mq[j] = 0;
          // the product t g is rounded once, to the nearest integer (ties to even): the exact product
          // of two binary32 numbers fits a binary64
          for (int j = 0; j <= i; ++j) mq[j] = rne_clamp_exact_product(t[j], fmul(f[j / SB], inv));
          if (rowmax) rowmax[(t0 + i) * H + h] = rmax;
          if (Mq) {
            int8_t* o = Mq + ((((i64)b * c + k) * H + h) * Q + i) * Q;
            for (int j = 0; j < Q; ++j) o[j] = mq[j];
          }
          const double dec = std::exp((double)csk[i]);
          const double s_m = (double)s_cb[g] * (double)rmax / 127.0;
          for (int p = 0; p < P; ++p) {
            int32_t ao = 0;
            for (int n = 0; n < N; ++n)
              ao += (int32_t)Cq[((t0 + i) * G + g) * N + n] * (int32_t)hqk[(size_t)p * N + n];
            int32_t ad = 0;
            for (int j = 0; j <= i; ++j)
              ad += (int32_t)mq[j] * (int32_t)xq[((t0 + j) * H + h) * P + p];
            const i64 o = ((t0 + i) * H + h) * P + p;
            if (acc_off) acc_off[o] = ao;
            if (acc_diag) acc_diag[o] = ad;
            double v = dec * (double)s_C[g] * (double)s_h[h * P + p] * (double)ao +
                       s_m * (double)s_x[h * P + p] * (double)ad;
            if (D) v += (double)D[h] * (double)s_x[h * P + p] * (double)xq[o];
            if (corr) v += (double)corr[h * P + p];
            y[o] = v;
          }
        }
      }
    }
}

// ---------------------------------------------------------------------------
// PLAIN DEFINITIONS (fp64, libm).  Nothing below is blocked, factorised or reordered.

inline int8_t rne_clamp64(double v) {
  double r = std::nearbyint(v);          // ties to even
  if (!(r >= -127.0)) r = -127.0;
  if (r > 127.0) r = 127.0;
  return (int8_t)(int)r;
}

// Eq. 3, plain: X_scaled[i,p] = LUT_state[i] x[i,p] with LUT_state[i] = dt_i exp(cs_last - cs_i)
// (Algorithm 2 module 2) and x = s_x xq; its code is round(X_scaled / s_xs).  Writes the real
// quotient v = X_scaled / s_xs [b,L,H,P] (may be NULL) and the code (may be NULL).
void orc_chunk_state_plain(const Dims* d, const int8_t* xq, const float* s_x, const float* s_xs,
                           const float* dt, const float* cs, double* v_out, int8_t* Xsq) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, Q = d->chunk, c = L / Q;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int k = 0; k < c; ++k) {
        const float* csk = cs + (((i64)b * H + h) * c + k) * Q;
        for (int i = 0; i < Q; ++i) {
          const i64 t = (i64)b * L + (i64)k * Q + i;
          const double lut = (double)dt[t * H + h] * std::exp((double)csk[Q - 1] - (double)csk[i]);
          for (int p = 0; p < P; ++p) {
            const i64 o = (t * H + h) * P + p;
            const double v = (double)xq[o] * (double)s_x[h * P + p] * lut / (double)s_xs[h * P + p];
            if (v_out) v_out[o] = v;
            if (Xsq) Xsq[o] = rne_clamp64(v);
          }
        }
      }
}

// Eq. 4, plain: the code of a state element is round(State / s_h), per-(H,P) step size.
// S [b,c,H,P,N] (the state entering each chunk) -> v = S / s_h and its code.
void orc_state_codes_plain(const Dims* d, const float* S, const float* s_h, double* v_out,
                           int8_t* hq) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            Q = d->chunk, c = L / Q;
  for (i64 u = 0; u < (i64)b_ * c; ++u)
    for (int h = 0; h < H; ++h)
      for (int p = 0; p < P; ++p)
        for (int n = 0; n < N; ++n) {
          const i64 o = ((u * H + h) * P + p) * N + n;
          const double v = (double)S[o] / (double)s_h[h * P + p];
          if (v_out) v_out[o] = v;
          if (hq) hq[o] = rne_clamp64(v);
        }
}

// Algorithm 2 modules 5 and 6 and the output sum, plain.
//   ChunkScan1  y_off[i,p]  = exp(cs_i) sum_n C[i,n] State[p,n],  C = s_C Cq, State = s_h hq
//   ChunkScan2  LUT_scan2[i,j] = dt_j exp(cs_i - cs_j), j <= i (0 above the diagonal)
//               M[i,j]      = CB[i,j] LUT_scan2[i,j],  CB = s_cb CBq
//     int8 operand (flags bit 0 clear): Eq. 1 applied to each row of M,
//               s_M[i] = max_j |M[i,j]| / 127 (1 if the row is zero), Mq = round(M / s_M),
//               y_diag[i,p] = s_M[i] s_x[p] sum_j Mq[i,j] xq[j,p]
//     FP16 operand (flags bit 0 set; Section 4.2): M16 = half(M),
//               y_diag[i,p] = s_x[p] sum_j M16[i,j] xq[j,p]
//   y = y_off + y_diag + D s_x xq + corr
// Optional outputs: M [b,c,H,Q,Q] (the real operand, zero above the diagonal), sM [b,L,H]
// (int8 mode), Mq [b,c,H,Q,Q] (int8 mode).
void orc_chunk_scan_plain(const Dims* d, const int8_t* xq, const int8_t* Cq, const int8_t* CBq,
                          const int8_t* hq, const float* s_x, const float* s_C, const float* s_cb,
                          const float* s_h, const float* dt, const float* cs, const float* D,
                          const float* corr, double* M_out, double* sM_out, int8_t* Mq_out,
                          double* y, uint32_t flags) {
  const bool fp16_operand = (flags & 1u) != 0;
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<double> M(Q), W(Q);
      for (int k = 0; k < c; ++k) {
        const i64 t0 = (i64)b * L + (i64)k * Q;
        const float* csk = cs + (((i64)b * H + h) * c + k) * Q;
        const int8_t* cbk = CBq + (((i64)b * c + k) * G + g) * Q * Q;
        const int8_t* hqk = hq + (((i64)b * c + k) * H + h) * P * N;
        for (int i = 0; i < Q; ++i) {
          double amax = 0.0;
          for (int j = 0; j < Q; ++j) {
            M[j] = 0.0;
            if (j <= i) {
              const double lut = (double)dt[(t0 + j) * H + h] * std::exp((double)csk[i] - (double)csk[j]);
              M[j] = (double)s_cb[g] * (double)cbk[(size_t)i * Q + j] * lut;
            }
            amax = std::fmax(amax, std::fabs(M[j]));
          }
          const i64 row = ((((i64)b * c + k) * H + h) * Q + i) * Q;
          if (M_out) for (int j = 0; j < Q; ++j) M_out[row + j] = M[j];
          double sM = 1.0;
          if (fp16_operand) {
            for (int j = 0; j < Q; ++j) W[j] = orc_round_half(M[j]);
          } else {
            sM = (amax == 0.0) ? 1.0 : amax / 127.0;
            for (int j = 0; j < Q; ++j) {
              const int8_t q = rne_clamp64(M[j] / sM);
              W[j] = (double)q;
              if (Mq_out) Mq_out[row + j] = q;
            }
            if (sM_out) sM_out[(t0 + i) * H + h] = sM;
          }
          const double dec = std::exp((double)csk[i]);
          for (int p = 0; p < P; ++p) {
            double off = 0.0;
            for (int n = 0; n < N; ++n)
              off += (double)Cq[((t0 + i) * G + g) * N + n] * (double)hqk[(size_t)p * N + n];
            double diag = 0.0;
            for (int j = 0; j <= i; ++j) diag += W[j] * (double)xq[((t0 + j) * H + h) * P + p];
            const i64 o = ((t0 + i) * H + h) * P + p;
            double v = dec * (double)s_C[g] * (double)s_h[h * P + p] * off +
                       sM * (double)s_x[h * P + p] * diag;
            if (D) v += (double)D[h] * (double)s_x[h * P + p] * (double)xq[o];
            if (corr) v += (double)corr[h * P + p];
            y[o] = v;
          }
        }
      }
    }
}

// The whole SSDi8 forward from the plain definitions alone (Algorithm 2 with Eq. 1, 3, 4; fp32
// inter-chunk states replaced by fp64 ones), every rounding decided on fp64 values.  It shares
// only the exact integer stages and the cumulative sum with orc_ssdi8_fwd.  y fp64, final fp64.
void orc_ssdi8_fwd_plain(const Dims* d, const int8_t* xq, const int8_t* Bq, const int8_t* Cq,
                         const float* s_x, const float* s_B, const float* s_C, const float* dt,
                         const float* A, const float* D, const float* corr, const float* s_xs,
                         const float* s_cb, const float* s_h, const float* init, double* y,
                         double* final_state, uint32_t flags) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
  std::vector<float> cs((size_t)b_ * H * L);
  orc_chunk_cumsum(d, dt, A, cs.data());                       // module 1
  // module 4: ChunkBMM, one INT32 -> INT8 step (Section 4.2)
  std::vector<int32_t> acc_cb((size_t)b_ * c * G * Q * Q);
  std::vector<int8_t> CBq(acc_cb.size());
  orc_chunk_bmm(d, Cq, Bq, s_C, s_B, nullptr, acc_cb.data(), nullptr);
  for (i64 u = 0; u < (i64)b_ * c; ++u)
    for (int g = 0; g < G; ++g)
      for (i64 e = 0; e < (i64)Q * Q; ++e) {
        const i64 o = (u * G + g) * Q * Q + e;
        CBq[o] = rne_clamp64((double)acc_cb[o] * (double)s_C[g] * (double)s_B[g] / (double)s_cb[g]);
      }
  // module 2: ChunkState (Eq. 3), exact integer product, Eq. 4 rescale to a real-valued state
  std::vector<int8_t> Xsq((size_t)b_ * L * H * P);
  orc_chunk_state_plain(d, xq, s_x, s_xs, dt, cs.data(), nullptr, Xsq.data());
  const size_t nst = (size_t)b_ * c * H * P * N;
  std::vector<int8_t> hq(nst);
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      std::vector<double> S((size_t)P * N, 0.0);
      if (init) for (int e = 0; e < P * N; ++e) S[e] = (double)init[((i64)b * H + h) * P * N + e];
      for (int k = 0; k < c; ++k) {
        const i64 t0 = (i64)b * L + (i64)k * Q;
        const double gam = std::exp((double)cs[(((i64)b * H + h) * c + k) * Q + Q - 1]);  // Eq. 5
        for (int p = 0; p < P; ++p)
          for (int n = 0; n < N; ++n) {
            const i64 o = ((((i64)b * c + k) * H + h) * P + p) * N + n;
            hq[o] = rne_clamp64(S[(size_t)p * N + n] / (double)s_h[h * P + p]);   // Eq. 4
            i64 a = 0;
            for (int i = 0; i < Q; ++i)
              a += (i64)Xsq[((t0 + i) * H + h) * P + p] * (i64)Bq[((t0 + i) * G + g) * N + n];
            const double loc = (double)a * (double)s_xs[h * P + p] * (double)s_B[g];
            S[(size_t)p * N + n] = loc + gam * S[(size_t)p * N + n];               // Eq. 6
          }
      }
      if (final_state)
        for (int e = 0; e < P * N; ++e) final_state[((i64)b * H + h) * P * N + e] = S[e];
    }
  orc_chunk_scan_plain(d, xq, Cq, CBq.data(), hq.data(), s_x, s_C, s_cb, s_h, dt, cs.data(), D,
                       corr, nullptr, nullptr, nullptr, y, flags);
}

// ---------------------------------------------------------------------------
// Diagnostic of Proposition 1 (Appendix A): mean squared error of the two ways of putting
// y = x (.) lut on an 8-bit grid, on real-valued x [b,L,H,P]:
//   out[0] = error of deq(Q(x (.) LUT_state))   (the reformulation, Eq. 3: quantise X_scaled),
//            mean over all elements (the proof's MSE_x_scaled: an expectation per element)
//   out[1] = error of deq(Q(x)) (.) LUT_state   (quantise X, scale afterwards), mean over all elements
//   out[2] = fraction of Q(X_scaled) codes that are zero (the proof's 1 - rho)
//   out[3] = the proof's MSE_x: the squared norm of the second error over the l axis of one chunk
//            (its Step 3 sums over l), mean over chunks, heads and channels; equals out[1] * Q.
// The proposition as printed compares out[0] with out[3], i.e. a per-element mean with a per-vector
// sum; both normalisations are returned.  Each Q is Eq. 1 with one step size per channel (h,p)
// calibrated on the tensor it is applied to (absmax / 127), LUT_state[i] = dt_i exp(cs_last - cs_i).
void orc_prop1_mse(const Dims* d, const float* x, const float* dt, const float* cs, double* out) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, Q = d->chunk, c = L / Q;
  const i64 T = (i64)b_ * L;
  std::vector<double> lut((size_t)T * H), ax((size_t)H * P, 0.0), ay((size_t)H * P, 0.0);
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int k = 0; k < c; ++k) {
        const float* csk = cs + (((i64)b * H + h) * c + k) * Q;
        for (int i = 0; i < Q; ++i) {
          const i64 t = (i64)b * L + (i64)k * Q + i;
          lut[t * H + h] = (double)dt[t * H + h] * std::exp((double)csk[Q - 1] - (double)csk[i]);
        }
      }
  for (i64 t = 0; t < T; ++t)
    for (int ch = 0; ch < H * P; ++ch) {
      const double xv = (double)x[t * H * P + ch], yv = xv * lut[t * H + ch / P];
      ax[ch] = std::fmax(ax[ch], std::fabs(xv));
      ay[ch] = std::fmax(ay[ch], std::fabs(yv));
    }
  double e_scaled = 0.0, e_x = 0.0;
  i64 zeros = 0;
  for (i64 t = 0; t < T; ++t)
    for (int ch = 0; ch < H * P; ++ch) {
      const double l = lut[t * H + ch / P], xv = (double)x[t * H * P + ch], yv = xv * l;
      const double sx = ax[ch] == 0.0 ? 1.0 : ax[ch] / 127.0, sy = ay[ch] == 0.0 ? 1.0 : ay[ch] / 127.0;
      const int qy = (int)rne_clamp64(yv / sy), qx = (int)rne_clamp64(xv / sx);
      zeros += (qy == 0);
      const double ea = sy * qy - yv, eb = sx * qx * l - yv;
      e_scaled += ea * ea;
      e_x += eb * eb;
    }
  const double n = (double)T * H * P;
  out[0] = e_scaled / n;
  out[1] = e_x / n;
  out[2] = (double)zeros / n;
  out[3] = out[1] * (double)Q;
}

// ---------------------------------------------------------------------------
// Static calibration of the internal step sizes (Eq. 1 applied to the internal
// tensors, once, on the tensors given):
//   s_xs[h,p] over (b,t) of |fmul(fmul(float(xq), s_x), LUT_state)|
//   s_cb[g]   over the causal half of |acc_cb| * fmul(s_C, s_B)
//   s_h[h,p]  over init and every S_k (k = 0..c-1), all b and n   (one scale for all chunks)
// Each is fdiv(absmax, 127), or 1 if the absmax is 0.
void orc_calibrate(const Dims* d, const int8_t* xq, const int8_t* Bq, const int8_t* Cq,
                   const float* s_x, const float* s_B, const float* s_C, const float* dt,
                   const float* A, const float* init, float* s_xs, float* s_cb, float* s_h) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q, hpg = H / G;
  std::vector<float> cs((size_t)b_ * H * L), gamma((size_t)b_ * H * c);
  orc_chunk_cumsum(d, dt, A, cs.data());
  orc_chunk_decay(d, cs.data(), gamma.data());
  // s_xs
  std::vector<float> mx((size_t)H * P, 0.0f);
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int k = 0; k < c; ++k) {
        const float* csk = cs.data() + (((i64)b * H + h) * c + k) * Q;
        for (int i = 0; i < Q; ++i) {
          const i64 t = (i64)b * L + (i64)k * Q + i;
          const float lut = fmul(dt[t * H + h], exp32(fsub(csk[Q - 1], csk[i])));
          for (int p = 0; p < P; ++p) {
            const float v = std::fabs(fmul(fmul((float)xq[(t * H + h) * P + p], s_x[h * P + p]), lut));
            if (v > mx[h * P + p]) mx[h * P + p] = v;
          }
        }
      }
  for (int k = 0; k < H * P; ++k) s_xs[k] = mx[k] == 0.0f ? 1.0f : fdiv(mx[k], 127.0f);
  // s_cb
  std::vector<int32_t> acc((size_t)b_ * c * G * Q * Q);
  orc_chunk_bmm(d, Cq, Bq, s_C, s_B, nullptr, acc.data(), nullptr);
  for (int g = 0; g < G; ++g) {
    int32_t m = 0;
    for (int b = 0; b < b_; ++b)
      for (int k = 0; k < c; ++k)
        for (int i = 0; i < Q; ++i)
          for (int j = 0; j <= i; ++j) {
            int32_t v = std::abs(acc[((((i64)b * c + k) * G + g) * Q + i) * Q + j]);
            if (v > m) m = v;
          }
    s_cb[g] = m == 0 ? 1.0f : fdiv(fmul((float)m, fmul(s_C[g], s_B[g])), 127.0f);
  }
  // s_h
  std::vector<float> loc((size_t)b_ * c * H * P * N), prev(loc.size()), fin((size_t)b_ * H * P * N);
  orc_chunk_state(d, xq, Bq, s_x, s_xs, s_B, dt, cs.data(), nullptr, nullptr, loc.data());
  orc_state_passing(d, loc.data(), gamma.data(), init, nullptr, prev.data(), fin.data(), nullptr);
  for (int k = 0; k < H * P; ++k) mx[k] = 0.0f;
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h)
      for (int p = 0; p < P; ++p) {
        float m = mx[h * P + p];
        for (int n = 0; n < N; ++n) {
          for (int k = 0; k < c; ++k) {
            float v = std::fabs(prev[((((i64)b * c + k) * H + h) * P + p) * N + n]);
            if (v > m) m = v;
          }
          float v = std::fabs(fin[(((i64)b * H + h) * P + p) * N + n]);
          if (v > m) m = v;
        }
        mx[h * P + p] = m;
      }
  for (int k = 0; k < H * P; ++k) s_h[k] = mx[k] == 0.0f ? 1.0f : fdiv(mx[k], 127.0f);
  (void)hpg;
}

// ---------------------------------------------------------------------------
// L2: the whole SSDi8 layer forward.  Any tap pointer may be NULL.
struct Taps {
  float* cs; int32_t* acc_cb; int8_t* CBq; int8_t* Xsq; int32_t* acc_st; float* loc;
  float* prev; int8_t* hq; int32_t* acc_off; float* rowmax; int8_t* Mq; int32_t* acc_diag;
};

// flags bit 0 (value 1): the paper's FP16 ChunkScan2 operand (see orc_chunk_scan).
// flags bit 1 (value 2): the paper's persistent INT8 states (orc_state_passing_int8) instead of
// fp32 states; the loc and prev taps are not produced in that mode.
void orc_ssdi8_fwd(const Dims* d, const int8_t* xq, const int8_t* Bq, const int8_t* Cq,
                   const float* s_x, const float* s_B, const float* s_C, const float* dt,
                   const float* A, const float* D, const float* corr, const float* s_xs,
                   const float* s_cb, const float* s_h, const float* init, double* y,
                   float* final_state, const Taps* taps, uint32_t flags) {
  const int b_ = d->batch, L = d->seqlen, H = d->nheads, P = d->headdim, N = d->dstate,
            G = d->ngroups, Q = d->chunk, c = L / Q;
  Taps none;
  std::memset(&none, 0, sizeof(none));
  const Taps* tp = taps ? taps : &none;
  const size_t nst = (size_t)b_ * c * H * P * N;
  std::vector<float> cs_v, gamma((size_t)b_ * H * c), loc_v, prev_v;
  std::vector<int8_t> cbq_v, hq_v;
  float* cs = tp->cs;
  if (!cs) { cs_v.resize((size_t)b_ * H * L); cs = cs_v.data(); }
  int8_t* CBq = tp->CBq;
  if (!CBq) { cbq_v.resize((size_t)b_ * c * G * Q * Q); CBq = cbq_v.data(); }
  float* loc = tp->loc;
  if (!loc) { loc_v.resize(nst); loc = loc_v.data(); }
  float* prev = tp->prev;
  if (!prev) { prev_v.resize(nst); prev = prev_v.data(); }
  int8_t* hq = tp->hq;
  if (!hq) { hq_v.resize(nst); hq = hq_v.data(); }

  orc_chunk_cumsum(d, dt, A, cs);
  orc_chunk_decay(d, cs, gamma.data());
  orc_chunk_bmm(d, Cq, Bq, s_C, s_B, s_cb, tp->acc_cb, CBq);
  if (flags & 2u) {
    std::vector<int32_t> acc_v;
    int32_t* acc = tp->acc_st;
    if (!acc) { acc_v.resize(nst); acc = acc_v.data(); }
    orc_chunk_state(d, xq, Bq, s_x, s_xs, s_B, dt, cs, tp->Xsq, acc, nullptr);
    orc_state_passing_int8(d, acc, gamma.data(), init, s_xs, s_B, s_h, hq, final_state);
  } else {
    orc_chunk_state(d, xq, Bq, s_x, s_xs, s_B, dt, cs, tp->Xsq, tp->acc_st, loc);
    orc_state_passing(d, loc, gamma.data(), init, s_h, prev, final_state, hq);
  }
  orc_chunk_scan(d, xq, Cq, CBq, hq, s_x, s_C, s_cb, s_h, dt, cs, D, corr, tp->acc_off,
                 tp->rowmax, tp->Mq, tp->acc_diag, y, flags, nullptr);
}

// ---------------------------------------------------------------------------
// L3: one recurrent-mode token for every sequence of the batch (the recurrence
// of L0 restated per token on int8 inputs; the paper gives no algorithm for
// it).  state [b,H,P,N] fp64 is updated in place; y uses the UPDATED state.
//   a = exp(dt A_h);  S[p,n] = a S[p,n] + (dt s_x[h,p] s_B[g]) xq[p] Bq[n]
//   y[p] = s_C[g] sum_n Cq[n] S[p,n] + D_h s_x[h,p] xq[p] + corr[h,p]
void orc_ssd_step(const Dims* d, const int8_t* xq, const float* s_x, const int8_t* Bq,
                  const float* s_B, const int8_t* Cq, const float* s_C, const float* dt,
                  const float* A, const float* D, const float* corr, double* state, double* y) {
  const int b_ = d->batch, H = d->nheads, P = d->headdim, N = d->dstate, G = d->ngroups,
            hpg = H / G;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < b_; ++b)
    for (int h = 0; h < H; ++h) {
      const int g = h / hpg;
      const double dtt = dt[(i64)b * H + h];
      const double a = std::exp(dtt * (double)A[h]);
      const int8_t* Bt = Bq + ((i64)b * G + g) * N;
      const int8_t* Ct = Cq + ((i64)b * G + g) * N;
      for (int p = 0; p < P; ++p) {
        const i64 o = ((i64)b * H + h) * P + p;
        const double xv = (double)s_x[h * P + p] * (double)xq[o];
        double* S = state + o * N;
        double acc = 0.0;
        for (int n = 0; n < N; ++n) {
          const double s = a * S[n] + dtt * xv * ((double)s_B[g] * (double)Bt[n]);
          S[n] = s;
          acc += (double)Ct[n] * s;
        }
        double v = (double)s_C[g] * acc;
        if (D) v += (double)D[h] * xv;
        if (corr) v += (double)corr[h * P + p];
        y[o] = v;
      }
    }
}

// ---------------------------------------------------------------------------
// Eq. 8: the least-squares optimal per-channel correction is the mean error,
// c_p = eta * mean_i (Y - Y')_{i,p}.  Y, Yq are [rows][Ch].
void orc_mean_correction(const double* Y, const double* Yq, i64 rows, i64 Ch, double eta,
                         double* c) {
  for (i64 ch = 0; ch < Ch; ++ch) {
    double s = 0.0;
    for (i64 r = 0; r < rows; ++r) s += Y[r * Ch + ch] - Yq[r * Ch + ch];
    c[ch] = eta * s / (double)rows;
  }
}

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
