// Channel-gated convolution layer: slow, plain CPU oracle.
//
// THIS FILE IS TEST INFRASTRUCTURE.  It exists to check the CUDA library and to
// be timed as a CPU baseline.  It shares no code with the CUDA path and the
// product never calls it.
//
// What it computes (Channel Gating Neural Networks, arXiv 1805.12549):
//   * Section 3.1: the input channels are split statically into a base part
//     x_p (the first c_in/G channels) and a conditional part x_r (the rest);
//     W is split the same way, so W*x = W_p*x_p + W_r*x_r.
//   * Eq. 1: per output activation, y = f(W_p*x_p) when the decision d is 0
//     and y = f(W_p*x_p + W_r*x_r) otherwise.
//   * Eq. 2: the Heaviside step theta(v) = 1 when v >= 0 (a tie fires).
//   * Eq. 3 (merged gate): d = theta(P - Delta*sqrt(Var) - E), with one
//     threshold per output channel, P the partial sum W_p*x_p.
//   * Eq. 4 (channel-wise gate, optional): per image, an output channel keeps
//     its conditional path iff the number of its activations that fire is at
//     least tau_c * w' * h'; otherwise all its activations take the first case
//     of Eq. 1.
//   * Section 3.3 (channel grouping, optional): output group i takes input
//     group i as x_p and the other groups as x_r.
//   * Section 4, first paragraph and its footnote: the two paths are
//     normalised by two batch norms BN1 (base result) and BN2 (full result)
//     that share gamma and beta; at inference each is a scale and a shift.
//   * Section 4, "Inducing sparsity": the cost of the base path is
//     eta*c_l*k^2*w'*h'*c_{l+1} multiplications; the conditional path costs the
//     remaining (1-eta)*c_l*k^2 multiplications for every activation that fires.
//
// The layer runs in the three steps of the definition: partial sums and
// activation-wise decisions for every output, then the channel-wise decision,
// then the conditional path and the batch norm of the path taken.
// Everything is a direct convolution written as nested loops over
// (n, h', w', c_out, r, s, c_in) in NHWC order.  No blocking, no im2col,
// no reordering.  Floating-point sums run in fp32 in the order (r, s, c_in)
// with a separate multiply and add (build with -ffp-contract=off), or in
// fp64 when acc_double is set.
//
// Parity pins (tests/test_oracle_pins.py): all-open gate vs a library dense
// convolution, all-shut gate vs a base-only convolution, the tie rule, the
// merged vs unmerged gate, monotonicity in Delta, the Gaussian firing rate,
// the multiplication-count closed form, a hand-computed 3x3 case, an
// exact integer re-computation of the quantised variant, and for Eq. 4 a
// hand-computed two-image case, its limits (tau_c = 0, tau_c > 1), a
// restatement on the unpacked decisions and per-image independence.
// Trained-model behaviour (accuracy, the tables' FLOP reductions, the
// partial/final-sum correlations) is "parity unpinned": it needs data sets and
// trained weights that are not available.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

struct cgo_desc {
  int32_t n, h, w, c_in, c_out;
  int32_t kh, kw, stride, pad;
  int32_t groups;       // G; base channels are [0, c_in/G)
  float bn_eps;         // added inside every sqrt(var + eps)
  int32_t relu;         // 1: f = ReLU, 0: f = identity
  int32_t out_bf16;     // 1: round y to bfloat16 (nearest even) before returning it as fp32
  int32_t acc_double;   // 1: accumulate P and R in fp64 instead of fp32
  int32_t gate_form;    // 0: merged gate of Eq. 3; 1: normalise P first, then compare with Delta
  int32_t grouped;      // 0: Fig. 5(a), base = channels [0,c_in/G); 1: Fig. 5(b), channel grouping
  float channel_tau;    // tau_c of the channel-wise gate (Eq. 4); <= 0: no channel-wise gate
  const float* delta_high;   // [c_out] upper thresholds of the two-sided gate of Section 3.2,
                             // s = theta(Delta_h - x) o theta(x - Delta_l), in normalised units
                             // like Delta; NULL: the one-sided gate theta(x - Delta)
};

struct cgo_counts {
  int64_t outputs;      // n*h'*w'*c_out
  int64_t active;       // activations whose gate fired
  int64_t base_macs;    // multiplications on the base path (padding taps counted)
  int64_t cond_macs;    // multiplications on the conditional path
  int64_t dense_macs;   // multiplications of the ungated layer
  int64_t channels;          // n * c_out output channels (one per image)
  int64_t channels_skipped;  // of those, channels whose conditional path Eq. 4 switched off
};

int cgo_out_dim(int in, int k, int stride, int pad) { return (in + 2 * pad - k) / stride + 1; }

int cgo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// float -> bfloat16 -> float, round to nearest, ties to even.
float cgo_round_bf16(float v) {
  uint32_t u;
  std::memcpy(&u, &v, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) {          // NaN stays NaN
    u = (u | 0x00400000u) & 0xffff0000u;
  } else {
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
  }
  float r;
  std::memcpy(&r, &u, 4);
  return r;
}

// Per-channel constants.  t = Delta*sqrt(var_g+eps) + mean_g (Eq. 3 with the
// usual batch-norm epsilon inside the root); a = gamma/sqrt(var+eps),
// b = beta - a*mean (a batch norm at inference is a scale and a shift).
void cgo_fold_params(const cgo_desc* d, const float* gamma, const float* beta,
                     const float* mean_base, const float* var_base,
                     const float* mean_full, const float* var_full,
                     const float* gate_mean, const float* gate_var, const float* delta,
                     float* t, float* a1, float* b1, float* a2, float* b2) {
  const float* gm = gate_mean ? gate_mean : mean_base;
  const float* gv = gate_var ? gate_var : var_base;
  for (int c = 0; c < d->c_out; ++c) {
    const float sg = std::sqrt(gv[c] + d->bn_eps);
    const float prod = delta[c] * sg;
    t[c] = prod + gm[c];
    const float s1 = std::sqrt(var_base[c] + d->bn_eps);
    a1[c] = gamma[c] / s1;
    const float m1 = a1[c] * mean_base[c];
    b1[c] = beta[c] - m1;
    const float s2 = std::sqrt(var_full[c] + d->bn_eps);
    a2[c] = gamma[c] / s2;
    const float m2 = a2[c] * mean_full[c];
    b2[c] = beta[c] - m2;
  }
}

}  // extern "C"

namespace {

// Sum over the taps (r, s) and the input channels [c_lo, c_hi) of one output
// activation.  Taps that fall in the zero padding contribute nothing.
// Weights are [c_out][kh][kw][c_hi - c_lo].
template <typename Acc>
inline Acc conv_point(const cgo_desc* d, const float* x, const float* w, int n, int ho, int wo,
                      int co, int c_lo, int c_hi) {
  const int cw = c_hi - c_lo;
  Acc acc = 0;
  for (int r = 0; r < d->kh; ++r) {
    const int hi = ho * d->stride + r - d->pad;
    for (int s = 0; s < d->kw; ++s) {
      const int wi = wo * d->stride + s - d->pad;
      if (hi < 0 || hi >= d->h || wi < 0 || wi >= d->w) continue;
      const float* xp = x + (((int64_t)n * d->h + hi) * d->w + wi) * d->c_in + c_lo;
      const float* wp = w + (((int64_t)co * d->kh + r) * d->kw + s) * cw;
      for (int ci = 0; ci < cw; ++ci) {
        const Acc prod = (Acc)xp[ci] * (Acc)wp[ci];
        acc = acc + prod;
      }
    }
  }
  return acc;
}

// Channel grouping (Section 3.3): output group g uses input group g as x_p
// and the other G-1 groups, in ascending order, as x_r.
template <typename Acc>
inline Acc conv_point_grouped(const cgo_desc* d, const float* x, const float* w, int n, int ho,
                              int wo, int co, int group, bool base) {
  const int cp = d->c_in / d->groups;
  const int cw = base ? cp : d->c_in - cp;
  Acc acc = 0;
  for (int r = 0; r < d->kh; ++r) {
    const int hi = ho * d->stride + r - d->pad;
    for (int s = 0; s < d->kw; ++s) {
      const int wi = wo * d->stride + s - d->pad;
      if (hi < 0 || hi >= d->h || wi < 0 || wi >= d->w) continue;
      const float* xp = x + (((int64_t)n * d->h + hi) * d->w + wi) * d->c_in;
      const float* wp = w + (((int64_t)co * d->kh + r) * d->kw + s) * cw;
      if (base) {
        for (int ci = 0; ci < cp; ++ci) {
          const Acc prod = (Acc)xp[group * cp + ci] * (Acc)wp[ci];
          acc = acc + prod;
        }
      } else {
        int j = 0;
        for (int ci = 0; ci < d->c_in; ++ci) {
          if (ci / cp == group) continue;
          const Acc prod = (Acc)xp[ci] * (Acc)wp[j];
          acc = acc + prod;
          ++j;
        }
      }
    }
  }
  return acc;
}

template <typename Acc>
int gated_conv_impl(const cgo_desc* d, const float* x, const float* w_base, const float* w_cond,
                    const float* gamma, const float* beta, const float* mean_base,
                    const float* var_base, const float* mean_full, const float* var_full,
                    const float* gate_mean, const float* gate_var, const float* delta,
                    const float* residual, float* y, uint32_t* mask, float* p_out,
                    cgo_counts* counts) {
  const int cp = d->c_in / d->groups;
  const int cr = d->c_in - cp;
  const int ho_n = cgo_out_dim(d->h, d->kh, d->stride, d->pad);
  const int wo_n = cgo_out_dim(d->w, d->kw, d->stride, d->pad);
  const int words = (d->c_out + 31) / 32;
  const int og = d->grouped ? d->c_out / d->groups : d->c_out;   // output channels per group

  std::vector<float> t(d->c_out), a1(d->c_out), b1(d->c_out), a2(d->c_out), b2(d->c_out);
  cgo_fold_params(d, gamma, beta, mean_base, var_base, mean_full, var_full, gate_mean, gate_var,
                  delta, t.data(), a1.data(), b1.data(), a2.data(), b2.data());
  const float* gm = gate_mean ? gate_mean : mean_base;
  const float* gv = gate_var ? gate_var : var_base;

  // Step 1 -- base path and activation-wise gate of every output (Section 3.1, Eq. 2, Eq. 3).
  const int64_t outputs = (int64_t)d->n * ho_n * wo_n * d->c_out;
  std::vector<Acc> p_all((size_t)outputs);
  std::vector<uint8_t> fire_all((size_t)outputs);
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int n = 0; n < d->n; ++n) {
    for (int ho = 0; ho < ho_n; ++ho) {
      for (int wo = 0; wo < wo_n; ++wo) {
        const int64_t m = ((int64_t)n * ho_n + ho) * wo_n + wo;
        for (int co = 0; co < d->c_out; ++co) {
          // Base path: always computed (Section 3.1).
          const Acc p_acc = d->grouped
              ? conv_point_grouped<Acc>(d, x, w_base, n, ho, wo, co, co / og, true)
              : conv_point<Acc>(d, x, w_base, n, ho, wo, co, 0, cp);
          const float p = (float)p_acc;
          p_all[(size_t)(m * d->c_out + co)] = p_acc;
          if (p_out) p_out[m * d->c_out + co] = p;
          // Gate (Eq. 2, Eq. 3): a tie fires; a NaN partial sum does not.
          bool fire;
          if (d->gate_form == 0) {
            fire = (p >= t[co]);
          } else {
            const float sg = std::sqrt(gv[co] + d->bn_eps);
            const float centred = p - gm[co];
            const float p_hat = centred / sg;
            fire = (p_hat >= delta[co]);
          }
          // Two-sided gate (Section 3.2): the activation must also stay below the upper
          // threshold; theta(0) = 1 on this side too.
          if (d->delta_high) {
            const float sg = std::sqrt(gv[co] + d->bn_eps);
            if (d->gate_form == 0) {
              const float prod = d->delta_high[co] * sg;
              const float t_hi = prod + gm[co];
              fire = fire && (p <= t_hi);
            } else {
              const float centred = p - gm[co];
              const float p_hat = centred / sg;
              fire = fire && (p_hat <= d->delta_high[co]);
            }
          }
          fire_all[(size_t)(m * d->c_out + co)] = fire ? 1 : 0;
        }
      }
    }
  }

  // Step 2 -- channel-wise gate (Eq. 4): output channel i of one image keeps its conditional
  // path iff  sum_{j,k} s(x, Delta)  >=  tau_c * w' * h'  (theta(0) = 1, as for Eq. 2); the sum
  // runs over the positions of that image's feature map.  Both sides are compared in fp32.
  const bool channel_gate = d->channel_tau > 0.f;
  std::vector<uint8_t> chan_on((size_t)d->n * d->c_out, 1);
  int64_t channels_skipped = 0;
  if (channel_gate) {
    const float need = d->channel_tau * (float)(ho_n * wo_n);
    for (int n = 0; n < d->n; ++n) {
      for (int co = 0; co < d->c_out; ++co) {
        int64_t cnt = 0;
        for (int px = 0; px < ho_n * wo_n; ++px)
          cnt += fire_all[(size_t)(((int64_t)n * ho_n * wo_n + px) * d->c_out + co)];
        const bool on = ((float)cnt >= need);
        chan_on[(size_t)n * d->c_out + co] = on ? 1 : 0;
        if (!on) ++channels_skipped;
      }
    }
  }

  // Step 3 -- conditional path where both gates allow it, batch norm of the path taken,
  // activation (Eq. 1, Section 4).
  int64_t active = 0, base_macs = 0, cond_macs = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(+ : active, base_macs, cond_macs)
  for (int n = 0; n < d->n; ++n) {
    for (int ho = 0; ho < ho_n; ++ho) {
      for (int wo = 0; wo < wo_n; ++wo) {
        const int64_t m = ((int64_t)n * ho_n + ho) * wo_n + wo;
        if (mask) for (int q = 0; q < words; ++q) mask[m * words + q] = 0u;
        for (int co = 0; co < d->c_out; ++co) {
          const Acc p_acc = p_all[(size_t)(m * d->c_out + co)];
          const float p = (float)p_acc;
          base_macs += (int64_t)d->kh * d->kw * cp;
          const bool fire = fire_all[(size_t)(m * d->c_out + co)] && chan_on[(size_t)n * d->c_out + co];
          float v;
          if (fire) {
            // Conditional path: only where the gate fires (Eq. 1, second case).
            const Acc r_acc = d->grouped
                ? conv_point_grouped<Acc>(d, x, w_cond, n, ho, wo, co, co / og, false)
                : conv_point<Acc>(d, x, w_cond, n, ho, wo, co, cp, d->c_in);
            cond_macs += (int64_t)d->kh * d->kw * cr;
            active += 1;
            const float full = (float)(p_acc + r_acc);
            const float scaled = a2[co] * full;
            v = scaled + b2[co];
            if (mask) mask[m * words + (co >> 5)] |= (1u << (co & 31));
          } else {
            const float scaled = a1[co] * p;
            v = scaled + b1[co];
          }
          if (residual) v = v + residual[m * d->c_out + co];
          if (d->relu) v = (v > 0.f) ? v : 0.f;   // NaN -> 0
          if (d->out_bf16) v = cgo_round_bf16(v);
          y[m * d->c_out + co] = v;
        }
      }
    }
  }
  if (counts) {
    counts->outputs = (int64_t)d->n * ho_n * wo_n * d->c_out;
    counts->active = active;
    counts->base_macs = base_macs;
    counts->cond_macs = cond_macs;
    counts->dense_macs = counts->outputs * d->kh * d->kw * d->c_in;
    counts->channels = (int64_t)d->n * d->c_out;
    counts->channels_skipped = channels_skipped;
  }
  return 0;
}

bool desc_ok(const cgo_desc* d) {
  if (!d) return false;
  if (d->n < 0 || d->h <= 0 || d->w <= 0 || d->c_in <= 0 || d->c_out <= 0) return false;
  if (d->kh <= 0 || d->kw <= 0 || d->stride <= 0 || d->pad < 0) return false;
  if (d->groups <= 0 || d->c_in % d->groups != 0) return false;
  if (d->grouped && d->c_out % d->groups != 0) return false;
  if (cgo_out_dim(d->h, d->kh, d->stride, d->pad) <= 0) return false;
  if (cgo_out_dim(d->w, d->kw, d->stride, d->pad) <= 0) return false;
  return true;
}

}  // namespace

extern "C" {

// Floating-point layer.  x: [n][h][w][c_in]; w_base: [c_out][kh][kw][c_in/G];
// w_cond: [c_out][kh][kw][c_in - c_in/G]; per-channel vectors have c_out
// entries; gate_mean/gate_var may be NULL (then BN1's statistics are used,
// since both normalise the partial sum); residual may be NULL; y:
// [n][h'][w'][c_out]; mask: one bit per activation, bit (c & 31) of word
// m*ceil(c_out/32) + (c >> 5), may be NULL; p_out (may be NULL) receives the
// partial sums.  For bf16 workloads pass inputs already rounded to bf16.
int cgo_gated_conv(const cgo_desc* d, const float* x, const float* w_base, const float* w_cond,
                   const float* gamma, const float* beta, const float* mean_base,
                   const float* var_base, const float* mean_full, const float* var_full,
                   const float* gate_mean, const float* gate_var, const float* delta,
                   const float* residual, float* y, uint32_t* mask, float* p_out,
                   cgo_counts* counts) {
  if (!desc_ok(d)) return 1;
  if (d->acc_double)
    return gated_conv_impl<double>(d, x, w_base, w_cond, gamma, beta, mean_base, var_base,
                                   mean_full, var_full, gate_mean, gate_var, delta, residual, y,
                                   mask, p_out, counts);
  return gated_conv_impl<float>(d, x, w_base, w_cond, gamma, beta, mean_base, var_base, mean_full,
                                var_full, gate_mean, gate_var, delta, residual, y, mask, p_out,
                                counts);
}

// Quantised layer.  The paper only says "a quantized ResNet-18"; the scheme
// here is a convention of this library: int8 activations and weights, int32
// sums, d = (P >= q_gate_thr[c]); acc = d ? P+R : P;
// z = (int64)acc*q_mul_sel[c] + q_off_sel[c] with sel = full when d else base;
// q = (z + 2^(S-1)) >> S (arithmetic shift); y = clamp(q, lo, 127) with lo = 0
// when relu is set (the clamp is the ReLU) and -128 otherwise.
int cgo_gated_conv_i8(const cgo_desc* d, int32_t shift, const int8_t* x, const int8_t* w_base,
                      const int8_t* w_cond, const int32_t* q_gate_thr, const int32_t* q_mul_base,
                      const int32_t* q_mul_full, const int64_t* q_off_base,
                      const int64_t* q_off_full, int8_t* y, uint32_t* mask, int32_t* p_out,
                      cgo_counts* counts) {
  if (!desc_ok(d) || shift < 1 || shift > 31 || d->grouped) return 1;
  const int cp = d->c_in / d->groups;
  const int cr = d->c_in - cp;
  const int ho_n = cgo_out_dim(d->h, d->kh, d->stride, d->pad);
  const int wo_n = cgo_out_dim(d->w, d->kw, d->stride, d->pad);
  const int words = (d->c_out + 31) / 32;
  int64_t active = 0, base_macs = 0, cond_macs = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(+ : active, base_macs, cond_macs)
  for (int n = 0; n < d->n; ++n) {
    for (int ho = 0; ho < ho_n; ++ho) {
      for (int wo = 0; wo < wo_n; ++wo) {
        const int64_t m = ((int64_t)n * ho_n + ho) * wo_n + wo;
        if (mask) for (int q = 0; q < words; ++q) mask[m * words + q] = 0u;
        for (int co = 0; co < d->c_out; ++co) {
          int32_t p = 0, rsum = 0;
          for (int r = 0; r < d->kh; ++r) {
            const int hi = ho * d->stride + r - d->pad;
            for (int s = 0; s < d->kw; ++s) {
              const int wi = wo * d->stride + s - d->pad;
              if (hi < 0 || hi >= d->h || wi < 0 || wi >= d->w) continue;
              const int8_t* xp = x + (((int64_t)n * d->h + hi) * d->w + wi) * d->c_in;
              const int8_t* wp = w_base + (((int64_t)co * d->kh + r) * d->kw + s) * cp;
              for (int ci = 0; ci < cp; ++ci) p += (int32_t)xp[ci] * (int32_t)wp[ci];
            }
          }
          base_macs += (int64_t)d->kh * d->kw * cp;
          if (p_out) p_out[m * d->c_out + co] = p;
          const bool fire = (p >= q_gate_thr[co]);
          if (fire) {
            for (int r = 0; r < d->kh; ++r) {
              const int hi = ho * d->stride + r - d->pad;
              for (int s = 0; s < d->kw; ++s) {
                const int wi = wo * d->stride + s - d->pad;
                if (hi < 0 || hi >= d->h || wi < 0 || wi >= d->w) continue;
                const int8_t* xp = x + (((int64_t)n * d->h + hi) * d->w + wi) * d->c_in + cp;
                const int8_t* wp = w_cond + (((int64_t)co * d->kh + r) * d->kw + s) * cr;
                for (int ci = 0; ci < cr; ++ci) rsum += (int32_t)xp[ci] * (int32_t)wp[ci];
              }
            }
            cond_macs += (int64_t)d->kh * d->kw * cr;
            active += 1;
            if (mask) mask[m * words + (co >> 5)] |= (1u << (co & 31));
          }
          const int64_t acc = fire ? (int64_t)p + (int64_t)rsum : (int64_t)p;
          const int64_t mul = fire ? q_mul_full[co] : q_mul_base[co];
          const int64_t off = fire ? q_off_full[co] : q_off_base[co];
          const int64_t z = acc * mul + off;
          int64_t q = (z + ((int64_t)1 << (shift - 1))) >> shift;
          const int64_t lo = d->relu ? 0 : -128;
          if (q < lo) q = lo;
          if (q > 127) q = 127;
          y[m * d->c_out + co] = (int8_t)q;
        }
      }
    }
  }
  if (counts) {
    counts->outputs = (int64_t)d->n * ho_n * wo_n * d->c_out;
    counts->active = active;
    counts->base_macs = base_macs;
    counts->cond_macs = cond_macs;
    counts->dense_macs = counts->outputs * d->kh * d->kw * d->c_in;
    counts->channels = (int64_t)d->n * d->c_out;
    counts->channels_skipped = 0;
  }
  return 0;
}

}  // extern "C"
