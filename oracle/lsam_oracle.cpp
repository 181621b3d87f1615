// lsam_oracle.cpp -- CPU oracle (TEST INFRASTRUCTURE ONLY; see lsam_oracle.h).
//
// Written from the paper's statement of the method:
//   * SAM perturbation  x~ = x + rho * grad f(x; xi) / (||grad f(x; xi)|| + gamma)      (Eq. 3, look-back map)
//   * SAM gradient      g  = grad f(x~; xi), the SAME minibatch xi in both passes        (Theorems 3 and 4)
//   * worker score      G  = g + lambda (x - y)                                          (Algorithm 1, first update)
//                       (other stationary kernels phi(x - y): G = g + grad phi(x - y), Corollary 8 and its remark)
//   * sampler           Nesterov-momentum step on G                                      (Section 4.3)
//   * centre update     g' = (1/(n tau)) sum_i sum_s x_s^(i) - y ;  g = g' + beta (g' - g'_prev) ;
//                       y <- y + eta' g ; counters reset                                 (Algorithm 2, sync branch)
// All arithmetic is double.  Loops are written in the order of the definitions; the only
// parallelism is OpenMP over the independent replicas.
#include "lsam_oracle.h"

#include <cmath>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---- schedule hash: splitmix64 finaliser (Steele, Lea, Flood 2014), chained over (seed^tag, t, k*2^20+j)
inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
  z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
  return z ^ (z >> 31);
}
const uint64_t TAG_IDX = 0x6c73616d5f696478ULL;    // ASCII "lsam_idx"
const uint64_t TAG_STALE = 0x6c73616d5f73746cULL;  // ASCII "lsam_stl"
const uint64_t TAG_ACT = 0x6c73616d5f616374ULL;    // ASCII "lsam_act"
const uint64_t TAG_ORD = 0x6c73616d5f6f7264ULL;    // ASCII "lsam_ord"
inline uint64_t hash5(uint64_t seed, uint64_t tag, uint64_t t, uint64_t k, uint64_t j) {
  return mix64(mix64(mix64(seed ^ tag) + t) + ((k << 20) + j));
}

// ---- Langevin noise: Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC 2011) + Box-Muller.
// One block gives the four normals of one group of four consecutive parameters of a segment (W_l: segment 2l,
// b_l: segment 2l+1; least squares / flat vector: segment 0):
//   counter = (group low 32 bits, segment, worker, tick low 32 bits), key = (seed low ^ "lang", seed high ^ tick high)
//   u = ((r >> 8) + 0.5) 2^-24 from each 32-bit output r (exact in binary32, never 0 or 1)
//   (z0, z1) = sqrt(-2 ln u0) (cos 2 pi u1, sin 2 pi u1), (z2, z3) likewise from (u2, u3)
inline void philox4x32_10(const uint32_t c_in[4], const uint32_t k_in[2], uint32_t out[4]) {
  uint32_t c[4] = {c_in[0], c_in[1], c_in[2], c_in[3]};
  uint32_t k0 = k_in[0], k1 = k_in[1];
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0], p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0, hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c[1] ^ k0, n1 = lo1, n2 = hi0 ^ c[3] ^ k1, n3 = lo0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
  }
  for (int i = 0; i < 4; ++i) out[i] = c[i];
}
inline void noise4(uint64_t seed, uint64_t t, uint64_t k, uint32_t seg, uint64_t group, double z[4]) {
  const uint32_t ctr[4] = {(uint32_t)group, seg, (uint32_t)k, (uint32_t)t};
  const uint32_t key[2] = {(uint32_t)seed ^ 0x6c616e67u, (uint32_t)(seed >> 32) ^ (uint32_t)(t >> 32)};
  uint32_t r[4];
  philox4x32_10(ctr, key, r);
  const double two_pi = 6.283185307179586476925286766559;
  for (int h = 0; h < 2; ++h) {
    const double u0 = ((double)(r[2 * h] >> 8) + 0.5) / 16777216.0, u1 = ((double)(r[2 * h + 1] >> 8) + 0.5) / 16777216.0;
    const double rad = std::sqrt(-2.0 * std::log(u0));
    z[2 * h] = rad * std::cos(two_pi * u1);
    z[2 * h + 1] = rad * std::sin(two_pi * u1);
  }
}

// ---- bf16 round-to-nearest-even of an fp32 value (published format: 1-8-7, top half of binary32)
inline float bf16_round(float v) {
  uint32_t u;
  std::memcpy(&u, &v, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return v;  // inf / nan unchanged
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  float r;
  std::memcpy(&r, &u, 4);
  return r;
}

// ---- stationary kernels k(x, y) = phi(x - y), radial: phi depends on r = ||x - y|| only (Corollary 8 and its remark).
// kernel_phi is the kernel itself, kernel_weight the factor w(r) = phi'(r) / r of its gradient grad phi(z) = w(||z||) z.
//   GAUSSIAN     phi = (lambda / 2) r^2                                   w = lambda          (Algorithm 1)
//   EXP_POWER    phi = (lambda / a) r^a, a = param in [1, 2]              w = lambda r^(a-2)  (w(0) := 0 for a < 2)
//   CAUCHY       phi = (lambda s^2 / 2) log(1 + r^2 / s^2), s = param     w = lambda / (1 + r^2 / s^2)
//   MATERN32     exp(-phi) = (1 + c r) exp(-c r), c = sqrt(lambda)        w = lambda / (1 + c r)
// Every one of them has w -> lambda for r -> 0 (a = 2 / s -> infinity / c r -> 0), the Gaussian pull.
inline double kernel_phi(int kind, double lambda, double param, double r) {
  switch (kind) {
    case ORACLE_KERNEL_EXP_POWER: return lambda / param * std::pow(r, param);
    case ORACLE_KERNEL_CAUCHY: return 0.5 * lambda * param * param * std::log1p(r * r / (param * param));
    case ORACLE_KERNEL_MATERN32: { const double cr = std::sqrt(lambda) * r; return cr - std::log1p(cr); }
    default: return 0.5 * lambda * r * r;
  }
}
inline double kernel_weight(int kind, double lambda, double param, double r) {
  switch (kind) {
    case ORACLE_KERNEL_EXP_POWER: return (param == 2.0) ? lambda : (r > 0.0 ? lambda * std::pow(r, param - 2.0) : 0.0);
    case ORACLE_KERNEL_CAUCHY: return lambda / (1.0 + r * r / (param * param));
    case ORACLE_KERNEL_MATERN32: return lambda / (1.0 + std::sqrt(lambda) * r);
    default: return lambda;
  }
}

struct Layer {
  int in, out;
  int64_t w_off, b_off;  // offsets in the unpadded parameter vector; b_off = -1: no bias
  bool residual;         // h_next = h + relu(W h + b)
  // convolution layer: 3x3, stride 1, zero padding 1, ReLU, then 2x2 max-pooling; in = Cin H W, out = Cout (H/2) (W/2)
  bool conv = false;
  int Cin = 0, Cout = 0, H = 0, W = 0;
};

struct Net {
  int model = 0;
  bool bf16 = false;
  std::vector<Layer> layers;
  int64_t d = 0;
  int in0 = 0;

  double q(double v) const { return bf16 ? (double)bf16_round((float)v) : v; }
};

bool build_net(const oracle_config& c, Net& net) {
  net.model = c.model;
  net.bf16 = (c.gemm_dtype == ORACLE_GEMM_BF16);
  net.layers.clear();
  if (c.K < 1) return false;
  if (c.model == ORACLE_MODEL_FLAT) {
    if (c.flat_d < 1) return false;
    net.d = c.flat_d;
    return true;
  }
  if (c.batch < 1 || c.n_samples < 1) return false;
  if (c.model == ORACLE_MODEL_LSQ) {
    if (c.widths[0] < 1) return false;
    net.in0 = c.widths[0];
    net.layers.push_back({c.widths[0], 1, 0, -1, false});
    net.d = c.widths[0];
    return true;
  }
  if (c.model != ORACLE_MODEL_MLP && c.model != ORACLE_MODEL_RESMLP && c.model != ORACLE_MODEL_CNN) return false;
  if (c.n_layers < 1 || c.n_layers > 8) return false;
  const bool cnn = c.model == ORACLE_MODEL_CNN;
  if (cnn && (c.n_conv < 1 || c.n_conv >= c.n_layers || c.img_h < 1 || c.img_w < 1 || c.img_h % (1 << c.n_conv) || c.img_w % (1 << c.n_conv))) return false;
  int64_t off = 0;
  int H = c.img_h, W = c.img_w;
  for (int l = 0; l < c.n_layers; ++l) {
    Layer L;
    if (c.widths[l] < 1 || c.widths[l + 1] < 1) return false;
    if (cnn && l < c.n_conv) {
      L.conv = true;
      L.Cin = c.widths[l]; L.Cout = c.widths[l + 1]; L.H = H; L.W = W;
      L.in = L.Cin * H * W;
      H /= 2; W /= 2;
      L.out = L.Cout * H * W;
      L.w_off = off;
      off += (int64_t)L.Cout * L.Cin * 9;
      L.b_off = off;
      off += L.Cout;
      L.residual = false;
      net.layers.push_back(L);
      continue;
    }
    L.in = (cnn && l == c.n_conv) ? net.layers.back().out : c.widths[l];  // the first dense layer takes the flattened feature maps
    L.out = c.widths[l + 1];
    L.w_off = off;
    off += (int64_t)L.in * L.out;
    L.b_off = off;
    off += L.out;
    // residual MLP: every hidden layer whose input and output widths agree carries a skip connection
    L.residual = (c.model == ORACLE_MODEL_RESMLP) && (l < c.n_layers - 1) && (L.in == L.out);
    net.layers.push_back(L);
  }
  net.d = off;
  net.in0 = net.layers[0].in;
  return true;
}

// Gradient w.r.t. the pre-activation of a hidden layer from the gradient dh w.r.t. its output: dense layers pass it where the
// ReLU was active; a convolution layer routes each pooled gradient to the element of its 2x2 window that was the maximum,
// if that element's ReLU was active ([B][Cout][H][W] from [B][Cout][H/2][W/2]).
std::vector<double> unpool_or_mask(const Layer& lp, const std::vector<double>& dh, const std::vector<unsigned char>& mask,
                                   const std::vector<unsigned char>& arg, int B) {
  if (!lp.conv) {
    std::vector<double> dz((size_t)B * lp.out);
    for (size_t e = 0; e < dz.size(); ++e) dz[e] = mask[e] ? dh[e] : 0.0;
    return dz;
  }
  const int Hh = lp.H, Ww = lp.W, Ho = Hh / 2, Wo = Ww / 2;
  std::vector<double> dz((size_t)B * lp.Cout * Hh * Ww, 0.0);
  for (int b = 0; b < B; ++b)
    for (int co = 0; co < lp.Cout; ++co)
      for (int y = 0; y < Ho; ++y)
        for (int x = 0; x < Wo; ++x) {
          const size_t e = (size_t)b * lp.out + ((size_t)co * Ho + y) * Wo + x;
          const int a = arg[e];
          const size_t f = (size_t)b * lp.Cout * Hh * Ww + ((size_t)co * Hh + 2 * y + (a >> 1)) * Ww + 2 * x + (a & 1);
          if (mask[f]) dz[f] = dh[e];
        }
  return dz;
}

// Mean loss over the minibatch and its gradient.  a0: [B, in0] inputs (already rounded in bf16 mode).
// If logits_out != nullptr only the forward pass is run and the head outputs are returned.
double net_loss_grad(const Net& net, const double* params, const std::vector<double>& a0, int B,
                     const float* y_f, const int32_t* y_i, const int32_t* idx, double* grad, double* logits_out) {
  const int L = (int)net.layers.size();
  if (net.model == ORACLE_MODEL_LSQ) {
    // f = (1/(2B)) sum_b (a_b . w - y_b)^2 ;  grad = (1/B) sum_b (a_b . w - y_b) a_b
    const int n = net.in0;
    std::vector<double> r(B);
    double loss = 0.0;
    for (int b = 0; b < B; ++b) {
      double p = 0.0;
      for (int i = 0; i < n; ++i) p += a0[(size_t)b * n + i] * params[i];
      if (logits_out) logits_out[b] = p;
      r[b] = logits_out ? 0.0 : p - (double)y_f[idx[b]];
      loss += r[b] * r[b];
    }
    if (logits_out) return 0.0;
    loss /= (2.0 * B);
    for (int i = 0; i < n; ++i) {
      double s = 0.0;
      for (int b = 0; b < B; ++b) s += r[b] * a0[(size_t)b * n + i];
      grad[i] = s / B;
    }
    return loss;
  }

  // operand copy of the parameters (bf16 mode: every weight and bias rounded once; fp32 mode: unchanged)
  std::vector<double> pq((size_t)net.d);
  for (int64_t e = 0; e < net.d; ++e) pq[(size_t)e] = net.q(params[e]);

  // ---- forward
  std::vector<std::vector<double>> h(L + 1);       // h[l]: input of layer l, [B, in_l]
  std::vector<std::vector<unsigned char>> mask(L);  // mask[l][b*out+o] = (pre-activation > 0), hidden layers (convolutions: before pooling)
  std::vector<std::vector<unsigned char>> pool_arg(L);  // convolutions: which element of its 2x2 window each pooled output took
  h[0] = a0;
  std::vector<double> logits;
  for (int l = 0; l < L; ++l) {
    const Layer& ly = net.layers[l];
    const bool head = (l == L - 1);
    if (ly.conv) {
      // z[b][co][y][x] = bias[co] + sum_{ci,kh,kw} W[co][ci*9 + kh*3 + kw] a[b][ci][y+kh-1][x+kw-1]  (zero outside the image);
      // r = relu(z); pooled[b][co][y/2][x/2] = max of the 2x2 window (first maximum in row-major order)
      const int Hh = ly.H, Ww = ly.W, Ho = Hh / 2, Wo = Ww / 2;
      std::vector<double> r((size_t)B * ly.Cout * Hh * Ww);
      mask[l].assign(r.size(), 0);
      for (int b = 0; b < B; ++b)
        for (int co = 0; co < ly.Cout; ++co)
          for (int y = 0; y < Hh; ++y)
            for (int x = 0; x < Ww; ++x) {
              double s = 0.0;
              for (int ci = 0; ci < ly.Cin; ++ci)
                for (int kh = 0; kh < 3; ++kh)
                  for (int kw = 0; kw < 3; ++kw) {
                    const int yy = y + kh - 1, xx = x + kw - 1;
                    if (yy < 0 || yy >= Hh || xx < 0 || xx >= Ww) continue;
                    s += pq[(size_t)(ly.w_off + (int64_t)co * ly.Cin * 9 + ci * 9 + kh * 3 + kw)] *
                         h[l][(size_t)b * ly.in + ((size_t)ci * Hh + yy) * Ww + xx];
                  }
              s += pq[(size_t)(ly.b_off + co)];
              const size_t e = (size_t)b * ly.Cout * Hh * Ww + ((size_t)co * Hh + y) * Ww + x;
              mask[l][e] = s > 0.0;
              // the ReLU output is a stored activation (bf16 mode: rounded), and the pooling compares the stored values: its
              // choice of the maximum is a discrete decision, taken on both sides in the precision the activations are kept in
              r[e] = net.q(s > 0.0 ? s : 0.0);
            }
      h[l + 1].resize((size_t)B * ly.out);
      pool_arg[l].assign((size_t)B * ly.out, 0);
      for (int b = 0; b < B; ++b)
        for (int co = 0; co < ly.Cout; ++co)
          for (int y = 0; y < Ho; ++y)
            for (int x = 0; x < Wo; ++x) {
              double best = -1.0;
              int arg = 0;
              for (int dy = 0; dy < 2; ++dy)
                for (int dx = 0; dx < 2; ++dx) {
                  const double v = r[(size_t)b * ly.Cout * Hh * Ww + ((size_t)co * Hh + 2 * y + dy) * Ww + 2 * x + dx];
                  if (v > best) { best = v; arg = dy * 2 + dx; }
                }
              const size_t e = (size_t)b * ly.out + ((size_t)co * Ho + y) * Wo + x;
              h[l + 1][e] = best;  // the maximum of stored values
              pool_arg[l][e] = (unsigned char)arg;
            }
      continue;
    }
    std::vector<double> z((size_t)B * ly.out);
    for (int b = 0; b < B; ++b)
      for (int o = 0; o < ly.out; ++o) {
        const double* w = pq.data() + ly.w_off + (int64_t)o * ly.in;
        const double* a = h[l].data() + (size_t)b * ly.in;
        double s = 0.0;
        for (int i = 0; i < ly.in; ++i) s += w[i] * a[i];
        z[(size_t)b * ly.out + o] = s + pq[(size_t)(ly.b_off + o)];
      }
    if (head) {
      logits.swap(z);
    } else {
      mask[l].resize((size_t)B * ly.out);
      h[l + 1].resize((size_t)B * ly.out);
      for (size_t e = 0; e < z.size(); ++e) {
        const double r = z[e] > 0.0 ? z[e] : 0.0;
        mask[l][e] = z[e] > 0.0;
        const double skip = ly.residual ? h[l][e] : 0.0;  // in == out for residual layers
        h[l + 1][e] = net.q(skip + r);                     // stored activation (bf16 mode: rounded)
      }
    }
  }
  const int C = net.layers[L - 1].out;
  if (logits_out) {
    std::memcpy(logits_out, logits.data(), sizeof(double) * (size_t)B * C);
    return 0.0;
  }

  // ---- softmax cross-entropy, mean over the batch
  double loss = 0.0;
  std::vector<double> dz((size_t)B * C);
  for (int b = 0; b < B; ++b) {
    const double* lg = logits.data() + (size_t)b * C;
    double m = lg[0];
    for (int c = 1; c < C; ++c) m = lg[c] > m ? lg[c] : m;
    double se = 0.0;
    for (int c = 0; c < C; ++c) se += std::exp(lg[c] - m);
    const int y = y_i[idx[b]];
    loss += (m + std::log(se)) - lg[y];
    for (int c = 0; c < C; ++c) {
      const double p = std::exp(lg[c] - m) / se;
      dz[(size_t)b * C + c] = net.q((p - (c == y ? 1.0 : 0.0)) / B);
    }
  }
  loss /= B;

  // ---- backward: dz = gradient w.r.t. the pre-activation of layer l; dh = gradient w.r.t. its input
  std::vector<double> dh_next;  // gradient w.r.t. h[l+1] (needed by residual layers)
  for (int l = L - 1; l >= 0; --l) {
    const Layer& ly = net.layers[l];
    if (ly.conv) {
      // dz here: gradient w.r.t. the convolution's pre-activation, [B][Cout][H][W]
      const int Hh = ly.H, Ww = ly.W;
      const size_t plane = (size_t)Hh * Ww;
      for (int co = 0; co < ly.Cout; ++co) {
        double sb = 0.0;
        for (int b = 0; b < B; ++b)
          for (size_t e = 0; e < plane; ++e) sb += dz[((size_t)b * ly.Cout + co) * plane + e];
        grad[ly.b_off + co] = sb;
        for (int ci = 0; ci < ly.Cin; ++ci)
          for (int kh = 0; kh < 3; ++kh)
            for (int kw = 0; kw < 3; ++kw) {
              double s = 0.0;  // samples, then rows, then columns, ascending
              for (int b = 0; b < B; ++b)
                for (int y = 0; y < Hh; ++y) {
                  const int yy = y + kh - 1;
                  if (yy < 0 || yy >= Hh) continue;
                  for (int x = 0; x < Ww; ++x) {
                    const int xx = x + kw - 1;
                    if (xx < 0 || xx >= Ww) continue;
                    s += dz[((size_t)b * ly.Cout + co) * plane + (size_t)y * Ww + x] * h[l][(size_t)b * ly.in + ((size_t)ci * Hh + yy) * Ww + xx];
                  }
                }
              grad[ly.w_off + (int64_t)co * ly.Cin * 9 + ci * 9 + kh * 3 + kw] = s;
            }
      }
      if (l == 0) break;
      // gradient w.r.t. the layer's input: dh[b][ci][yy][xx] = sum_{co,kh,kw} dz[b][co][yy-kh+1][xx-kw+1] W[co][ci*9+kh*3+kw]
      std::vector<double> dh((size_t)B * ly.in, 0.0);
      for (int b = 0; b < B; ++b)
        for (int ci = 0; ci < ly.Cin; ++ci)
          for (int yy = 0; yy < Hh; ++yy)
            for (int xx = 0; xx < Ww; ++xx) {
              double s = 0.0;
              for (int co = 0; co < ly.Cout; ++co)
                for (int kh = 0; kh < 3; ++kh)
                  for (int kw = 0; kw < 3; ++kw) {
                    const int y = yy - kh + 1, x = xx - kw + 1;
                    if (y < 0 || y >= Hh || x < 0 || x >= Ww) continue;
                    s += dz[((size_t)b * ly.Cout + co) * plane + (size_t)y * Ww + x] * pq[(size_t)(ly.w_off + (int64_t)co * ly.Cin * 9 + ci * 9 + kh * 3 + kw)];
                  }
              dh[(size_t)b * ly.in + ((size_t)ci * Hh + yy) * Ww + xx] = net.q(s);
            }
      dz = unpool_or_mask(net.layers[l - 1], dh, mask[l - 1], pool_arg[l - 1], B);
      dh_next.swap(dh);
      continue;
    }
    for (int o = 0; o < ly.out; ++o) {
      double sb = 0.0;
      for (int b = 0; b < B; ++b) sb += dz[(size_t)b * ly.out + o];
      grad[ly.b_off + o] = sb;
      // dW[o][i] = sum_b dz[b][o] h[b][i], samples added in ascending order
      double* gw = grad + ly.w_off + (int64_t)o * ly.in;
      for (int i = 0; i < ly.in; ++i) gw[i] = 0.0;
      for (int b = 0; b < B; ++b) {
        const double dzbo = dz[(size_t)b * ly.out + o];
        const double* a = h[l].data() + (size_t)b * ly.in;
        for (int i = 0; i < ly.in; ++i) gw[i] += dzbo * a[i];
      }
    }
    if (l == 0) break;
    std::vector<double> dh((size_t)B * ly.in);
    for (int b = 0; b < B; ++b) {
      // dh[b][i] = sum_o dz[b][o] W[o][i]  (+ the skip path of a residual layer), output units in ascending order
      double* dhb = dh.data() + (size_t)b * ly.in;
      for (int i = 0; i < ly.in; ++i) dhb[i] = 0.0;
      for (int o = 0; o < ly.out; ++o) {
        const double dzbo = dz[(size_t)b * ly.out + o];
        const double* w = pq.data() + ly.w_off + (int64_t)o * ly.in;
        for (int i = 0; i < ly.in; ++i) dhb[i] += dzbo * w[i];
      }
      for (int i = 0; i < ly.in; ++i) {
        const double skip = ly.residual ? dh_next[(size_t)b * ly.in + i] : 0.0;
        dhb[i] = net.q(dhb[i] + skip);
      }
    }
    // pre-activation gradient of layer l-1 (always a hidden layer here)
    dz = unpool_or_mask(net.layers[l - 1], dh, mask[l - 1], pool_arg[l - 1], B);
    dh_next.swap(dh);
  }
  return loss;
}

void gather_inputs(const Net& net, const float* X, const int32_t* idx, int B, std::vector<double>& a0) {
  const int n = net.in0;
  a0.resize((size_t)B * n);
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < n; ++i) a0[(size_t)b * n + i] = net.q((double)X[(int64_t)idx[b] * n + i]);
}

}  // namespace

struct oracle_ctx {
  oracle_config cfg;
  Net net;
  const float* X = nullptr;
  const float* Yf = nullptr;
  const int32_t* Yi = nullptr;
  std::vector<int32_t> rid;
  int64_t d = 0;
  std::vector<double> x, v, acc, g1, g2, xp;  // [K, d]
  std::vector<std::vector<double>> y_hist;    // centre versions; y_hist[t_y] is current
  std::vector<double> gprev;
  bool have_prev = false;
  int64_t t = 0, t_y = 0;
  std::vector<int64_t> t_x;
  std::vector<int64_t> ver_at_step;  // ver_at_step[s] = centre version that was current when step s started
  std::vector<double> loss, gn1, gn2, pullw;
  std::vector<int32_t> active;       // which workers stepped at the last tick
  const float* eg1 = nullptr;
  const float* eg2 = nullptr;
};

extern "C" {

void oracle_philox4x32_10(const uint32_t* counter, const uint32_t* key, uint32_t* out) { philox4x32_10(counter, key, out); }
void oracle_noise4(uint64_t seed, uint64_t t, uint64_t k, uint32_t seg, uint64_t group, double* out) { noise4(seed, t, k, seg, group, out); }
uint64_t oracle_mix64(uint64_t z) { return mix64(z); }
uint64_t oracle_hash(uint64_t seed, uint64_t tag, uint64_t t, uint64_t k, uint64_t j) { return hash5(seed, tag, t, k, j); }
uint64_t oracle_tag_idx(void) { return TAG_IDX; }
uint64_t oracle_tag_stale(void) { return TAG_STALE; }
uint64_t oracle_tag_active(void) { return TAG_ACT; }
uint64_t oracle_tag_order(void) { return TAG_ORD; }
float oracle_bf16_round(float v) { return bf16_round(v); }
int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int64_t oracle_param_count(const oracle_config* cfg) {
  Net net;
  if (!cfg || !build_net(*cfg, net)) return -1;
  return net.d;
}

oracle_ctx* oracle_create(const oracle_config* cfg, const float* X, const void* Y, const double* x0,
                          const double* y0, const int32_t* replica_ids) {
  if (!cfg || !x0 || !y0) return nullptr;
  oracle_ctx* o = new oracle_ctx();
  o->cfg = *cfg;
  const bool kernel_ok = cfg->kernel_kind == ORACLE_KERNEL_GAUSSIAN ||
                         (cfg->kernel_kind == ORACLE_KERNEL_EXP_POWER && cfg->kernel_param >= 1.0 && cfg->kernel_param <= 2.0) ||
                         (cfg->kernel_kind == ORACLE_KERNEL_CAUCHY && cfg->kernel_param > 0.0) || cfg->kernel_kind == ORACLE_KERNEL_MATERN32;
  const bool dp_ok = !cfg->dp_average || cfg->active_num <= 0 || cfg->active_num >= 256;  // synchronous by definition
  if (!build_net(*cfg, o->net) || cfg->tau < 1 || cfg->stale_max < 0 || !kernel_ok || !dp_ok) {
    delete o;
    return nullptr;
  }
  if (cfg->model != ORACLE_MODEL_FLAT && (!X || !Y)) {
    delete o;
    return nullptr;
  }
  o->X = X;
  if (cfg->model == ORACLE_MODEL_LSQ) o->Yf = (const float*)Y;
  else o->Yi = (const int32_t*)Y;
  const int K = cfg->K;
  o->d = o->net.d;
  const size_t n = (size_t)K * o->d;
  o->rid.resize(K);
  for (int k = 0; k < K; ++k) o->rid[k] = replica_ids ? replica_ids[k] : k;
  o->x.assign(x0, x0 + n);
  o->v.assign(n, 0.0);
  o->acc.assign(n, 0.0);
  o->g1.assign(n, 0.0);
  o->g2.assign(n, 0.0);
  o->xp.assign(n, 0.0);
  o->y_hist.emplace_back(y0, y0 + o->d);
  o->gprev.assign(o->d, 0.0);
  o->t_x.assign(K, 0);
  o->loss.assign(K, 0.0);
  o->gn1.assign(K, 0.0);
  o->gn2.assign(K, 0.0);
  o->pullw.assign(K, 0.0);
  o->active.assign(K, 1);
  return o;
}

void oracle_destroy(oracle_ctx* o) { delete o; }

static void schedule_of(const oracle_ctx* o, int64_t t, int k, int32_t* idx, int32_t* stale, int32_t* ver) {
  const oracle_config& c = o->cfg;
  const uint64_t kid = (uint64_t)o->rid[k];
  if (idx && c.model != ORACLE_MODEL_FLAT)
    for (int j = 0; j < c.batch; ++j)
      idx[j] = (int32_t)(hash5(c.seed, TAG_IDX, (uint64_t)t, kid, (uint64_t)j) % (uint64_t)c.n_samples);
  const int64_t s = (int64_t)(hash5(c.seed, TAG_STALE, (uint64_t)t, kid, 0) % (uint64_t)(c.stale_max + 1));
  if (stale) *stale = (int32_t)s;
  if (ver) {
    const int64_t ts = t - s > 0 ? t - s : 0;
    *ver = (ts < (int64_t)o->ver_at_step.size()) ? (int32_t)o->ver_at_step[ts] : -1;
  }
}

int oracle_step(oracle_ctx* o, double eta, double rho) {
  if (!o) return 1;
  const oracle_config& c = o->cfg;
  const int K = c.K;
  const int64_t d = o->d;
  if (c.model == ORACLE_MODEL_FLAT && (!o->eg1 || !o->eg2)) return 2;
  o->ver_at_step.push_back(o->t_y);  // centre version current when this tick starts
  const int64_t t = o->t;
  // Asynchronous progress (Algorithm 2: each worker advances its own counter; the sync fires when the total count of
  // iterations reaches n tau).  A worker is ready at this tick with probability active_num/256; ready workers are served
  // in the order of a seeded key, and only as many as are still missing to n tau: the others wait, like the workers that
  // block on the shared request queue while the servers run the distributed step.
  {
    int64_t done = 0;
    for (int64_t c_ : o->t_x) done += c_;
    const int64_t budget = (int64_t)K * c.tau - done;
    if (budget <= 0) {  // the sync is due: every worker waits until oracle_couple() has run
      o->ver_at_step.pop_back();
      return 4;
    }
    const bool always = (c.active_num <= 0 || c.active_num >= 256);
    std::vector<int> ready(K);
    std::vector<uint64_t> key(K);
    for (int k = 0; k < K; ++k) {
      const uint64_t kid = (uint64_t)o->rid[k];
      ready[k] = always || (hash5(c.seed, TAG_ACT, (uint64_t)t, kid, 0) % 256ULL) < (uint64_t)c.active_num;
      key[k] = hash5(c.seed, TAG_ORD, (uint64_t)t, kid, 0);
    }
    for (int k = 0; k < K; ++k) {
      int64_t rank = 0;  // ready workers served before worker k
      for (int j = 0; j < K; ++j)
        if (ready[j] && (key[j] < key[k] || (key[j] == key[k] && j < k))) rank += 1;
      o->active[k] = (ready[k] && rank < budget) ? 1 : 0;
    }
  }
  // ---- ascent gradient g1_k = grad of the minibatch loss at x_k (workers are independent: OpenMP over them only)
  std::vector<std::vector<int32_t>> idx_of(K);
  std::vector<std::vector<double>> a0_of(K);
  std::vector<int32_t> ver_of(K, 0);
#pragma omp parallel for schedule(dynamic, 1)
  for (int k = 0; k < K; ++k) {
    if (!o->active[k]) continue;
    double* g1 = o->g1.data() + (size_t)k * d;
    idx_of[k].resize(c.model == ORACLE_MODEL_FLAT ? 0 : c.batch);
    int32_t s;
    schedule_of(o, t, k, idx_of[k].data(), &s, &ver_of[k]);
    if (c.model == ORACLE_MODEL_FLAT) {
      for (int64_t j = 0; j < d; ++j) g1[j] = (double)o->eg1[(size_t)k * d + j];
      o->loss[k] = 0.0;
    } else {
      gather_inputs(o->net, o->X, idx_of[k].data(), c.batch, a0_of[k]);
      o->loss[k] = net_loss_grad(o->net, o->x.data() + (size_t)k * d, a0_of[k], c.batch, o->Yf, o->Yi, idx_of[k].data(), g1, nullptr);
    }
  }
  // Synchronous data parallelism (the DP-SGD / DP-SAM baselines of Section 5.2: the workers' gradients are aggregated at
  // every iteration): every worker continues with the mean over the workers, k ascending, of this pass's gradients.
  auto average_over_workers = [&](std::vector<double>& g) {
    std::vector<double> mean((size_t)d, 0.0);
    for (int k = 0; k < K; ++k)
      for (int64_t j = 0; j < d; ++j) mean[(size_t)j] += g[(size_t)k * d + j];
    for (int64_t j = 0; j < d; ++j) mean[(size_t)j] /= (double)K;
    for (int k = 0; k < K; ++k)
      for (int64_t j = 0; j < d; ++j) g[(size_t)k * d + j] = mean[(size_t)j];
  };
  if (c.dp_average) average_over_workers(o->g1);
  // ---- look-back map and descent gradient
#pragma omp parallel for schedule(dynamic, 1)
  for (int k = 0; k < K; ++k) {
    if (!o->active[k]) continue;
    const double* x = o->x.data() + (size_t)k * d;
    const double* g1 = o->g1.data() + (size_t)k * d;
    double* g2 = o->g2.data() + (size_t)k * d;
    double* xp = o->xp.data() + (size_t)k * d;
    double ss = 0.0;
    for (int64_t j = 0; j < d; ++j) ss += g1[j] * g1[j];
    const double n1 = std::sqrt(ss);
    o->gn1[k] = n1;
    // look-back map: x~ = x + rho g1 / (||g1|| + gamma)   (Eq. 3 knows one gradient: no rounding in any mode)
    for (int64_t j = 0; j < d; ++j) xp[j] = x[j] + rho * g1[j] / (n1 + c.gamma);
    // descent gradient at x~ on the same minibatch
    if (c.model == ORACLE_MODEL_FLAT) {
      for (int64_t j = 0; j < d; ++j) g2[j] = (double)o->eg2[(size_t)k * d + j];
    } else {
      net_loss_grad(o->net, xp, a0_of[k], c.batch, o->Yf, o->Yi, idx_of[k].data(), g2, nullptr);
    }
  }
  if (c.dp_average) average_over_workers(o->g2);
  // ---- sampler
#pragma omp parallel for schedule(dynamic, 1)
  for (int k = 0; k < K; ++k) {
    if (!o->active[k]) continue;
    double* x = o->x.data() + (size_t)k * d;
    double* v = o->v.data() + (size_t)k * d;
    double* acc = o->acc.data() + (size_t)k * d;
    const double* g2 = o->g2.data() + (size_t)k * d;
    const double* yk = o->y_hist[ver_of[k]].data();  // possibly stale centre seen by this worker
    double ss2 = 0.0;
    for (int64_t j = 0; j < d; ++j) ss2 += g2[j] * g2[j];
    o->gn2[k] = std::sqrt(ss2);
    // pull of the stationary kernel k(x, y) = phi(x - y) (Corollary 8 and the remark after it): grad_x phi = w(r) (x - y)
    // with r = ||x - y||; the Gaussian kernel of Algorithm 1 has the constant weight lambda
    double r2 = 0.0;
    for (int64_t j = 0; j < d; ++j) r2 += (x[j] - yk[j]) * (x[j] - yk[j]);
    const double wk = kernel_weight(c.kernel_kind, c.lambda, c.kernel_param, std::sqrt(r2));
    o->pullw[k] = wk;
    // momentum step on G = g2 + grad_x phi(x - y); the pull is evaluated at x_k, not at x~
    for (int64_t j = 0; j < d; ++j) {
      const double G = g2[j] + wk * (x[j] - yk[j]);  // Algorithm 1, first update: the gradient as computed
      v[j] = c.mu * v[j] + G;
      x[j] = c.nesterov ? x[j] - eta * (G + c.mu * v[j]) : x[j] - eta * v[j];
    }
    if (c.noise_temp > 0.0) {
      // Langevin sampler: x <- x + sqrt(2 eta T) xi, xi ~ N(0, I) (Section 4.1; comment of Algorithm 1)
      const double sigma = std::sqrt(2.0 * eta * c.noise_temp);
      auto add_noise = [&](uint32_t seg, int64_t off, int64_t len) {
        for (int64_t e = 0; e < len; e += 4) {
          double z[4];
          noise4(c.seed, (uint64_t)t, (uint64_t)o->rid[k], seg, (uint64_t)(e / 4), z);
          for (int i = 0; i < 4 && e + i < len; ++i) x[off + e + i] += sigma * z[i];
        }
      };
      if (o->net.layers.empty() || c.model == ORACLE_MODEL_LSQ) {
        add_noise(0, 0, d);
      } else {
        for (size_t l = 0; l < o->net.layers.size(); ++l) {
          const Layer& ly = o->net.layers[l];
          add_noise((uint32_t)(2 * l), ly.w_off, (int64_t)ly.in * ly.out);
          add_noise((uint32_t)(2 * l + 1), ly.b_off, ly.out);
        }
      }
    }
    for (int64_t j = 0; j < d; ++j) acc[j] += x[j];  // running sum of post-update iterates since the last sync
    o->t_x[k] += 1;
  }
  o->t += 1;
  return 0;
}

int oracle_should_couple(const oracle_ctx* o) {
  if (!o) return 0;
  int64_t s = 0;
  for (int64_t c : o->t_x) s += c;
  return (s > 0 && s % ((int64_t)o->cfg.K * o->cfg.tau) == 0) ? 1 : 0;
}

int oracle_couple(oracle_ctx* o) { return o ? oracle_couple_sharded(o, o->cfg.K, nullptr) : 1; }

// Sync branch of Algorithm 2 when the n workers of the job are spread over several contexts: the sum of iterates runs over
// ALL workers (total_acc, the element-wise sum of every context's accumulators; NULL = the workers held here are all
// there are) and the divisor is n tau.
int oracle_couple_sharded(oracle_ctx* o, int32_t n_total, const double* total_acc) {
  if (!o || n_total < o->cfg.K) return 1;
  if (!oracle_should_couple(o)) return 3;
  const oracle_config& c = o->cfg;
  const int64_t d = o->d;
  const std::vector<double>& y = o->y_hist.back();
  std::vector<double> yn(d);
  const double ntau = (double)n_total * (double)c.tau;
  for (int64_t j = 0; j < d; ++j) {
    double s = 0.0;
    if (total_acc) s = total_acc[j];
    else for (int k = 0; k < c.K; ++k) s += o->acc[(size_t)k * d + j];
    const double gp = s / ntau - y[j];                                        // g'
    const double g = o->have_prev ? gp + c.beta * (gp - o->gprev[j]) : gp;    // look-ahead direction
    yn[j] = y[j] + c.eta_prime * g;                                           // ascent on log pi_LSAM
    o->gprev[j] = gp;
  }
  o->y_hist.push_back(std::move(yn));
  o->have_prev = true;
  std::fill(o->acc.begin(), o->acc.end(), 0.0);
  std::fill(o->t_x.begin(), o->t_x.end(), 0);
  o->t_y += 1;
  return 0;
}

int oracle_read_params(const oracle_ctx* o, int which, double* dst) {
  if (!o || !dst || which < -1 || which >= o->cfg.K) return 1;
  const double* src = which < 0 ? o->y_hist.back().data() : o->x.data() + (size_t)which * o->d;
  std::memcpy(dst, src, sizeof(double) * (size_t)o->d);
  return 0;
}

int oracle_read_state(const oracle_ctx* o, double* x, double* v, double* y, double* acc, double* gprev) {
  if (!o) return 1;
  const size_t n = (size_t)o->cfg.K * o->d;
  if (x) std::memcpy(x, o->x.data(), sizeof(double) * n);
  if (v) std::memcpy(v, o->v.data(), sizeof(double) * n);
  if (acc) std::memcpy(acc, o->acc.data(), sizeof(double) * n);
  if (y) std::memcpy(y, o->y_hist.back().data(), sizeof(double) * (size_t)o->d);
  if (gprev) std::memcpy(gprev, o->gprev.data(), sizeof(double) * (size_t)o->d);
  return 0;
}

int oracle_write_state(oracle_ctx* o, const double* x, const double* v, const double* y) {
  if (!o) return 1;
  const size_t n = (size_t)o->cfg.K * o->d;
  if (x) o->x.assign(x, x + n);
  if (v) o->v.assign(v, v + n);
  if (y) o->y_hist.back().assign(y, y + o->d);
  return 0;
}

int oracle_read_schedule(const oracle_ctx* o, int64_t t, int32_t* idx, int32_t* stale, int32_t* ver) {
  if (!o || t < 0) return 1;
  for (int k = 0; k < o->cfg.K; ++k)
    schedule_of(o, t, k, idx ? idx + (size_t)k * o->cfg.batch : nullptr, stale ? stale + k : nullptr,
                ver ? ver + k : nullptr);
  return 0;
}

int oracle_read_step_info(const oracle_ctx* o, double* loss, double* gnorm1, double* gnorm2) {
  if (!o) return 1;
  const size_t n = sizeof(double) * (size_t)o->cfg.K;
  if (loss) std::memcpy(loss, o->loss.data(), n);
  if (gnorm1) std::memcpy(gnorm1, o->gn1.data(), n);
  if (gnorm2) std::memcpy(gnorm2, o->gn2.data(), n);
  return 0;
}

int oracle_read_grads(const oracle_ctx* o, double* g1, double* g2, double* x_pert) {
  if (!o) return 1;
  const size_t n = sizeof(double) * (size_t)o->cfg.K * o->d;
  if (g1) std::memcpy(g1, o->g1.data(), n);
  if (g2) std::memcpy(g2, o->g2.data(), n);
  if (x_pert) std::memcpy(x_pert, o->xp.data(), n);
  return 0;
}

int oracle_set_external_grads(oracle_ctx* o, const float* g1, const float* g2) {
  if (!o || o->cfg.model != ORACLE_MODEL_FLAT) return 1;
  o->eg1 = g1;
  o->eg2 = g2;
  return 0;
}

double oracle_kernel_phi(int32_t kind, double lambda, double param, double r) { return kernel_phi(kind, lambda, param, r); }
double oracle_kernel_weight(int32_t kind, double lambda, double param, double r) { return kernel_weight(kind, lambda, param, r); }
int oracle_read_pull_weights(const oracle_ctx* o, double* w) {
  if (!o || !w) return 1;
  std::memcpy(w, o->pullw.data(), sizeof(double) * (size_t)o->cfg.K);
  return 0;
}

int oracle_read_active(const oracle_ctx* o, int32_t* active) {
  if (!o || !active) return 1;
  std::memcpy(active, o->active.data(), sizeof(int32_t) * (size_t)o->cfg.K);
  return 0;
}

int oracle_read_counters(const oracle_ctx* o, int64_t* t, int64_t* t_y, int64_t* t_x) {
  if (!o) return 1;
  if (t) *t = o->t;
  if (t_y) *t_y = o->t_y;
  if (t_x) std::memcpy(t_x, o->t_x.data(), sizeof(int64_t) * (size_t)o->cfg.K);
  return 0;
}

int oracle_loss_grad(const oracle_config* cfg, const float* X, const void* Y, const double* params,
                     const int32_t* idx, int32_t n_idx, double* loss, double* grad) {
  Net net;
  if (!cfg || !build_net(*cfg, net) || cfg->model == ORACLE_MODEL_FLAT) return 1;
  std::vector<double> a0;
  gather_inputs(net, X, idx, n_idx, a0);
  const float* yf = cfg->model == ORACLE_MODEL_LSQ ? (const float*)Y : nullptr;
  const int32_t* yi = cfg->model == ORACLE_MODEL_LSQ ? nullptr : (const int32_t*)Y;
  const double l = net_loss_grad(net, params, a0, n_idx, yf, yi, idx, grad, nullptr);
  if (loss) *loss = l;
  return 0;
}

int oracle_forward(const oracle_config* cfg, const float* X, const double* params, const int32_t* idx,
                   int32_t n_idx, double* out) {
  Net net;
  if (!cfg || !build_net(*cfg, net) || cfg->model == ORACLE_MODEL_FLAT || !out) return 1;
  std::vector<double> a0;
  gather_inputs(net, X, idx, n_idx, a0);
  std::vector<double> dummy;
  net_loss_grad(net, params, a0, n_idx, nullptr, nullptr, idx, nullptr, out);
  return 0;
}

}  // extern "C"
