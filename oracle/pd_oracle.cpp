// CPU oracle for the encoder-layer operator kernels.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain definition of every
// operator, evaluated in double precision on one thread.  It is deliberately
// slow and obvious: no blocking, no SIMD intrinsics, no BLAS, no threads, and
// it shares no code, header, table or constant with the CUDA library.  Only
// the tests, the smoke check and the benchmark's CPU-baseline leg call it; the
// product path never does.
//
// Each operator is written as the loop nest it has in the paper's textual
// representation (Section 2.1 "Representation", Table "Supported
// representation features in PerfDojo": element-wise, broadcast, constant and
// reduction operations over named iteration scopes).  The operators are the
// ones in Table "ML operators optimized using PerfLLM" (softmax, layernorm,
// matmul, bmm, add) composed into a post-LN transformer encoder layer.  The
// paper states its softmax only pictorially (Figure "Softmax kernel
// representations"), so the standard definitions are used:
//
//   softmax    N M  m[i]   = max(m[i], x[i,j])
//              N M  e[i,j] = exp(x[i,j] - m[i])
//              N M  s[i]  += e[i,j]
//              N M  y[i,j] = e[i,j] / s[i]
//   layernorm  N M  mu[i] += x[i,j] / M
//              N M  v[i]  += (x[i,j] - mu[i])^2 / M          (biased variance)
//              N M  y[i,j] = (x[i,j] - mu[i]) / sqrt(v[i] + eps) * g[j] + b[j]
//   rmsnorm    N M  q[i]  += x[i,j]^2 / M;  y[i,j] = x[i,j] / sqrt(q[i] + eps) * g[j]
//   bias_gelu  N M  z = x[i,j] + bias[j]
//                   out[i,j] = 0.5 * z * (1 + erf(z / sqrt(2))) + r[i,j]
//   gemm       M N K  c[m,n] += a[m,k] * b[k,n]
//
// Every function returns 0 on success and a negative number on a bad argument.
// All pointers are host pointers to dense row-major arrays of double.
// Parity pins: see tests/test_oracle_*.py (closed forms, invariants, brute
// force on tiny integer inputs, an independent erf series, torch float64).

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <limits>
#include <vector>

extern "C" {

// Row-wise softmax over the last dimension (operator "softmax", Table "ML
// operators optimized using PerfLLM"; reduction + broadcast + element-wise
// features of Table "Supported representation features").
int oracle_softmax(const double* x, double* y, int64_t rows, int64_t cols) {
  if (!x || !y || rows < 0 || cols <= 0) return -1;
  for (int64_t i = 0; i < rows; ++i) {
    const double* xi = x + i * cols;
    double* yi = y + i * cols;
    double m = -std::numeric_limits<double>::infinity();
    for (int64_t j = 0; j < cols; ++j) m = std::fmax(m, xi[j]);
    double s = 0.0;
    for (int64_t j = 0; j < cols; ++j) {
      yi[j] = std::exp(xi[j] - m);
      s += yi[j];
    }
    for (int64_t j = 0; j < cols; ++j) yi[j] = yi[j] / s;
  }
  return 0;
}

// Layer normalisation over the last dimension with a biased (1/M) variance and
// eps inside the square root (operators "layernorm 1/2" of the same table).
int oracle_layernorm(const double* x, const double* gamma, const double* beta, double* y,
                     int64_t rows, int64_t cols, double eps) {
  if (!x || !gamma || !beta || !y || rows < 0 || cols <= 0) return -1;
  const double M = static_cast<double>(cols);
  for (int64_t i = 0; i < rows; ++i) {
    const double* xi = x + i * cols;
    double* yi = y + i * cols;
    double mu = 0.0;
    for (int64_t j = 0; j < cols; ++j) mu += xi[j] / M;
    double v = 0.0;
    for (int64_t j = 0; j < cols; ++j) v += (xi[j] - mu) * (xi[j] - mu) / M;
    const double denom = std::sqrt(v + eps);
    for (int64_t j = 0; j < cols; ++j) yi[j] = (xi[j] - mu) / denom * gamma[j] + beta[j];
  }
  return 0;
}

// Root-mean-square normalisation over the last dimension (operator "rmsnorm"):
//   N M  q[i]  += x[i,j]^2 / M
//   N M  y[i,j] = x[i,j] / sqrt(q[i] + eps) * g[j]
int oracle_rmsnorm(const double* x, const double* gamma, double* y, int64_t rows, int64_t cols, double eps) {
  if (!x || !gamma || !y || rows < 0 || cols <= 0) return -1;
  const double M = static_cast<double>(cols);
  for (int64_t i = 0; i < rows; ++i) {
    const double* xi = x + i * cols;
    double q = 0.0;
    for (int64_t j = 0; j < cols; ++j) q += xi[j] * xi[j] / M;
    const double denom = std::sqrt(q + eps);
    for (int64_t j = 0; j < cols; ++j) y[i * cols + j] = xi[j] / denom * gamma[j];
  }
  return 0;
}

// Mean over the last dimension (operator "reducemean"):
//   N M  y[i] += x[i,j] / M
int oracle_reducemean(const double* x, double* y, int64_t rows, int64_t cols) {
  if (!x || !y || rows < 0 || cols <= 0) return -1;
  const double M = static_cast<double>(cols);
  for (int64_t i = 0; i < rows; ++i) {
    double acc = 0.0;
    for (int64_t j = 0; j < cols; ++j) acc += x[i * cols + j] / M;
    y[i] = acc;
  }
  return 0;
}

// GELU in its erf form.
static double gelu_erf(double z) { return 0.5 * z * (1.0 + std::erf(z / std::sqrt(2.0))); }

// out = GELU(x + bias) + r, bias broadcast over rows; r may be null (no residual
// term).  Element-wise + broadcast features; the paper's nearest operators are
// "add" and "relu" of Table "ML operators optimized using PerfLLM".
int oracle_bias_gelu_residual(const double* x, const double* bias, const double* r, double* out,
                              int64_t rows, int64_t cols) {
  if (!x || !bias || !out || rows < 0 || cols <= 0) return -1;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const double z = x[i * cols + j] + bias[j];
      const double g = gelu_erf(z);
      out[i * cols + j] = r ? g + r[i * cols + j] : g;
    }
  return 0;
}

// out = ReLU(x + bias) + r, ReLU(z) = max(z, 0) (operator "relu" with the bias
// and residual terms of the fused projection epilogue); bias and r may be null.
int oracle_bias_relu_residual(const double* x, const double* bias, const double* r, double* out,
                              int64_t rows, int64_t cols) {
  if (!x || !out || rows < 0 || cols <= 0) return -1;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const double z = x[i * cols + j] + (bias ? bias[j] : 0.0);
      const double a = z > 0.0 ? z : 0.0;
      out[i * cols + j] = r ? a + r[i * cols + j] : a;
    }
  return 0;
}

// Element-wise part of operator "swiglu": out = SiLU(g) * u, SiLU(g) = g / (1 + exp(-g)).
int oracle_swiglu(const double* g, const double* u, double* out, int64_t n) {
  if (!g || !u || !out || n < 0) return -1;
  for (int64_t i = 0; i < n; ++i) out[i] = g[i] / (1.0 + std::exp(-g[i])) * u[i];
  return 0;
}

// C[M,N] = A[M,K] * B[K,N] (operator "matmul").  The loops run m, k, n so that
// B is walked along its rows; every c[m,n] still receives its K products in
// ascending k, so the result is bit-identical to the M N K nest above.
int oracle_gemm(const double* a, const double* b, double* c, int64_t M, int64_t N, int64_t K) {
  if (!a || !b || !c || M < 0 || N < 0 || K <= 0) return -1;
  for (int64_t m = 0; m < M; ++m) {
    double* cm = c + m * N;
    for (int64_t n = 0; n < N; ++n) cm[n] = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      const double amk = a[m * K + k];
      const double* bk = b + k * N;
      for (int64_t n = 0; n < N; ++n) cm[n] += amk * bk[n];
    }
  }
  return 0;
}

// Multi-head scaled-dot-product attention on a packed projection
// qkv[tokens, 3*hidden] = [Q | K | V], head h in columns h*d .. h*d+d-1 of each
// block, token t = b*seq + s.  For every (batch b, head h):
//   S = Q_bh * K_bh^T / sqrt(d);  P = softmax_rows(S);  Ctx_bh = P * V_bh
// (operator "bmm" twice with "softmax" between).  ctx is [tokens, hidden] with
// the heads written back to their column blocks.  probs, when not null,
// receives P as [batch, heads, seq, seq].
int oracle_attention(const double* qkv, double* ctx, double* probs,
                     int64_t batch, int64_t seq, int64_t heads, int64_t head_dim) {
  if (!qkv || !ctx || batch < 0 || seq <= 0 || heads <= 0 || head_dim <= 0) return -1;
  const int64_t hidden = heads * head_dim, ld = 3 * hidden;
  const double scale = 1.0 / std::sqrt(static_cast<double>(head_dim));
  std::vector<double> s(static_cast<size_t>(seq) * seq), p(static_cast<size_t>(seq) * seq);
  for (int64_t b = 0; b < batch; ++b)
    for (int64_t h = 0; h < heads; ++h) {
      const double* q = qkv + b * seq * ld + h * head_dim;
      const double* k = q + hidden;
      const double* v = q + 2 * hidden;
      for (int64_t i = 0; i < seq; ++i)
        for (int64_t j = 0; j < seq; ++j) {
          double acc = 0.0;
          for (int64_t e = 0; e < head_dim; ++e) acc += q[i * ld + e] * k[j * ld + e];
          s[i * seq + j] = acc * scale;
        }
      oracle_softmax(s.data(), p.data(), seq, seq);
      if (probs)
        for (int64_t i = 0; i < seq * seq; ++i) probs[((b * heads + h) * seq) * seq + i] = p[i];
      for (int64_t i = 0; i < seq; ++i)
        for (int64_t e = 0; e < head_dim; ++e) {
          double acc = 0.0;
          for (int64_t j = 0; j < seq; ++j) acc += p[i * seq + j] * v[j * ld + e];
          ctx[(b * seq + i) * hidden + h * head_dim + e] = acc;
        }
    }
  return 0;
}

// y[rows, cols] = a[rows, cols] + bias[cols] (+ r[rows, cols] when r is not null).
static void add_bias_residual(const double* a, const double* bias, const double* r, double* y,
                              int64_t rows, int64_t cols) {
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j)
      y[i * cols + j] = a[i * cols + j] + bias[j] + (r ? r[i * cols + j] : 0.0);
}

// Forward pass of one post-LN encoder layer, no dropout, no mask:
//   1. QKV = X Wqkv + bqkv
//   2. Ctx = attention(QKV)
//   3. H1  = layernorm(Ctx Wo + bo + X; gamma1, beta1)
//   4. Mid = GELU(H1 W1 + b1)
//   5. Y   = layernorm(Mid W2 + b2 + H1; gamma2, beta2)
// Weight matrices are [in, out] row-major.  No intermediate is rounded.  The
// four optional outputs (qkv_out [T,3H], ctx_out [T,H], h1_out [T,H], mid_out
// [T,F]) receive the intermediates when not null.
int oracle_encoder_layer(int64_t batch, int64_t seq, int64_t hidden, int64_t heads, int64_t ffn,
                         double ln_eps, const double* x,
                         const double* w_qkv, const double* b_qkv, const double* w_o, const double* b_o,
                         const double* w_ffn1, const double* b_ffn1, const double* w_ffn2,
                         const double* b_ffn2, const double* ln1_gamma, const double* ln1_beta,
                         const double* ln2_gamma, const double* ln2_beta, double* y,
                         double* qkv_out, double* ctx_out, double* h1_out, double* mid_out) {
  if (!x || !y || !w_qkv || !b_qkv || !w_o || !b_o || !w_ffn1 || !b_ffn1 || !w_ffn2 || !b_ffn2 ||
      !ln1_gamma || !ln1_beta || !ln2_gamma || !ln2_beta)
    return -1;
  if (batch < 0 || seq <= 0 || hidden <= 0 || heads <= 0 || ffn <= 0 || hidden % heads != 0) return -2;
  const int64_t T = batch * seq, H = hidden, F = ffn;
  std::vector<double> zero_h(static_cast<size_t>(H), 0.0);
  std::vector<double> qkv(static_cast<size_t>(T) * 3 * H), ctx(static_cast<size_t>(T) * H),
      proj(static_cast<size_t>(T) * H), pre(static_cast<size_t>(T) * H), h1(static_cast<size_t>(T) * H),
      up(static_cast<size_t>(T) * F), mid(static_cast<size_t>(T) * F);

  oracle_gemm(x, w_qkv, qkv.data(), T, 3 * H, H);
  add_bias_residual(qkv.data(), b_qkv, nullptr, qkv.data(), T, 3 * H);
  oracle_attention(qkv.data(), ctx.data(), nullptr, batch, seq, heads, H / heads);

  oracle_gemm(ctx.data(), w_o, proj.data(), T, H, H);
  add_bias_residual(proj.data(), b_o, x, pre.data(), T, H);
  oracle_layernorm(pre.data(), ln1_gamma, ln1_beta, h1.data(), T, H, ln_eps);

  oracle_gemm(h1.data(), w_ffn1, up.data(), T, F, H);
  oracle_bias_gelu_residual(up.data(), b_ffn1, nullptr, mid.data(), T, F);

  oracle_gemm(mid.data(), w_ffn2, proj.data(), T, H, F);
  add_bias_residual(proj.data(), b_ffn2, h1.data(), pre.data(), T, H);
  oracle_layernorm(pre.data(), ln2_gamma, ln2_beta, y, T, H, ln_eps);

  if (qkv_out) for (size_t i = 0; i < qkv.size(); ++i) qkv_out[i] = qkv[i];
  if (ctx_out) for (size_t i = 0; i < ctx.size(); ++i) ctx_out[i] = ctx[i];
  if (h1_out) for (size_t i = 0; i < h1.size(); ++i) h1_out[i] = h1[i];
  if (mid_out) for (size_t i = 0; i < mid.size(); ++i) mid_out[i] = mid[i];
  return 0;
}

}  // extern "C"
