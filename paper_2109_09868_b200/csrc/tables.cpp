// Host-side node tables (see tables.h).
#include "tables.h"

#include <cmath>
#include <cstring>
#include <map>
#include <memory>
#include <mutex>

namespace approxifer {

namespace {

const long double kPi = 3.14159265358979323846264338327950288L;

// sin(pi * p / den) for integers |p| <= den, den > 0.  The argument is folded
// into [0, 1/4] in integer arithmetic first, so the only rounding is that of
// one division and one sin/cos of a small argument.
long double sinpi_ratio(long long p, long long den) {
  if (p < 0) return -sinpi_ratio(-p, den);
  if (2 * p > den) p = den - p;  // sin(pi x) = sin(pi (1 - x))
  if (4 * p > den)               // sin(pi x) = cos(pi (1/2 - x))
    return cosl(kPi * (long double)(den - 2 * p) / (long double)(2 * den));
  return sinl(kPi * (long double)p / (long double)den);
}

}  // namespace

long double node_gap(int K, int W, int j, int i) {
  // a = pi (2j+1)/(2K), b = pi i/(W-1):
  //   (a+b)/2 = pi [(2j+1)(W-1) + 2Ki] / (4K(W-1)),  (a-b)/2 likewise with a minus.
  const long long den = 4LL * K * (W - 1);
  const long long s = (long long)(2 * j + 1) * (W - 1);
  const long long t = 2LL * K * i;
  return -2.0L * sinpi_ratio(s + t, den) * sinpi_ratio(s - t, den);
}

void build_encode_tables(int K, int W, EncodeTables* t) {
  std::memset(t, 0, sizeof(*t));
  for (int i = 0; i < W; ++i) {
    int hit = -1;
    for (int j = 0; j < K; ++j)
      if (nodes_coincide(K, W, j, i)) hit = j;
    if (hit >= 0) {  // u passes through the query: the row is one-hot
      t->w[i * K + hit] = 1.0f;
      continue;
    }
    // l_j(beta_i) = [(-1)^j/(beta_i - alpha_j)] / sum_k (-1)^k/(beta_i - alpha_k)
    long double term[kMaxK], den = 0.0L;
    for (int j = 0; j < K; ++j) {
      term[j] = ((j & 1) ? -1.0L : 1.0L) / (-node_gap(K, W, j, i));
      den += term[j];
    }
    for (int j = 0; j < K; ++j) t->w[i * K + j] = (float)(term[j] / den);
  }
}

void build_decode_tables(int K, int W, DecodeTables* t) {
  std::memset(t, 0, sizeof(*t));
  for (int j = 0; j < K; ++j) t->coin[j] = -1;
  for (int i = 0; i < W; ++i)
    for (int j = 0; j < K; ++j) {
      if (nodes_coincide(K, W, j, i)) {
        t->coin[j] = (int8_t)i;
        t->any_coin = 1;
        t->rg[i * K + j] = 0.0f;
      } else {
        t->rg[i * K + j] = (float)(1.0L / node_gap(K, W, j, i));
      }
    }
}

void build_locate_tables(int K, int W, LocateTables* t) {
  std::memset(t, 0, sizeof(*t));
  // beta_i = cos(pi i/(W-1)) = sin(pi (1/2 - i/(W-1)))
  for (int i = 0; i < W; ++i) t->beta[i] = (double)sinpi_ratio((long long)(W - 1) - 2 * i, 2LL * (W - 1));
  // alpha_j = cos(pi (2j+1)/(2K)) = sin(pi (K - 2j - 1)/(2K))
  for (int j = 0; j < K; ++j) t->alpha[j] = (double)sinpi_ratio((long long)K - 2 * j - 1, 2LL * K);
}

void build_locate_basis(int W, int M, LocateBasis* t) {
  std::memset(t, 0, sizeof(*t));
  if (M < 1 || M >= W) return;
  const int P = (W + 7) / 8 * 8;
  // Householder QR of the W x M matrix [T_k(beta_i)] (Chebyshev polynomials: the same column spaces as the
  // monomials, far better conditioned), in extended precision.  Columns M .. W-1 of Q = H_0 .. H_{M-1} are
  // the basis.
  long double a[kMaxW][kMaxW];  // a[i][k]
  long double v[kMaxW][kMaxW];  // v[k][i]: reflector k, H_k = I - v v^T with |v|^2 = 2
  for (int i = 0; i < W; ++i) {
    const long double b = sinpi_ratio((long long)(W - 1) - 2 * i, 2LL * (W - 1));
    a[i][0] = 1.0L;
    if (M > 1) a[i][1] = b;
    for (int k = 2; k < M; ++k) a[i][k] = 2.0L * b * a[i][k - 1] - a[i][k - 2];
  }
  for (int k = 0; k < M; ++k) {
    long double s2 = 0.0L;
    for (int i = k; i < W; ++i) s2 += a[i][k] * a[i][k];
    const long double normx = sqrtl(s2);
    const long double x0 = a[k][k];
    const long double akk = (x0 >= 0.0L) ? -normx : normx;
    const long double c = s2 + fabsl(x0) * normx;
    const long double scale = (c > 0.0L) ? 1.0L / sqrtl(c) : 0.0L;
    for (int i = 0; i < W; ++i) v[k][i] = (i < k) ? 0.0L : ((i == k) ? (x0 - akk) * scale : a[i][k] * scale);
    for (int j = k; j < M; ++j) {
      long double dot = 0.0L;
      for (int i = k; i < W; ++i) dot += v[k][i] * a[i][j];
      for (int i = k; i < W; ++i) a[i][j] -= dot * v[k][i];
    }
  }
  for (int d = 0; d < W - M; ++d) {
    long double q[kMaxW];
    for (int i = 0; i < W; ++i) q[i] = (i == M + d) ? 1.0L : 0.0L;
    for (int k = M - 1; k >= 0; --k) {
      long double dot = 0.0L;
      for (int i = k; i < W; ++i) dot += v[k][i] * q[i];
      for (int i = k; i < W; ++i) q[i] -= dot * v[k][i];
    }
    for (int i = 0; i < W; ++i) t->nft[d * P + i] = (double)q[i];
  }
}

namespace {

template <typename T, typename Build>
const T& cached(std::map<int, std::unique_ptr<T>>& cache, std::mutex& mu, int key, Build build) {
  std::lock_guard<std::mutex> lock(mu);
  std::unique_ptr<T>& slot = cache[key];
  if (!slot) {
    slot.reset(new T);
    build(slot.get());
  }
  return *slot;
}

}  // namespace

const EncodeTables& encode_tables(int K, int W) {
  static std::map<int, std::unique_ptr<EncodeTables>> cache;
  static std::mutex mu;
  return cached(cache, mu, K * 64 + W, [&](EncodeTables* t) { build_encode_tables(K, W, t); });
}

const DecodeTables& decode_tables(int K, int W) {
  static std::map<int, std::unique_ptr<DecodeTables>> cache;
  static std::mutex mu;
  return cached(cache, mu, K * 64 + W, [&](DecodeTables* t) { build_decode_tables(K, W, t); });
}

const LocateTables& locate_tables(int K, int W) {
  static std::map<int, std::unique_ptr<LocateTables>> cache;
  static std::mutex mu;
  return cached(cache, mu, K * 64 + W, [&](LocateTables* t) { build_locate_tables(K, W, t); });
}

const LocateBasis& locate_basis(int W, int M) {
  static std::map<int, std::unique_ptr<LocateBasis>> cache;
  static std::mutex mu;
  return cached(cache, mu, W * 64 + M, [&](LocateBasis* t) { build_locate_basis(W, M, t); });
}

}  // namespace approxifer
