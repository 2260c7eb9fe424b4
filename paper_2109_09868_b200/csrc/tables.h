// Host-side node tables of ApproxIFER (Section 3): Chebyshev nodes alpha_j
// (first kind) and beta_i (second kind), their gaps, and the encoder's weight
// matrix.  Everything here depends only on (K, W) and is evaluated once per
// call in extended precision, then rounded.
#pragma once
#include <cstdint>

namespace approxifer {

constexpr int kMaxK = 32;
constexpr int kMaxW = 32;

// Launch-constant tables for the decoder, passed to the kernel by value.
struct DecodeTables {
  // rg[i*K + j] = 1/(alpha_j - beta_i), 0 where the two nodes coincide.
  float rg[kMaxW * kMaxK];
  // coin[j] = the worker i with beta_i == alpha_j, or -1.
  int8_t coin[kMaxK];
  int32_t any_coin;
};

// Launch-constant weights of the encoder: w[i*K + j] = l_j(beta_i).
struct EncodeTables {
  float w[kMaxW * kMaxK];
};

// beta_i (and alpha_j, for Algorithm 3) in double for the locator.
struct LocateTables {
  double beta[kMaxW];
  double alpha[kMaxK];
};

// Orthonormal basis Nf of the orthogonal complement of {polynomials of degree < M} on the FULL node set
// beta_0 .. beta_{W-1} (all workers present), stored transposed and zero-padded the way the locator keeps it
// in shared memory: nft[d * P + i] = Nf[i][d] for i < W, d < W - M, with P = W rounded up to a multiple of 8;
// (P - M) * P entries are meaningful, the rest is 0.  The locator derives the basis of a group with a few
// workers missing from this one instead of factorising from scratch.
struct LocateBasis {
  double nft[kMaxW * kMaxW];
};

// alpha_j == beta_i exactly when (2j+1)(W-1) == 2 K i.
inline bool nodes_coincide(int K, int W, int j, int i) { return (2 * j + 1) * (W - 1) == 2 * K * i; }

// alpha_j - beta_i, evaluated without cancellation from
// cos a - cos b = -2 sin((a+b)/2) sin((a-b)/2) with exact rational arguments.
long double node_gap(int K, int W, int j, int i);

void build_encode_tables(int K, int W, EncodeTables* t);
void build_decode_tables(int K, int W, DecodeTables* t);
void build_locate_tables(int K, int W, LocateTables* t);
void build_locate_basis(int W, int M, LocateBasis* t);

// The tables depend on (K, W) only and cost 10-200 us of host time to build, so each is built once per
// process and (K, W) and then served from an immutable, mutex-protected cache.  The references stay valid
// for the life of the process.
const EncodeTables& encode_tables(int K, int W);
const DecodeTables& decode_tables(int K, int W);
const LocateTables& locate_tables(int K, int W);
const LocateBasis& locate_basis(int W, int M);

}  // namespace approxifer
