// Host construction of the SingleQuant rotation factors in float64:
//   R1 = (R1^U R^A)^T  [n1 x n1],   R2 = H R2^U  [n2 x n2]
// (paragraphs "Alignment Rotation Transformation", "Uniformity Rotation Transformation" and
// "The Overall SingleQuant Method"; Algorithm 1 for the factor pair).  Setup code: it runs once
// per layer on the host and is not on the timed path.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <numeric>
#include <vector>

#include "sq_internal.h"

namespace {

using Mat = std::vector<double>;   // row-major square matrix of order n

Mat identity(int n) {
  Mat I(static_cast<size_t>(n) * n, 0.0);
  for (int i = 0; i < n; ++i) I[static_cast<size_t>(i) * n + i] = 1.0;
  return I;
}

// C = A * B, all n x n.
Mat matmul(const Mat& A, const Mat& B, int n) {
  Mat C(static_cast<size_t>(n) * n, 0.0);
  for (int i = 0; i < n; ++i)
    for (int k = 0; k < n; ++k) {
      const double a = A[static_cast<size_t>(i) * n + k];
      if (a == 0.0) continue;
      const double* b = &B[static_cast<size_t>(k) * n];
      double* c = &C[static_cast<size_t>(i) * n];
      for (int j = 0; j < n; ++j) c[j] += a * b[j];
    }
  return C;
}

Mat transpose(const Mat& A, int n) {
  Mat T(A.size());
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) T[static_cast<size_t>(j) * n + i] = A[static_cast<size_t>(i) * n + j];
  return T;
}

// Right-multiplies R (n x n) in place by the Givens rotation of the plane (i, j) in the row
// convention of Lemma 1: for a row x, (x G)_i = x_i cos + x_j sin, (x G)_j = -x_i sin + x_j cos.
void apply_givens_right(Mat& R, int n, int i, int j, double c, double s) {
  for (int r = 0; r < n; ++r) {
    double* row = &R[static_cast<size_t>(r) * n];
    const double a = row[i], b = row[j];
    row[i] = a * c + b * s;
    row[j] = -a * s + b * c;
  }
}

// R_map with v R_map = ||v|| e_1: n-1 plane rotations on adjacent coordinates, last one first.
Mat chain_to_e1(std::vector<double> v) {
  const int n = static_cast<int>(v.size());
  Mat R = identity(n);
  for (int k = n - 1; k >= 1; --k) {
    const double th = std::atan2(v[k], v[k - 1]);
    const double c = std::cos(th), s = std::sin(th);
    const double a = v[k - 1], b = v[k];
    v[k - 1] = a * c + b * s;
    v[k] = -a * s + b * c;
    apply_givens_right(R, n, k - 1, k, c, s);
  }
  return R;
}

// The target of URT: the evenly spaced template q_k = (2k - n - 1)/n, assigned by the rank order of v
// and scaled to the norm of v.  Returns false for the degenerate inputs (n < 2, v = 0) whose URT
// is the identity.
bool uniform_target(const std::vector<double>& v, std::vector<double>& u) {
  const int n = static_cast<int>(v.size());
  bool any = false;
  for (double x : v) any = any || (x != 0.0);
  if (n < 2 || !any) return false;
  std::vector<int> order(n);
  std::iota(order.begin(), order.end(), 0);
  // entries closer than 1e-9 max|v| count as equal and keep their index order
  double vmax = 0.0;
  for (double x : v) vmax = std::max(vmax, std::fabs(x));
  std::vector<double> key(n);
  for (int k = 0; k < n; ++k) key[k] = std::nearbyint(v[k] / (1e-9 * vmax));
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return key[a] < key[b]; });
  double vnorm2 = 0.0, qnorm2 = 0.0;
  for (double x : v) vnorm2 += x * x;
  std::vector<double> q(n);
  for (int k = 1; k <= n; ++k) {
    q[k - 1] = (2.0 * k - n - 1.0) / n;
    qnorm2 += q[k - 1] * q[k - 1];
  }
  const double scale = std::sqrt(vnorm2) / std::sqrt(qnorm2);
  u.assign(n, 0.0);
  for (int k = 0; k < n; ++k) u[order[k]] = scale * q[k];
  return true;
}

// URT: R^U with v R^U = u, u the rank-preserving evenly spaced target of the same norm.
Mat urt(const std::vector<double>& v, std::vector<double>* u_out = nullptr) {
  const int n = static_cast<int>(v.size());
  std::vector<double> u;
  if (!uniform_target(v, u)) return identity(n);
  Mat Rv = chain_to_e1(v);
  Mat Ru = chain_to_e1(u);
  if (u_out) *u_out = u;
  return matmul(Rv, transpose(Ru, n), n);
}

// The (outlier, minimum) pair of ART: largest and smallest magnitude, ties to the lowest index.
// Magnitudes within a relative 1e-9 count as tied (after an ART step two entries are equal in exact
// arithmetic; rounding must not pick between them).
void art_pair(const std::vector<double>& c, int& i, int& j) {
  const int n = static_cast<int>(c.size());
  i = 0;
  for (int k = 1; k < n; ++k)
    if (std::fabs(c[k]) > std::fabs(c[i]) * (1.0 + 1e-9)) i = k;
  j = -1;
  for (int k = 0; k < n; ++k) {
    if (k == i) continue;
    if (j < 0 || std::fabs(c[k]) < std::fabs(c[j]) * (1.0 - 1e-9)) j = k;
  }
}

// ART matrix acting on the left of the column c: diag(G2, O) P_ij.
Mat art(const std::vector<double>& c, const double* O) {
  const int n = static_cast<int>(c.size());
  if (n < 2) return identity(n);
  int i, j;
  art_pair(c, i, j);
  std::vector<int> order;
  order.reserve(n);
  order.push_back(i);
  order.push_back(j);
  for (int k = 0; k < n; ++k)
    if (k != i && k != j) order.push_back(k);
  // D = diag(G2, O); result[r][order[k]] = D[r][k]
  Mat D = identity(n);
  const double a = c[i], b = c[j];
  if (a != 0.0 || b != 0.0) {
    const double th = std::atan2(b, a) - M_PI / 4.0;
    const double cs = std::cos(th), sn = std::sin(th);
    // the block that sends the column (a, b)^T to (r, r)^T / sqrt(2)
    D[0] = cs;
    D[1] = sn;
    D[static_cast<size_t>(n)] = -sn;
    D[static_cast<size_t>(n) + 1] = cs;
  }
  if (O != nullptr && n > 2) {
    const int m = n - 2;
    for (int r = 0; r < m; ++r)
      for (int k = 0; k < m; ++k)
        D[static_cast<size_t>(r + 2) * n + (k + 2)] = O[static_cast<size_t>(r) * m + k];
  }
  Mat RA(static_cast<size_t>(n) * n, 0.0);
  for (int r = 0; r < n; ++r)
    for (int k = 0; k < n; ++k) RA[static_cast<size_t>(r) * n + order[k]] = D[static_cast<size_t>(r) * n + k];
  return RA;
}

// One further ART step: the plane rotation in coordinates (outlier, minimum) of the current column
// that equalises the two (Lemma 1); every other coordinate is left alone.
Mat art_repeat_step(const std::vector<double>& c) {
  const int n = static_cast<int>(c.size());
  Mat M = identity(n);
  if (n < 2) return M;
  int i, j;
  art_pair(c, i, j);
  const double a = c[i], b = c[j];
  if (a == 0.0 && b == 0.0) return M;
  const double th = std::atan2(b, a) - M_PI / 4.0;
  const double cs = std::cos(th), sn = std::sin(th);
  M[static_cast<size_t>(i) * n + i] = cs;
  M[static_cast<size_t>(i) * n + j] = sn;
  M[static_cast<size_t>(j) * n + i] = -sn;
  M[static_cast<size_t>(j) * n + j] = cs;
  return M;
}

// Counter-based generator for the library's own random orthogonal block.
struct SplitMix64 {
  uint64_t s;
  explicit SplitMix64(uint64_t seed) : s(seed) {}
  uint64_t next() {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
  double uniform() { return (static_cast<double>(next() >> 11) + 0.5) * (1.0 / 9007199254740992.0); }
  double normal() {
    const double u1 = uniform(), u2 = uniform();
    return std::sqrt(-2.0 * std::log(u1)) * std::cos(2.0 * M_PI * u2);
  }
};

// Orthonormalises the columns of a Gaussian matrix (Gram-Schmidt, applied twice): the Q factor
// of its QR decomposition with positive diagonal, i.e. a Haar-distributed orthogonal matrix.
Mat random_orthogonal(int m, uint64_t seed) {
  Mat A(static_cast<size_t>(m) * m);
  SplitMix64 rng(seed);
  for (auto& x : A) x = rng.normal();
  for (int col = 0; col < m; ++col) {
    for (int pass = 0; pass < 2; ++pass)
      for (int prev = 0; prev < col; ++prev) {
        double dot = 0.0;
        for (int r = 0; r < m; ++r) dot += A[static_cast<size_t>(r) * m + col] * A[static_cast<size_t>(r) * m + prev];
        for (int r = 0; r < m; ++r) A[static_cast<size_t>(r) * m + col] -= dot * A[static_cast<size_t>(r) * m + prev];
      }
    double nrm = 0.0;
    for (int r = 0; r < m; ++r) nrm += A[static_cast<size_t>(r) * m + col] * A[static_cast<size_t>(r) * m + col];
    nrm = std::sqrt(nrm);
    for (int r = 0; r < m; ++r) A[static_cast<size_t>(r) * m + col] /= nrm;
  }
  return A;
}

Mat sylvester_hadamard(int n) {
  Mat H(static_cast<size_t>(n) * n);
  const double s = 1.0 / std::sqrt(static_cast<double>(n));
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < n; ++j) H[static_cast<size_t>(i) * n + j] = (__builtin_popcount(i & j) & 1) ? -s : s;
  return H;
}

}  // namespace

namespace sq {

sq_status_t build_factors_host(const float* calib, int64_t T, int64_t n, int32_t n1, int32_t n2,
                               uint32_t flags, uint64_t seed, const double* O,
                               std::vector<float>& R1out, std::vector<float>& R2out, R2Structure* s2) {
  // 1. the calibration token with the largest |entry|, and where that entry sits
  int64_t t_star = 0, pos = 0;
  float best = -1.0f;
  for (int64_t t = 0; t < T; ++t)
    for (int64_t c = 0; c < n; ++c) {
      const float a = std::fabs(calib[t * n + c]);
      if (a > best) {
        best = a;
        t_star = t;
        pos = c;
      }
    }
  const int q_star = static_cast<int>(pos % n2);
  std::vector<double> A(static_cast<size_t>(n));
  for (int64_t c = 0; c < n; ++c) A[c] = static_cast<double>(calib[t_star * n + c]);
  std::vector<double> col(n1);
  for (int p = 0; p < n1; ++p) col[p] = A[static_cast<size_t>(p) * n2 + q_star];

  // 2. ART on that column, 3. URT_1 on its image; L = (R^U)^T R^A is R1^T
  Mat RA;
  if (flags & SQ_ROT_ART) {
    Mat Oown;
    const double* Ouse = O;
    if (Ouse == nullptr && n1 > 2) {
      Oown = random_orthogonal(n1 - 2, seed);
      Ouse = Oown.data();
    }
    RA = art(col, Ouse);
    const int art_steps = static_cast<int>((flags >> 8) & 0x7FFu) + 1;
    for (int step = 1; step < art_steps; ++step) {         // repeated ART rotations on the column so far
      std::vector<double> cur(n1, 0.0);
      for (int r = 0; r < n1; ++r)
        for (int k = 0; k < n1; ++k) cur[r] += RA[static_cast<size_t>(r) * n1 + k] * col[k];
      RA = matmul(art_repeat_step(cur), RA, n1);
    }
  } else {
    RA = identity(n1);
  }
  std::vector<double> colp(n1, 0.0);
  for (int r = 0; r < n1; ++r)
    for (int k = 0; k < n1; ++k) colp[r] += RA[static_cast<size_t>(r) * n1 + k] * col[k];
  Mat RU1 = (flags & SQ_ROT_URT) ? urt(colp) : identity(n1);
  Mat L = matmul(transpose(RU1, n1), RA, n1);
  Mat R1 = transpose(L, n1);

  // 4. the row of L A with the largest |entry|; R2 = H URT(row H)
  int row = 0;
  double rbest = -1.0;
  std::vector<double> LA(static_cast<size_t>(n), 0.0);
  for (int r = 0; r < n1; ++r)
    for (int k = 0; k < n1; ++k) {
      const double l = L[static_cast<size_t>(r) * n1 + k];
      if (l == 0.0) continue;
      for (int q = 0; q < n2; ++q) LA[static_cast<size_t>(r) * n2 + q] += l * A[static_cast<size_t>(k) * n2 + q];
    }
  for (int r = 0; r < n1; ++r)
    for (int q = 0; q < n2; ++q) {
      const double a = std::fabs(LA[static_cast<size_t>(r) * n2 + q]);
      if (a > rbest) {
        rbest = a;
        row = r;
      }
    }
  Mat H = (flags & SQ_ROT_HADAMARD) ? sylvester_hadamard(n2) : identity(n2);
  std::vector<double> v(n2, 0.0);
  for (int q = 0; q < n2; ++q)
    for (int k = 0; k < n2; ++k) v[q] += LA[static_cast<size_t>(row) * n2 + k] * H[static_cast<size_t>(k) * n2 + q];
  std::vector<double> u;
  Mat RU2 = (flags & SQ_ROT_URT) ? urt(v, &u) : identity(n2);
  Mat R2 = matmul(H, RU2, n2);
  if (s2 != nullptr) {
    // How R2 was put together, for kernels that apply its pieces one after the other instead of
    // the dense product: x R2 = ((x H) R_map) R'_map^T with the two chains given by v and u.
    s2->known = true;
    s2->hadamard = (flags & SQ_ROT_HADAMARD) != 0 && n2 > 1;
    s2->urt = !u.empty();
    s2->v = s2->urt ? v : std::vector<double>();
    s2->u = u;
  }

  R1out.resize(R1.size());
  R2out.resize(R2.size());
  for (size_t k = 0; k < R1.size(); ++k) R1out[k] = static_cast<float>(R1[k]);
  for (size_t k = 0; k < R2.size(); ++k) R2out[k] = static_cast<float>(R2[k]);
  return SQ_OK;
}

}  // namespace sq
