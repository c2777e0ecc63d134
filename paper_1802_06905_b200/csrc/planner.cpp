// Host-side tile planner (no CUDA calls in this file).
//
//  * theorem1_terms : the five-term lower bound of Theorem 1 (Section 4.1).
//  * tiling_lp      : the linear program of Section 5 over log_M block sizes, solved with a small
//                     dense primal simplex (Bland's rule; 9 variables, at most 15 rows).
//  * choose_halo_tile: the "legaliser".  The LP is asymptotic (each array block <= M separately,
//                     halo written as b_w + b_r'); the kernel needs integer blocks that satisfy the
//                     tensor-core and TMA shape rules and whose EXACT footprints fit the shared and
//                     tensor memory of one SM together.  Candidates are enumerated and ranked with
//                     a cycle model whose terms are the paper's: words staged per tile (Image halo
//                     block + Filter block) against the arithmetic the tile performs.
#include "planner.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

namespace cconv {

void theorem1_terms(const Dims& d, double M, double t[5]) {
  const double F = double(d.B) * d.C * d.K * d.W * d.H;
  t[0] = double(d.B) * d.K * d.W * d.H;
  t[1] = double(d.sw) * d.sh * d.B * d.C * d.W * d.H;
  t[2] = double(d.C) * d.K * d.R * d.S;
  t[3] = F * d.R * d.S / M;
  t[4] = F * std::sqrt(double(d.R) * d.S * d.sw * d.sh / M);
}

namespace {

// maximise sum(x) s.t. A x <= b (b >= 0), x >= 0.  Tableau simplex, Bland's anti-cycling rule.
bool simplex_max_sum(const std::vector<std::vector<double>>& A, const std::vector<double>& b, int n,
                     std::vector<double>* x) {
  const int m = int(A.size());
  const int cols = n + m + 1;
  std::vector<std::vector<double>> T(m + 1, std::vector<double>(cols, 0.0));
  std::vector<int> basis(m);
  for (int i = 0; i < m; ++i) {
    for (int j = 0; j < n; ++j) T[i][j] = A[i][j];
    T[i][n + i] = 1.0;
    T[i][cols - 1] = b[i];
    basis[i] = n + i;
  }
  for (int j = 0; j < n; ++j) T[m][j] = -1.0;  // reduced costs of "max sum x"
  const double eps = 1e-12;
  for (int iter = 0; iter < 10000; ++iter) {
    int enter = -1;
    for (int j = 0; j < cols - 1; ++j)
      if (T[m][j] < -eps) {
        enter = j;
        break;
      }
    if (enter < 0) break;
    int leave = -1;
    double best = 0;
    for (int i = 0; i < m; ++i)
      if (T[i][enter] > eps) {
        const double ratio = T[i][cols - 1] / T[i][enter];
        if (leave < 0 || ratio < best - eps ||
            (std::fabs(ratio - best) <= eps && basis[i] < basis[leave])) {
          leave = i;
          best = ratio;
        }
      }
    if (leave < 0) return false;  // unbounded: cannot happen, every variable has an upper bound
    const double piv = T[leave][enter];
    for (double& v : T[leave]) v /= piv;
    for (int i = 0; i <= m; ++i)
      if (i != leave && std::fabs(T[i][enter]) > 0) {
        const double f = T[i][enter];
        for (int j = 0; j < cols; ++j) T[i][j] -= f * T[leave][j];
      }
    basis[leave] = enter;
  }
  x->assign(n, 0.0);
  for (int i = 0; i < m; ++i)
    if (basis[i] < n) (*x)[basis[i]] = std::max(0.0, T[i][cols - 1]);
  return true;
}

}  // namespace

bool tiling_lp(const Dims& d, double M, bool pooling, double tiles[9], double* G, double* words) {
  if (!d.positive() || !(M > 1.0)) return false;
  const double lm = std::log(M);
  auto L = [&](double v) { return std::log(v) / lm; };
  enum { b_, c_, k_, w_, h_, r1, r2, s1, s2, NV };
  std::vector<std::vector<double>> A;
  std::vector<double> rhs;
  auto row = [&](std::initializer_list<int> idx, double r) {
    std::vector<double> a(NV, 0.0);
    for (int i : idx) a[i] = 1.0;
    A.push_back(a);
    rhs.push_back(r);
  };
  row({b_, k_, w_, h_}, 1.0);                          // Out block <= M
  if (!pooling) row({c_, k_, r1, r2, s1, s2}, 1.0);    // Filter block <= M
  row({b_, c_, w_, h_, r2, s2}, 1.0);                  // Image block: the four cross terms
  row({b_, c_, w_, s1, r2, s2}, 1.0);
  row({b_, c_, r1, h_, r2, s2}, 1.0);
  row({b_, c_, r1, s1, r2, s2}, 1.0);
  const double ub[NV] = {L(d.B), L(d.C), L(d.K), L(d.W), L(d.H),
                         std::max(0.0, L(d.R) - L(d.sw)), L(d.sw),
                         std::max(0.0, L(d.S) - L(d.sh)), L(d.sh)};
  for (int i = 0; i < NV; ++i) row({i}, ub[i]);
  std::vector<double> x;
  if (!simplex_max_sum(A, rhs, NV, &x)) return false;
  double sum = 0;
  for (int i = 0; i < NV; ++i) {
    tiles[i] = std::exp(x[i] * lm);
    sum += x[i];
  }
  *G = std::exp(sum * lm);
  *words = d.macs() * M / *G;
  return true;
}

bool halo_supported(const Dims& d, const char** why) {
  const char* w = nullptr;
  if (d.B % 32 != 0)
    w = "B must be a multiple of 32 (one swizzled shared-memory row of images)";
  else if (d.C % 8 != 0)
    w = "C must be a multiple of 8 (16-byte TMA strides of Filter)";
  else if (d.R * d.S > 256)
    w = "R*S must be <= 256 (TMA box extent)";
  else if (d.K < 8)
    w = "K must be >= 8";
  if (why) *why = w;
  return w == nullptr;
}

bool choose_halo_tile(const Dims& d, const Machine& m, const int force[5], HaloTile* out) {
  if (!halo_supported(d, nullptr)) return false;
  const int reserve = 2048;  // barriers, TMEM slot, 1024-byte alignment slack
  const int cap = m.smem_optin_bytes - reserve;
  const double l2_bytes_per_clk = 48.0;  // per SM, sustained; calibrated on B200
  bool found = false;
  HaloTile best;
  const int c16 = (d.C + 15) / 16 * 16;
  for (int bb : {64, 32}) {
    if (d.B % bb) continue;
    if (force[4] && bb != force[4]) continue;
    for (int bc : {64, 32, 16}) {
      if (bc > c16 && bc != 16) continue;
      if (force[2] && bc != force[2]) continue;
      for (int bw = 1; bw <= std::min(d.W, 256 / bb); ++bw) {
        if (force[0] && bw != force[0]) continue;
        const int N = bb * bw;
        for (int bh = 1; bh <= d.H && N * bh <= m.tmem_cols; ++bh) {
          if (force[1] && bh != force[1]) continue;
          HaloTile t;
          t.bb = bb; t.bw = bw; t.bh = bh; t.bc = bc; t.bk = 128;
          t.halo_w = d.sw * (bw - 1) + d.R;
          t.halo_h = d.sh * (bh - 1) + d.S;
          if (t.halo_w > 256 || t.halo_h > 256) continue;
          t.filt_stage_bytes = uint32_t(d.R) * d.S * t.bk * bc * 2;
          t.img_stage_bytes = uint32_t(t.halo_w) * t.halo_h * bc * bb * 2;
          t.stage_bytes = t.filt_stage_bytes + t.img_stage_bytes;
          if (2ll * t.stage_bytes > cap) continue;
          t.cchunks = (d.C + bc - 1) / bc;
          t.stages = std::min({8, int(cap / t.stage_bytes), std::max(2, 2 * t.cchunks)});
          if (force[3]) {
            if (int(cap / t.stage_bytes) < force[3]) continue;
            t.stages = force[3];
          }
          const int acc_cols = N * bh;
          t.acc_bufs = (2 * acc_cols <= m.tmem_cols) ? 2 : 1;
          int cols = 32;
          while (cols < acc_cols * t.acc_bufs) cols *= 2;
          t.tmem_cols = cols;
          t.tiles_k = (d.K + t.bk - 1) / t.bk;
          t.tiles_b = d.B / bb;
          t.tiles_w = (d.W + bw - 1) / bw;
          t.tiles_h = (d.H + bh - 1) / bh;
          t.tiles = 1ll * t.tiles_k * t.tiles_b * t.tiles_w * t.tiles_h;
          t.grid = int(std::min<long long>(t.tiles, m.sm_count));
          // at least ~115 KB so that two CTAs never share an SM (each would want the tensor memory)
          t.smem_bytes = std::max(int(t.stages * t.stage_bytes) + reserve, 117760);
          // ---- cycle model (per SM) ------------------------------------------------------
          const double per_mma = std::max(N / 2.0, 32.0 + N / 4.0);  // math vs operand reads
          const double n_mma = double(t.cchunks) * (bc / 16) * d.R * d.S * bh;
          const double cyc_mma = n_mma * per_mma;
          const double cyc_l2 = double(t.cchunks) * t.stage_bytes / l2_bytes_per_clk;
          const double cyc_epi = acc_cols * 6.0 + 600.0;  // TMEM loads, convert, 128 rows of stores
          const double tile_cyc = (t.acc_bufs == 2) ? std::max({cyc_mma, cyc_l2, cyc_epi})
                                                    : std::max(cyc_mma, cyc_l2) + cyc_epi;
          const double waves = std::ceil(double(t.tiles) / t.grid);
          t.est_cycles = waves * tile_cyc + 4000.0;
          t.words_smem = double(t.tiles) * t.cchunks * (t.stage_bytes / 2) +
                         double(d.K) * d.H * d.W * d.B;
          if (!found || t.est_cycles < best.est_cycles * (1 - 1e-9) ||
              (std::fabs(t.est_cycles - best.est_cycles) <= 1e-9 * best.est_cycles &&
               t.words_smem < best.words_smem)) {
            best = t;
            found = true;
          }
        }
      }
    }
  }
  if (found) *out = best;
  return found;
}

}  // namespace cconv
