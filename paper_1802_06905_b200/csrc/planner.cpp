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

int theorem2_leaf(const Dims& d, double M, double* alb_words) {
  const double image = double(d.C) * d.H * d.W * d.B;   // CHWB (strides 1: the Image term)
  const double filter = double(d.K) * d.C * d.R * d.S;  // KCRS
  const double out = double(d.K) * d.H * d.W * d.B;     // KHWB
  const double rs = double(d.R) * d.S, bhw = double(d.B) * d.H * d.W;
  const double work = out * d.C;                        // KCHWB
  int leaf;
  double alb;
  if (std::min({image, filter, out}) <= M) {
    leaf = 1;      // one array fits: stream the other two once
    alb = std::max({image, filter, out});
  } else if (rs >= M) {
    leaf = 21;     // the filter window alone overflows the fast memory: no reuse at all
    alb = work * rs / M;
  } else if (M * rs >= bhw * bhw) {
    leaf = 221;    // few output positions: the Filter is the array to read once
    alb = filter;
  } else if (std::min(double(d.C), double(d.K)) >= std::sqrt(M / rs)) {
    leaf = 2221;   // the small-filter term of Theorem 1 is reached
    alb = work * std::sqrt(rs / M);
  } else {
    leaf = 2222;   // too few channels to fill a square block: an array-size term is reached
    alb = std::max(out, image);
  }
  if (alb_words) *alb_words = alb;
  return leaf;
}

void parallel_terms(const Dims& d, double M, const int a[4], double t[5]) {
  theorem1_terms(d, M, t);
  t[1] *= double(a[1]);
  t[2] *= double(a[0]) * a[2] * a[3];
}

bool choose_partition(const Dims& d, double M, int p, int a_out[4], double* bound_out) {
  if (p < 1 || p > 65536) return false;
  double base[5];
  theorem1_terms(d, M, base);
  bool found = false;
  long long best_prod = 0;
  double best_bound = 0, best_repl = 0;
  int best[4] = {1, 1, 1, 1};
  for (int aB = 1; aB <= std::min(d.B, p); ++aB)
    for (int aK = 1; aK <= std::min(d.K, p / aB); ++aK)
      for (int aH = 1; aH <= std::min(d.H, p / (aB * aK)); ++aH) {
        // for fixed aB, aK, aH every term grows with aW, but more processors come first
        for (int aW = 1; aW <= std::min(d.W, p / (aB * aK * aH)); ++aW) {
          const long long prod = 1ll * aB * aK * aH * aW;
          const double t2 = base[1] * aK, t3 = base[2] * aB * aH * aW;
          const double bound = std::max({base[0], t2, t3, base[3], base[4]});
          const double repl = t2 + t3;
          const int cand[4] = {aB, aK, aH, aW};
          bool better = !found || prod > best_prod;
          if (!better && prod == best_prod) {
            if (bound != best_bound) better = bound < best_bound;
            else if (repl != best_repl) better = repl < best_repl;
            else better = std::lexicographical_compare(cand, cand + 4, best, best + 4);
          }
          if (better) {
            found = true;
            best_prod = prod; best_bound = bound; best_repl = repl;
            std::copy(cand, cand + 4, best);
          }
        }
      }
  std::copy(best, best + 4, a_out);
  if (bound_out) *bound_out = best_bound;
  return found;
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
  if (d.B % 8 != 0)
    w = "B must be a multiple of 8 (the Image's channel stride must be a multiple of 16 bytes for TMA)";
  if (why) *why = w;
  return w == nullptr;
}

// Cycles that the compulsory HBM traffic of one call takes: reads at the copy rate (about
// 3400 B/clk) plus bf16 Out writes at the rate the epilogue's stores (one 32-byte sector per lane
// and out-channel plane) are absorbed: about 1900 B/clk in 128-byte runs (b_b = 64), about
// 1400 B/clk in 64-byte runs (b_b = 32); both measured on write-bound 1x1 shapes.
static double hbm_floor_cycles(const Dims& d, int bb) {
  return 2.0 * (double(d.Wi()) * d.Hi() * d.C * d.B + double(d.K) * d.R * d.S * d.C) / 3400.0 +
         2.0 * double(d.K) * d.H * d.W * d.B / (bb >= 64 ? 1900.0 : 1400.0);
}

bool choose_halo_tile(const Dims& d, const Machine& m, const int force[6], HaloTile* out) {
  if (!halo_supported(d, nullptr)) return false;
  const int reserve = 2048;  // barriers, TMEM slot, 1024-byte alignment slack
  const int cap = m.smem_optin_bytes - reserve;
  // Cost-model constants, measured on B200 with this kernel (SM cycles):
  //  * words staged into shared memory arrive at about 45 B/clk per SM in this kernel, with 98, 112
  //    or 140 CTAs pulling alike (tile sweeps on the 14x14 shapes; the copy engines alone reach
  //    about 88 B/clk per SM in a micro-benchmark, so this constant stands for the whole
  //    producer/consumer pipeline, not for L2) -- it rewards tiles that fill all SMs;
  //  * one elected thread issues a unit (b_h MMAs) in about 130 + 60*b_h cycles at best with the
  //    straight-line issue blocks (3x3 and 1x1 filters), 170 + 60*b_h with the generic tap loop
  //    (about 145 + 60*b_h where a filter column has four or more taps, which go out in blocks of four);
  //  * the epilogue drains an accumulator at about 14 cycles per TMEM column;
  //  * HBM: a call cannot end before its compulsory reads (about 3400 B/clk, the copy rate) and its
  //    Out writes (about 1900 B/clk with this epilogue's stores) have passed; on write-heavy 1x1
  //    shapes the two add up rather than overlap.
  const double l2_total_bytes_per_clk = 45.0 * m.sm_count, l2_sm_max_bytes_per_clk = 45.0;
  const int RS = d.R * d.S;
  const int c16 = (d.C + 15) / 16;
  const long long units = 1ll * c16 * RS;
  bool found = false;
  HaloTile best;
  for (int bb : {64, 32, 16, 8}) {
    // a batch block that does not divide B is padded by the TMA's out-of-bounds zero fill; take
    // such a block only when no exact one exists.  Blocks of 16 and 8 images (32-byte and 16-byte
    // rows in shared memory: slower copies, more pixels per MMA) are for batches that small ...
    if (bb >= 32 && d.B % bb != 0 && !(bb == 32 && d.B % 32 != 0)) continue;
    // (also for larger batches whose last block of 32 would be partly empty: B = 40 runs five blocks of 8)
    if (bb < 32 && (d.B % bb != 0 || (d.B > bb && d.B % 32 == 0) || (bb == 16 && d.B <= 8))) continue;
    if (force[4] && bb != force[4]) continue;
    for (int bc : {128, 64, 32, 16}) {
      if (bc > c16 * 16 && bc != 16) continue;
      if (force[2] && bc != force[2]) continue;
      // (blocks of 8 or 16 images: whole groups of 32 accumulator columns, i.e. 4 or 2 pixels, even
      // where that is wider than the output row)
      const int bw_max = bb >= 32 ? d.W : (d.W + 32 / bb - 1) / (32 / bb) * (32 / bb);
      for (int bw = 1; bw <= std::min(bw_max, 256 / bb); ++bw) {
        if (force[0] && bw != force[0]) continue;
        const int N = bb * bw;
        if (bb < 32 && N % 32 != 0) continue;
        for (int bh = 1; bh <= d.H && N * bh <= m.tmem_cols; ++bh) {
          if (force[1] && bh != force[1]) continue;
          // split = 2 (two CTAs per tile, half of the channels each): the exchange of partial sums
          // costs more than the shorter main loop saves wherever whole tiles fill the SMs, so this
          // loop searches it only on request (force[5] == 2); see the end of the function.
          for (int split : {1, 2, 4}) {
            if (split != (force[5] == 2 || force[5] == 4 ? force[5] : 1)) continue;
            HaloTile t;
            t.bb = bb; t.bw = bw; t.bh = bh; t.bc = bc; t.bk = 128;
            t.halo_w = d.sw * (bw - 1) + d.R;
            t.halo_h = d.sh * (bh - 1) + d.S;
            if (t.halo_w > 256 || t.halo_h > 256) continue;  // TMA box extents
            t.c16 = c16;
            t.cchunks = (d.C + bc - 1) / bc;
            t.split = split;
            // halves must be whole Image stages of whole 16-channel chunks, and whole 32-column groups
            if (split > 1 && (c16 % (split * (bc / 16)) != 0 || (N * bh) % (32 * split) != 0)) continue;
            // about nine units per Filter stage, a whole number of Image stages where those are
            // shorter (1x1 filters), so that stage boundaries of the two rings coincide
            const int upi = (bc / 16) * RS;
            int uf = 9;
            if (upi < 9 && 9 % upi != 0) uf = (9 / upi) * upi;
            t.uf = int(std::min<long long>(units, uf));
            t.filt_stage_bytes = uint32_t(t.uf) * 4096u;
            const long long img = 1ll * t.halo_w * t.halo_h * bc * bb * 2;
            if (img > cap) continue;
            t.img_stage_bytes = uint32_t(img);
            // Ring depths: shared memory is split between the rings in proportion to the bytes
            // each must deliver per unit (4 KB of Filter, img/upi of Image), since the bytes a ring
            // keeps in flight bound its delivery rate; 2..4 Filter stages, and two Image stages
            // wherever two fit (measured on the 14x14 shapes: 3x3 wants 4 Filter stages, 1x1 two).
            {
              const double per_unit_img = double(img) / upi;
              const double share_f = 4096.0 / (4096.0 + per_unit_img);
              int fs = int(share_f * cap / t.filt_stage_bytes);
              fs = std::max(2, std::min(4, fs));
              while (fs > 2 && (cap - 1ll * fs * t.filt_stage_bytes) / img < 2) --fs;
              t.f_stages = fs;
            }
            const long long left = cap - 1ll * t.f_stages * t.filt_stage_bytes;
            int is = int(std::min<long long>(6, left / img));
            if (force[3]) {
              if (is < force[3]) continue;
              is = force[3];
            }
            if (is < 1) continue;
            t.i_stages = is;  // a single Image stage (huge filters only) runs without overlap
            const int acc_cols = N * bh;
            // a split tile parks the peer's partial sums (128 rows x acc_cols/2 fp32) and stages its
            // own outgoing ones in the idle rings
            if (split > 1 && 1ll * is * img + 1ll * t.f_stages * t.filt_stage_bytes <
                                 1024ll * acc_cols * (split - 1) / split)
              continue;
            t.acc_bufs = (split == 1 && 2 * acc_cols <= m.tmem_cols) ? 2 : 1;
            int cols = 32;
            while (cols < acc_cols * t.acc_bufs) cols *= 2;
            t.tmem_cols = cols;
            t.tiles_k = (d.K + t.bk - 1) / t.bk;
            t.tiles_b = (d.B + bb - 1) / bb;
            t.tiles_w = (d.W + bw - 1) / bw;
            t.tiles_h = (d.H + bh - 1) / bh;
            t.tiles = 1ll * t.tiles_k * t.tiles_b * t.tiles_w * t.tiles_h;
            if (t.tiles > 0x7fffffffll) continue;
            // split tiles run as one wave; clusters of four CTAs stay inside a group of SMs, which
            // leaves some SMs of every group unused: 128 of 148 CTAs is what is counted on
            if (split > 1 && split * t.tiles > (split == 4 ? std::min(m.sm_count, 128) : m.sm_count)) continue;
            t.grid = split > 1 ? int(split * t.tiles) : int(std::min<long long>(t.tiles, m.sm_count));
            t.packed_filter_bytes = 1ll * t.tiles_k * units * 4096;
            // at least ~115 KB so that two CTAs never share an SM (each would want the tensor memory)
            t.smem_bytes = std::max(int(t.i_stages * t.img_stage_bytes +
                                        t.f_stages * t.filt_stage_bytes) + reserve, 117760);
            // ---- cycle model (per SM) ------------------------------------------------------
            const double exec = std::max(N / 2.0, (4096.0 + 32.0 * N) / 128.0);  // math vs operand reads
            const double issue0 = (RS == 9 && d.R == 3) || RS == 1 ? 130.0 : (d.S >= 4 || (d.S == 1 && d.R >= 4) ? 145.0 : 170.0);
            const double unit_clk = std::max(bh * exec, issue0 + 60.0 * bh);     // issue-rate floor
            // every stage of either ring costs the issuing thread a barrier wait and a commit
            const double stage_clk = 150.0;
            const double cyc_mma =
                (double(units) * unit_clk + (double(t.cchunks) + std::ceil(double(units) / t.uf)) * stage_clk) /
                split;
            const double tile_bytes =
                (double(t.cchunks) * double(img) + double(units) * 4096.0) / split;
            const double l2_rate = std::min(l2_sm_max_bytes_per_clk, l2_total_bytes_per_clk / t.grid);
            // 64-byte rows (bb = 32) use the copy engine and the swizzle half as well as 128-byte rows
            const double cyc_copy = tile_bytes / l2_rate * (bb >= 64 ? 1.0 : bb == 32 ? 1.08 : bb == 16 ? 1.4 : 2.0);
            // (64-byte runs of Out, b_b = 32, are absorbed more slowly than 128-byte runs)
            const double cyc_epi = (bb >= 64 ? 14.0 : bb == 32 ? 17.0 : bb == 16 ? 20.0 : 24.0) * acc_cols;
            // every asynchronous copy costs its issuing thread about 700 cycles whatever its
            // size, and a ring's stages are consumed in order: many small stages starve the MMAs
            const double cyc_issue_copies =
                700.0 * std::max(double(t.cchunks), std::ceil(double(units) / t.uf)) / split;
            double tile_cyc = (t.acc_bufs == 2)
                                  ? std::max({cyc_mma, cyc_copy, cyc_epi, cyc_issue_copies})
                                  : std::max({cyc_mma, cyc_copy, cyc_issue_copies}) + cyc_epi;
            if (t.i_stages == 1) {
              // one Image stage: the copy of a channel chunk cannot start before the MMAs on the
              // chunk in front of it are done (Filter copies still run ahead)
              const double cyc_img = double(t.cchunks) * double(img) / split / l2_rate;
              tile_cyc = std::max(cyc_mma + cyc_img, cyc_copy) + (t.acc_bufs == 2 ? 0.0 : cyc_epi);
              if (t.acc_bufs == 2) tile_cyc = std::max(tile_cyc, cyc_epi);
            }
            if (split > 1) {
              // two cluster barriers, all but one share of the fp32 accumulator (128 rows) pushed to
              // the peers (about 32 B/clk), then one share of an epilogue
              tile_cyc = (t.i_stages == 1 ? cyc_mma + cyc_copy : std::max(cyc_mma, cyc_copy)) +
                         1000.0 + 512.0 * acc_cols * (split - 1) / split / 32.0 + cyc_epi / split +
                         4.0 * acc_cols;
            }
            tile_cyc += 400.0;  // hand-overs at a tile boundary (accumulator full/empty, ring restart)
            const double waves = split > 1 ? 1.0 : std::ceil(double(t.tiles) / t.grid);
            t.tile_cycles = tile_cyc;
            // pipeline fill: nothing is issued before the first Image and Filter stages have landed
            const double fill = (double(img) + double(t.filt_stage_bytes)) / l2_rate;
            t.model_cycles = waves * tile_cyc + fill + cyc_epi + 4000.0;
            t.est_cycles = std::max(t.model_cycles, hbm_floor_cycles(d, bb) + 4000.0);
            t.words_smem = double(t.tiles) * (double(t.cchunks) * (img / 2) + double(units) * 2048.0) +
                           double(d.K) * d.H * d.W * d.B;
            // among tiles that the HBM floor makes equal, the one whose own pipeline is fastest
            const bool tie = found && std::fabs(t.est_cycles - best.est_cycles) <= 1e-9 * best.est_cycles;
            const bool tie2 = tie && std::fabs(t.model_cycles - best.model_cycles) <= 1e-9 * best.model_cycles;
            if (!found || (!tie && t.est_cycles < best.est_cycles) ||
                (tie && !tie2 && t.model_cycles < best.model_cycles) ||
                (tie2 && (t.words_smem < best.words_smem ||
                          (t.words_smem == best.words_smem && t.bh < best.bh)))) {
              best = t;
              found = true;
            }
          }
        }
      }
    }
  }
  // Split tiles (two CTAs of a cluster take half of the channels each and exchange partial sums on
  // chip) are searched on request, and for problems in which every CTA streams a long Filter slab
  // past few output pixels: filters of 9 or more taps with at least 144 units per tile
  // (C*R*S >= 2304), where a split tiling exists at all (its tiles run as one wave, so at most half
  // as many tiles as SMs).  Measured on 52 such shapes (B 8..64, C and K 128..2048, 4x4 to 14x14
  // outputs): where the model puts the split tile at 0.70 of the whole tile's time or below, and the
  // split tile at most doubles the accumulator columns computed (a wider batch block on a small
  // batch is mostly zero padding; up to four times the columns where four times as many CTAs then
  // work), the call takes 0.61-0.90 of the time; above 0.70 (14x14 outputs with 256 channels, the
  // benchmark shapes), with 1x1 filters and with shorter slabs it gains nothing or loses up to 30 %.
  if (found && force[5] == 0 && !force[0] && !force[1] && !force[2] && !force[3] && !force[4] &&
      RS >= 9 && units >= 144) {
    const HaloTile whole = best;
    for (int ways : {2, 4}) {
      // (a quarter of fewer than 288 units is too short a loop to pay for the three-way exchange:
      // 5 of 222 random shapes lost 10-14 % to four-way tiles, all of them with 144 units)
      if (ways == 4 && units < 288) continue;
      const int want_split[6] = {0, 0, 0, 0, 0, ways};
      HaloTile sp;
      if (!choose_halo_tile(d, m, want_split, &sp)) continue;
      const double cols_whole = double(whole.tiles) * whole.bb * whole.bw * whole.bh;
      const double cols_split = double(sp.tiles) * sp.bb * sp.bw * sp.bh;
      const bool cols_ok = cols_split <= 2.0 * cols_whole ||
                           (cols_split <= 4.0 * cols_whole && sp.grid >= 4 * whole.grid);
      if (sp.est_cycles <= 0.70 * whole.est_cycles && cols_ok && sp.est_cycles < best.est_cycles)
        best = sp;
    }
  }
  if (found) *out = best;
  return found;
}

bool direct_supported(const Dims& d, const char** why) {
  if (d.B % 8 != 0) {
    if (why) *why = "B must be a multiple of 8 (16-byte TMA strides of the Image)";
    return false;
  }
  if (d.C % 8 != 0) {
    if (why) *why = "C must be a multiple of 8 (16-byte TMA strides of the Filter)";
    return false;
  }
  return true;
}

bool choose_direct_tile(const Dims& d, const Machine& m, const int force[9], DirectTile* out) {
  if (!direct_supported(d, nullptr)) return false;
  const int reserve = 2048;  // barriers, TMEM slot, 1024-byte alignment slack
  const int cap = m.smem_optin_bytes - reserve;
  const int RS = d.R * d.S;
  const int c16 = (d.C + 15) / 16;
  // Cost model (SM cycles; constants measured on B200 with this kernel on the 14x14 benchmark shapes):
  //  * an MMA of 128 x N x 16 occupies the tensor pipe for N/2 cycles; the issue loop sustains
  //    about 87 % of that;
  //  * operands arrive in shared memory at about 44 B/clk per SM when all SMs pull (1 MB per CTA in
  //    21.7 k to 25 k cycles on four tilings);
  //  * a CTA spends about 5300 cycles before its first MMA (set-up, first copies from HBM) and
  //    drains an accumulator at about 15 cycles per column;
  //  * calls overlap (see cconv_direct_kernel): in a stream of calls the SMs stay busy, so the cost
  //    of a call is its SM time (CTAs x CTA lifetime) divided by the SMs; measured periods are that
  //    figure / 0.85 for grids of 28 to 98 CTAs.
  // Objective: the SM time of a call.  It favours few large tiles, whose lifetime is long: a call
  // that runs alone (or must wait for the call in front) takes a CTA lifetime, not the period.
  bool found = false;
  DirectTile best;
  for (int bb : {64, 32}) {
    if (force[0] && bb != force[0]) continue;
    if (!force[0] && bb == 64 && d.B <= 32) continue;  // half of the block would be padding
    for (int bc : {64, 32, 16}) {
      if (force[4] && bc != force[4]) continue;
      if (bc > c16 * 16 && bc != 16) continue;
      for (int kt : {1, 2}) {
        if (force[3] && kt != force[3]) continue;
        if (kt == 2 && d.K <= 128) continue;
        for (int bw = 1; bw <= std::min(d.W, 256 / bb); ++bw) {
          if (force[1] && bw != force[1]) continue;
          const int N = bb * bw;
          for (int bh = 1; bh <= d.H && N * bh * kt <= m.tmem_cols; ++bh) {
            if (force[2] && bh != force[2]) continue;
            DirectTile t;
            t.bb = bb; t.bw = bw; t.bh = bh; t.bc = bc; t.kt = kt;
            t.halo_w = d.sw * (bw - 1) + d.R;
            t.halo_h = d.sh * (bh - 1) + d.S;
            if (t.halo_w > 256 || t.halo_h > 256) continue;
            t.cchunks = (d.C + bc - 1) / bc;
            const long long img = 1ll * t.halo_w * t.halo_h * bc * bb * 2;
            const long long tap_bytes = 1ll * kt * 128 * bc * 2;
            // Filter stages of about 16 KB (whole taps)
            int tg = int(std::max<long long>(1, 16384 / tap_bytes));
            tg = std::min(tg, RS);
            if (force[5]) tg = std::min(force[5], RS);
            t.tg = tg;
            t.fgroups = (RS + tg - 1) / tg;
            const long long fst = tap_bytes * tg;
            if (img + fst > cap) continue;
            t.img_stage_bytes = uint32_t(img);
            t.filt_stage_bytes = uint32_t(fst);
            // Ring depths: shared memory split in proportion to the bytes each ring delivers per
            // channel block, at least two stages each where they fit
            const double per_chunk_f = double(tap_bytes) * RS;
            const double share_f = per_chunk_f / (per_chunk_f + double(img));
            int fs = int(share_f * cap / fst);
            fs = std::max(2, std::min(12, fs));
            while (fs > 2 && (cap - 1ll * fs * fst) / img < 2) --fs;
            if (force[7]) fs = force[7];
            long long left = cap - 1ll * fs * fst;
            if (left < img) continue;
            int is = int(std::min<long long>(6, left / img));
            if (force[6]) {
              if (is < force[6]) continue;
              is = force[6];
            }
            t.i_stages = is;
            t.f_stages = fs;
            if (!force[7]) {
              // left-over shared memory goes to the Filter ring
              left = cap - 1ll * is * img - 1ll * fs * fst;
              t.f_stages = int(std::min<long long>(12, fs + left / fst));
            }
            const int acc_cols = N * bh * kt;
            t.tiles_k = (d.K + 128 * kt - 1) / (128 * kt);
            t.tiles_b = (d.B + bb - 1) / bb;
            t.tiles_w = (d.W + bw - 1) / bw;
            t.tiles_h = (d.H + bh - 1) / bh;
            t.tiles = 1ll * t.tiles_k * t.tiles_b * t.tiles_w * t.tiles_h;
            if (t.tiles > 0x7fffffffll) continue;
            t.grid = int(std::min<long long>(t.tiles, m.sm_count));
            if (force[8]) t.grid = int(std::min<long long>(t.tiles, force[8]));
            const double tiles_per_cta = std::ceil(double(t.tiles) / t.grid);
            t.acc_bufs = (2 * acc_cols <= m.tmem_cols && tiles_per_cta > 1.0) ? 2 : 1;
            int cols = 32;
            while (cols < acc_cols * t.acc_bufs) cols *= 2;
            t.tmem_cols = cols;
            // CTAs that want more than half of the tensor memory must not share an SM
            const int used = int(t.i_stages * t.img_stage_bytes + t.f_stages * t.filt_stage_bytes) + reserve;
            t.smem_bytes = cols > 256 ? std::max(used, 117760) : used;
            // ---- cycle model ----
            const double units = double(c16) * RS;
            const double cyc_mma = units * kt * bh * std::max(N / 2.0, 40.0) / 0.87;
            const double tile_bytes = double(t.cchunks) * (double(img) + double(tap_bytes) * RS);
            const double cyc_copy = tile_bytes / 44.0;
            const double cyc_epi = (bb >= 64 ? 14.6 : 15.6) * acc_cols;
            // a single Image stage cannot be refilled while the MMAs on it run
            const double main_cyc = t.i_stages == 1 ? cyc_mma + double(t.cchunks) * double(img) / 44.0
                                                    : std::max(cyc_mma, cyc_copy);
            const double cta_cyc = 5300.0 + (t.acc_bufs == 2
                                                 ? tiles_per_cta * std::max(main_cyc, cyc_epi) + cyc_epi
                                                 : tiles_per_cta * (main_cyc + cyc_epi));
            t.tile_cycles = main_cyc;
            t.cta_cycles = cta_cyc;
            t.sm_cycles = cta_cyc * t.grid;
            t.est_cycles = t.sm_cycles / m.sm_count / 0.85;
            t.words_smem = double(t.tiles) * tile_bytes / 2.0 + double(d.K) * d.H * d.W * d.B;
            if (!found || t.est_cycles < best.est_cycles ||
                (t.est_cycles == best.est_cycles && t.words_smem < best.words_smem)) {
              best = t;
              found = true;
            }
          }
        }
      }
    }
  }
  if (found) *out = best;
  return found;
}

bool choose_halo_tail(const Dims& d, const Machine& m, const HaloTile& main, int* main_tiles_h,
                      HaloTile* tail) {
  if (main.tiles <= main.grid || main.tiles_h < 2) return false;
  const double waves = double(main.tiles) / main.grid;
  const double frac = waves - std::floor(waves);
  if (frac < 1e-9 || frac > 0.75) return false;  // the last wave is full enough
  const long long per_row = main.tiles / main.tiles_h;
  const int no_force[6] = {0, 0, 0, 0, 0, 1};  // the tail is never split
  bool found = false;
  double best = main.est_cycles * 0.97;  // must beat the single launch by 3 %
  for (int keep = main.tiles_h - 1; keep >= 1 && keep >= main.tiles_h - 4; --keep) {
    Dims dr = d;
    dr.H = d.H - keep * main.bh;
    if (dr.H <= 0) continue;
    HaloTile t;
    if (!choose_halo_tile(dr, m, no_force, &t)) continue;
    if (t.tiles > m.sm_count) continue;  // the tail is one partial wave
    const double main_cyc = std::ceil(double(per_row * keep) / main.grid) * main.tile_cycles;
    // the tail's CTAs start as SMs fall idle: it costs its own tile time after the main waves
    // (the second launch has costs of its own -- launch, set-up, first copies -- of about 6000 cycles)
    const double est = std::max(main_cyc + t.tile_cycles + 14.0 * t.bb * t.bw * t.bh,
                                hbm_floor_cycles(d, main.bb)) + 4000.0 + 6000.0;
    if (est < best) {
      best = est;
      *main_tiles_h = keep;
      *tail = t;
      found = true;
    }
  }
  return found;
}

bool choose_stem_tile(const Dims& d, const Machine& m, StemTile* out, int force_bw) {
  // the Image's row stride must be a multiple of 16 bytes for TMA; a block of 64 images is zero
  // padded past B
  if (d.B % 8 != 0) return false;
  const int reserve = 2048;
  const int cap = m.smem_optin_bytes - reserve;
  const int shc = d.sh * d.C;
  StemTile t;
  // Few out-channels leave MMA rows free: stack consecutive output rows there (row j*kpad + k).
  t.kpad = d.K <= 32 ? 32 : d.K <= 64 ? 64 : 128;
  t.tiles_k = (d.K + 127) / 128;
  bool found = false;
  for (int bhm = 128 / t.kpad; bhm >= 1 && !found; bhm /= 2) {
    if (bhm > 1 && bhm / 2 >= d.H) continue;  // rows past H would only widen the window
    const int kw = (shc * (bhm - 1) + d.S * d.C + 15) / 16 * 16;
    if (kw > 256) continue;
    const long long filt = 1ll * t.tiles_k * d.R * (kw / 16) * 4096;
    if (filt > cap) continue;
    for (int bw = 4; bw >= 1; --bw) {
      if (force_bw > 0 && bw != force_bw) continue;
      if (bw > 1 && bw - 1 >= d.W) continue;  // no wider than the output row
      const int halo_w = d.sw * (bw - 1) + d.R;
      if (halo_w > 256) continue;
      const long long img = 1ll * halo_w * kw * 128;
      if (2 * img + filt > cap) continue;
      t.bhm = bhm;
      t.kw = kw;
      t.khalves = kw / 16;
      t.filt_bytes = uint32_t(filt);
      t.bw = bw;
      t.halo_w = halo_w;
      t.img_stage_bytes = uint32_t(img);
      t.i_stages = int(std::min<long long>(4, (cap - filt) / img));
      found = true;
      break;
    }
  }
  if (!found) return false;
  t.packed_filter_bytes = t.filt_bytes;
  t.tmem_cols = 512;  // all of it: 512 / (64*bw) accumulator buffers (2 for bw = 3 or 4, 4 for bw = 2)
  t.tiles_w = (d.W + t.bw - 1) / t.bw;
  t.tiles_h = (d.H + t.bhm - 1) / t.bhm;
  t.tiles_b = (d.B + 63) / 64;
  t.tiles = 1ll * t.tiles_b * t.tiles_h * t.tiles_w * t.tiles_k;
  if (t.tiles > 0x7fffffffll) return false;
  t.grid = int(std::min<long long>(t.tiles, m.sm_count));
  t.smem_bytes =
      std::max(int(t.i_stages * t.img_stage_bytes + t.filt_bytes) + reserve, 117760);
  t.words_smem = double(t.tiles) * (t.img_stage_bytes / 2) + double(t.grid) * (t.filt_bytes / 2) +
                 double(d.K) * d.H * d.W * d.B;
  *out = t;
  return true;
}

}  // namespace cconv
