// TEST INFRASTRUCTURE -- CPU oracle for the Scaled Outer Product per-layer candidate sweep.
//
// A plain, slow, single-threaded C++17 statement of what the sweep computes, written from the
// paper's definitions.  It shares no code, header, table or constant with the CUDA library: only
// tests, the smoke check and the benchmark's CPU-baseline leg may load it.  Build with
//   g++ -std=c++17 -O2 -ffp-contract=off -shared -fPIC   (see oracle/build.py)
// so that every float operation below is one IEEE-754 binary32 operation, rounded to nearest even,
// and fused multiply-adds happen only where std::fmaf / std::fma is written.
//
// Passages followed (paper section / equation):
//   bpw arithmetic s/g + b ............................ Section "Block Scaling", first paragraph
//   reconstruction W ~ s_W * Q_W, absmax scale ........ Section "Block Scaling" (absmax rule);
//                                                       scale taken against max(LUT): "LUT-scale coupling"
//   round_q nearest entry ............................. Section "Block Scaling", Q = round_q(X / s)
//   channel norms c_j = sqrt(E[x_j^2]) ................ Section "Channel Norms"
//   ACos (c-weighted block cosine, mean over blocks) .. Section "Activation-Weighted Cosine Similarity"
//   scale word SwExMy, bit placement .................. Section "Scale Format and Metabit Allocation"
//   F_layer integer shift k* .......................... paragraph "Per-layer scale shift"
//   pair search step 4 (per-block best of both LUTs and, for signed scales, both signs),
//   sign-negated atoms as separate candidates ......... Section "Per-Layer Pair Search"
//   data-derived DD-n by Lloyd updates + snap ......... Section "Per-Layer Pair Search" (steps 2-3, PO2 description)
//   payload: 2n bytes of codes per g = 16 block ....... Section "Overview", item 4
//   element grids by parameters (FP8/10/12 class, HIF7/HIF8) ... Section "Promotion Profiles";
//                                                       paragraph "HIF7/HIF8 hardware rationale"
//   design axes (i)-(iv): partition metric, reassignment metric, Lloyd weighting, pool definition
//                                                       paragraph "Pair-search design axes"
//   outlier extraction before the search (OPQ) ........ Section "Outlier Per-Quantum Extraction (OPQ)"
//   sparse correction of the residual (Wr) ............ Section "Sparse Residual Correction (Wr)"
//
// Where the paper is silent the reading taken is stated at the function that needs it.
//
// Pins: every function here is pinned by tests/test_oracle_*.py against values the paper prints
// (bpw examples, the seven scale-word layouts, 63-value E2M3 grid, hosting ratios), closed forms,
// exact-rational brute force on tiny inputs, and symmetry invariants.  The one thing that cannot
// be pinned is agreement with the paper's own result tables, which need model weights that are
// not available: "parity unpinned" for those tables only.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr int G = 16;  // block size along K (the paper's default g = 16)

enum { KIND_LUT = 0, KIND_FP_E2M3 = 1, KIND_FP_E4M3 = 2, KIND_FP_GRID = 3 };

struct ScaleFmt { int sign_bits, exp_bits, man_bits, bias, top_exp_reserved; };
struct Atom {
  int n_bits, kind, negated, scope; float tmax; int n_entries; float lut[32];
  // KIND_FP_GRID only: a floating-point element grid given by its parameters (see grid_value)
  int grid_exp_bits, grid_man_bits, grid_bias; float grid_neg_max;
};
struct PairStat { double acos, mse; long long n_sel1, n_neg; };

inline float bf16_to_float(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

inline float snap_bf16(float f) {  // round to nearest bf16, ties to even
  uint32_t u;
  std::memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  std::memcpy(&f, &u, 4);
  return f;
}

// ---------------------------------------------------------------------------------------------
// Scale format.  Reading: round to nearest even on the y-bit mantissa, gradual underflow at E = 0,
// bias 2^(x-1)-1, every exponent code finite unless top_exp_reserved, overflow saturates to the
// largest finite value, a positive scale that would round to zero is raised to the smallest
// subnormal.  The F_layer shift 2^k is applied before rounding and undone after decoding.
// ---------------------------------------------------------------------------------------------
struct QScale { float s_hat; uint32_t E, M; };

int fmt_emin(const ScaleFmt& f) { return 1 - f.bias; }
int fmt_emax(const ScaleFmt& f) { return ((1 << f.exp_bits) - 1 - (f.top_exp_reserved ? 1 : 0)) - f.bias; }

QScale scale_quantize(const ScaleFmt& f, float sigma, int k) {
  QScale r{0.0f, 0u, 0u};
  if (!(sigma > 0.0f)) return r;                       // all-zero block: scale word 0, s_hat 0
  const int y = f.man_bits, emin = fmt_emin(f), emax = fmt_emax(f);
  const double v = std::ldexp((double)sigma, k);       // exact
  const double vmax = (2.0 - std::ldexp(1.0, -y)) * std::ldexp(1.0, emax);
  const int e = std::ilogb(v);
  const int eq = std::max(e, emin);
  const double quantum = std::ldexp(1.0, eq - y);
  double q = std::nearbyint(v / quantum) * quantum;    // division by a power of two: exact; RNE
  if (q > vmax) q = vmax;
  if (q == 0.0) q = std::ldexp(1.0, emin - y);
  if (q < std::ldexp(1.0, emin)) {
    r.E = 0;
    r.M = (uint32_t)std::llrint(q / std::ldexp(1.0, emin - y));
  } else {
    const int eo = std::ilogb(q);
    r.E = (uint32_t)(eo + f.bias);
    r.M = (uint32_t)std::llrint(q / std::ldexp(1.0, eo - y)) - (1u << y);
  }
  r.s_hat = (float)std::ldexp(q, -k);                  // one rounding, only if below the fp32 normal range
  return r;
}

float scale_decode(const ScaleFmt& f, uint32_t E, uint32_t M, int k) {
  const int y = f.man_bits;
  double q = (E == 0) ? (double)M * std::ldexp(1.0, fmt_emin(f) - y)
                      : (double)((1u << y) + M) * std::ldexp(1.0, (int)E - f.bias - y);
  return (float)std::ldexp(q, -k);
}

// F_layer.  Reading: a block counts as "in the normal range" when the unrounded exponent of its
// shifted scale satisfies emin <= e + k <= emax; k is searched in [-64, 64]; the count is
// maximised; ties go to the smallest |k|, then to positive k.  Zero scales are ignored.
int f_layer(const ScaleFmt& f, const float* sigma, long long n) {
  std::vector<long long> hist(400, 0);
  for (long long i = 0; i < n; ++i)
    if (sigma[i] > 0.0f) hist[std::ilogb(sigma[i]) + 200]++;
  const int emin = fmt_emin(f), emax = fmt_emax(f);
  int best_k = 0;
  long long best = -1;
  for (int mag = 0; mag <= 64; ++mag) {
    for (int sgn = 0; sgn < 2; ++sgn) {
      if (mag == 0 && sgn == 1) continue;
      const int k = sgn == 0 ? mag : -mag;
      long long cnt = 0;
      for (int e = -200; e < 200; ++e)
        if (e + k >= emin && e + k <= emax) cnt += hist[e + 200];
      if (cnt > best) { best = cnt; best_k = k; }
    }
  }
  return best_k;
}

// Scale word (bit placement).  b-bit container, w_word sign bits, m = b - w_word - x - y metabits.
// w_word = 1: sign at bit b-1, metabits at bits m-1..0, magnitude (E then M) above them.
// w_word = 0, m >= 1: first metabit at bit b-1, the other m-1 at bits m-2..0.
// The selector is the first metabit: bit 0 when w_word = 1, bit b-1 when w_word = 0.
// Returns 0xFFFFFFFF when the requested sign / selector has no bit to live in.
uint32_t scale_word(const ScaleFmt& f, int b, int w_word, uint32_t sign, uint32_t E, uint32_t M, uint32_t selector) {
  const int x = f.exp_bits, y = f.man_bits;
  const int m = b - w_word - x - y;
  if (m < 0 || (sign && !w_word) || (selector && m < 1)) return 0xFFFFFFFFu;
  const uint32_t mag = (E << y) | M;
  if (w_word) return (sign << (b - 1)) | (mag << m) | (m >= 1 ? selector : 0u);
  if (m >= 1) return (selector << (b - 1)) | (mag << (m - 1));
  return mag;
}

// ---------------------------------------------------------------------------------------------
// Encoding.
// LUT: nearest entry in exact arithmetic, ties to the lowest index.  For ascending entries
// a < b, entry b is strictly closer to u than a iff 2u > a + b; 2u and a + b are formed in
// double, where they are exact (fp32 operands, exponent gap far below 2^29).  A repeated entry
// (a == b) is never strictly closer, so the lower index keeps it.
// ---------------------------------------------------------------------------------------------
int encode_lut(const float* lut, int n, float u) {
  int best = 0;
  for (int j = 1; j < n; ++j)
    if (lut[j] > lut[best] && 2.0 * (double)u > (double)lut[best] + (double)lut[j]) best = j;
  return best;
}

// FP element grids.  Reading: E2M3 = 1 sign, 2 exponent, 3 mantissa bits, bias 1, subnormals,
// every code finite (63 distinct values, largest 7.5).  E4M3 = OCP flavour: bias 7, subnormals,
// largest finite 448 (the all-ones code is not a number).  Rounding is to the nearest grid value,
// ties to the even mantissa code, saturating at the largest magnitude.  The code returned is the
// format's own bit pattern sign|E|M.
double fp_grid_value(int kind, int code) {
  const int xb = kind == KIND_FP_E2M3 ? 2 : 4, yb = 3;
  const int bias = kind == KIND_FP_E2M3 ? 1 : 7;
  const int s = (code >> (xb + yb)) & 1, E = (code >> yb) & ((1 << xb) - 1), M = code & ((1 << yb) - 1);
  double mag = E == 0 ? std::ldexp((double)M, 1 - bias - yb) : std::ldexp((double)((1 << yb) + M), E - bias - yb);
  return s ? -mag : mag;
}

float fp_quantize(int kind, float u, int* code_out) {
  const int bits = kind == KIND_FP_E2M3 ? 6 : 8;
  const int half = 1 << (bits - 1);
  const int n_mag = kind == KIND_FP_E2M3 ? half : half - 1;  // E4M3: magnitude code 0x7F excluded
  const double au = std::fabs((double)u);
  int best = 0;
  for (int j = 1; j < n_mag; ++j) {  // magnitude codes ascend with value
    const double a = fp_grid_value(kind, best), b = fp_grid_value(kind, j);
    if (2.0 * au > a + b) best = j;
    else if (2.0 * au == a + b && (j & 1) == 0) best = j;  // tie: even mantissa code
  }
  const bool neg = std::signbit(u);
  if (code_out) *code_out = best | (neg ? half : 0);
  const float q = (float)fp_grid_value(kind, best);
  return neg ? -q : q;
}

// A floating-point element grid by its parameters (promotion-profile formats: FP8 / FP10 / FP12 class
// grids, Section "Promotion Profiles"; HIF7 / HIF8, paragraph "HIF7/HIF8 hardware rationale").
// Magnitude number j = E * 2^y + M has the value (M / 2^y) 2^(1 - bias) for E = 0 and
// (1 + M / 2^y) 2^(E - bias) otherwise: gradual underflow, then binades of 2^y steps.  The grid is the
// magnitudes up to tmax on the positive side and up to neg_max (>= tmax) on the negative side: a
// two's-complement coefficient reaches one step further below zero (HIF7: +120 / -128).  Rounding is to
// the nearest grid value, ties to the even magnitude number, saturating.  The code is sign | j with the
// sign above x + y bits (x = 0: a grid without a sign|E|M code; the sign then sits at bit n_bits - 1).
double grid_value(const Atom& a, int j) {
  const int y = a.grid_man_bits, E = j >> y, M = j & ((1 << y) - 1);
  return E == 0 ? std::ldexp((double)M, 1 - a.grid_bias - y) : std::ldexp((double)((1 << y) + M), E - a.grid_bias - y);
}

float grid_quantize(const Atom& a, float u, int* code_out) {
  const bool neg = std::signbit(u);
  const double limit = neg ? (double)a.grid_neg_max : (double)a.tmax;
  const double au = std::fabs((double)u);
  int best = 0;
  for (int j = 1; grid_value(a, j) <= limit; ++j) {
    const double lo = grid_value(a, best), hi = grid_value(a, j);
    if (2.0 * au > lo + hi) best = j;
    else if (2.0 * au == lo + hi && (j & 1) == 0) best = j;   // tie: even magnitude number
  }
  const int sign_pos = a.grid_exp_bits > 0 ? a.grid_exp_bits + a.grid_man_bits : a.n_bits - 1;
  if (code_out) *code_out = best | (neg ? 1 << sign_pos : 0);
  const float q = (float)grid_value(a, best);
  return neg ? -q : q;
}

// ---------------------------------------------------------------------------------------------
// Per-block evaluation of one candidate.
// Order of the 16-term fp32 sums (paper silent): four quads of 4 consecutive elements, inside a
// quad acc = fmaf(x_r, y_r, acc) for ascending r starting from 0, block value (Q0+Q1)+(Q2+Q3).
// ---------------------------------------------------------------------------------------------
float quad_tree_dot(const float* x, const float* y) {
  float q[4];
  for (int h = 0; h < 4; ++h) {
    float acc = 0.0f;
    for (int r = 0; r < 4; ++r) acc = std::fmaf(x[4 * h + r], y[4 * h + r], acc);
    q[h] = acc;
  }
  return (q[0] + q[1]) + (q[2] + q[3]);
}

struct BlockEval { float cos, sse, s_hat; uint32_t E, M; int code[G]; float q[G]; };

// layer_pot_scale is used when atom.scope == 0 (one power-of-two scale per layer).
BlockEval eval_block(const float* w, const float* c, const Atom& a, const ScaleFmt& f, int k, float layer_pot_scale) {
  BlockEval r{};
  float absmax = 0.0f;
  for (int i = 0; i < G; ++i) absmax = std::max(absmax, std::fabs(w[i]));
  if (a.scope == 0) {
    r.s_hat = absmax > 0.0f ? layer_pot_scale : 0.0f;
  } else {
    const float sigma = absmax / a.tmax;               // s = |w|max / max(LUT)
    const QScale qs = scale_quantize(f, sigma, k);
    r.s_hat = qs.s_hat; r.E = qs.E; r.M = qs.M;
  }
  const float rcp = r.s_hat > 0.0f ? 1.0f / r.s_hat : 0.0f;  // one reciprocal per block, then multiply
  float cw[G], cq[G], err[G];
  for (int i = 0; i < G; ++i) {
    const float u = w[i] * rcp;
    if (a.kind == KIND_LUT) {
      // a negated candidate -(lut) is evaluated by running the base table on -u
      const float uu = a.negated ? -u : u;
      r.code[i] = encode_lut(a.lut, a.n_entries, uu);
      r.q[i] = a.negated ? -a.lut[r.code[i]] : a.lut[r.code[i]];
    } else if (a.kind == KIND_FP_GRID) {
      r.q[i] = grid_quantize(a, u, &r.code[i]);
    } else {
      r.q[i] = fp_quantize(a.kind, u, &r.code[i]);
    }
    cw[i] = c[i] * w[i];
    cq[i] = c[i] * r.q[i];
    err[i] = std::fmaf(-r.s_hat, r.q[i], w[i]);
  }
  // <a, b>_c = sum_i c_i a_i b_i; association (paper silent): <w, w> as (c w) w, <q, q> as (c q) q,
  // <w, q> as (c q) w
  const float nw = quad_tree_dot(cw, w);
  const float dot = quad_tree_dot(cq, w);
  const float nq = quad_tree_dot(cq, r.q);
  r.sse = quad_tree_dot(err, err);
  // zero norms (paper silent): both zero -> 1, exactly one zero -> 0
  if (nw == 0.0f && nq == 0.0f) r.cos = 1.0f;
  else if (nw == 0.0f || nq == 0.0f) r.cos = 0.0f;
  else r.cos = dot / std::sqrt(nw * nq);
  return r;
}

// layer-max power-of-two scale ("^0" scope): 2^ceil(log2(max|W| / tmax)), never saturating
float layer_pot_scale(float wmax, float tmax) {
  if (!(wmax > 0.0f)) return 0.0f;
  const float sigma = wmax / tmax;
  int e = std::ilogb(sigma);
  if (std::ldexp(1.0f, e) < sigma) e += 1;
  return std::ldexp(1.0f, e);
}

void load_block(const uint16_t* W, long long ldw, long long m, long long j, float* w) {
  for (int i = 0; i < G; ++i) w[i] = bf16_to_float(W[m * ldw + j * G + i]);
}

bool same_lut(const Atom& a, const Atom& b) {
  if (a.kind != KIND_LUT || b.kind != KIND_LUT || a.n_entries != b.n_entries || a.tmax != b.tmax) return false;
  return std::memcmp(a.lut, b.lut, sizeof(float) * a.n_entries) == 0;
}

}  // namespace

extern "C" {

// s/g + b bits per weight
double osop_bpw(int scale_bits, int g, int elem_bits) { return (double)scale_bits / (double)g + (double)elem_bits; }

// c_k = sqrt(mean_t X[t,k]^2), FP64 accumulation.  Order (paper silent): chunks of 64 rows,
// sequential fma inside a chunk, chunk partials added in chunk order.
void osop_channel_norms(const float* X, long long T, long long K, long long ldx, float* c) {
  for (long long k = 0; k < K; ++k) {
    double total = 0.0;
    for (long long t0 = 0; t0 < T; t0 += 64) {
      double part = 0.0;
      for (long long t = t0; t < std::min(T, t0 + 64); ++t) {
        const double x = (double)X[t * ldx + k];
        part = std::fma(x, x, part);
      }
      total += part;
    }
    c[k] = (float)std::sqrt(total / (double)T);
  }
}

void osop_scale_quantize(const ScaleFmt* f, float sigma, int k, float* s_hat, unsigned* E, unsigned* M) {
  const QScale q = scale_quantize(*f, sigma, k);
  *s_hat = q.s_hat; *E = q.E; *M = q.M;
}
float osop_scale_decode(const ScaleFmt* f, unsigned E, unsigned M, int k) { return scale_decode(*f, E, M, k); }
unsigned osop_scale_word(const ScaleFmt* f, int b, int w_word, unsigned sign, unsigned E, unsigned M, unsigned sel) {
  return scale_word(*f, b, w_word, sign, E, M, sel);
}
int osop_f_layer(const ScaleFmt* f, const float* sigma, long long n) { return f_layer(*f, sigma, n); }
int osop_encode_lut(const float* lut, int n, float u) { return encode_lut(lut, n, u); }
float osop_fp_quantize(int kind, float u, int* code) { return fp_quantize(kind, u, code); }
double osop_fp_grid_value(int kind, int code) { return fp_grid_value(kind, code); }
float osop_layer_pot_scale(float wmax, float tmax) { return layer_pot_scale(wmax, tmax); }
float osop_grid_quantize(const Atom* a, float u, int* code) { return grid_quantize(*a, u, code); }
double osop_grid_value(const Atom* a, int j) { return grid_value(*a, j); }

// one block under one candidate: cos, sse, s_hat, E, M, codes[16], q[16]
void osop_eval_block(const float* w, const float* c, const Atom* a, const ScaleFmt* f, int k, float pot_scale,
                     float* cos_out, float* sse_out, float* s_hat, unsigned* E, unsigned* M, int* codes, float* q) {
  const BlockEval r = eval_block(w, c, *a, *f, k, pot_scale);
  *cos_out = r.cos; *sse_out = r.sse; *s_hat = r.s_hat; *E = r.E; *M = r.M;
  for (int i = 0; i < G; ++i) { codes[i] = r.code[i]; q[i] = r.q[i]; }
}

// k* per atom (atoms with the same tmax get the same value); k_mode: -1000 = search, else the shift itself.
// Also returns the layer power-of-two scales for scope-0 atoms.
static void layer_prepass(const uint16_t* W, long long M, long long K, long long ldw, const ScaleFmt& f, int k_mode,
                          const Atom* atoms, int n_atoms, int* k_out, float* pot_out) {
  const long long nbk = K / G, NB = M * nbk;
  std::vector<float> amax(NB);
  float wmax = 0.0f;
  for (long long m = 0; m < M; ++m)
    for (long long j = 0; j < nbk; ++j) {
      float w[G], a = 0.0f;
      load_block(W, ldw, m, j, w);
      for (int i = 0; i < G; ++i) a = std::max(a, std::fabs(w[i]));
      amax[m * nbk + j] = a;
      wmax = std::max(wmax, a);
    }
  std::vector<float> sigma(NB);
  for (int i = 0; i < n_atoms; ++i) {
    pot_out[i] = 0.0f;
    k_out[i] = 0;
    if (atoms[i].scope == 0) { pot_out[i] = layer_pot_scale(wmax, atoms[i].tmax); continue; }
    if (k_mode != -1000) { k_out[i] = k_mode; continue; }
    for (long long b = 0; b < NB; ++b) sigma[b] = amax[b] / atoms[i].tmax;
    k_out[i] = f_layer(f, sigma.data(), NB);
  }
}

// The full candidate sweep of one layer.
//   pair_table [n_atoms x n_atoms]: entry [a][a] is candidate a alone; entry [a][a'] (a < a', both LUT
//     candidates of the same width) is the two-codebook quantisation with per-block selector
//     mu_b = [cos_{b,a'} > cos_{b,a}] (tie keeps a).  ACos = mean over blocks of the selected cosine,
//     mse = sum of selected squared errors / (M K), n_sel1 = number of blocks with mu_b = 1.
//     Entries that are not defined have n_sel1 = -1.
//   signed_table (filled when the scale format has a sign bit): for base atoms i <= j, each followed
//     in the alphabet by its own negation, the per-block best of {i, -i, j, -j} with ties resolved in
//     that order; n_sel1 counts blocks that chose j or -j, n_neg blocks that chose a negated table.
//   best[5] = {best_a, best_b (a < b by ACos, ties to the smallest (a, b)), best single LUT candidate,
//              best signed pair i, j}; -1 where undefined.
//   block_cos / block_sse (optional) [n_atoms x N_b].
//   select_metric (design axis ii, the metric of the per-block finishing reassignment): 0 = block
//     cosine (the larger wins), 1 = block squared error (the smaller wins); ties keep the earlier
//     candidate either way.  The reported ACos / mse / counts are those of the resulting assignment;
//     the best pair is ranked by ACos in both cases.
void osop_pair_search_axes(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f,
                           int k_mode, const Atom* atoms, int n_atoms, int select_metric, PairStat* pair_table,
                           PairStat* signed_table, int* k_out, int* best, float* block_cos, float* block_sse) {
  const long long nbk = K / G, NB = M * nbk;
  std::vector<float> pot(n_atoms);
  layer_prepass(W, M, K, ldw, *f, k_mode, atoms, n_atoms, k_out, pot.data());
  const int A = n_atoms;
  std::vector<double> S(A * A, 0.0), E(A * A, 0.0), SS(A * A, 0.0), ES(A * A, 0.0);
  std::vector<long long> N1(A * A, 0), NS1(A * A, 0), NSN(A * A, 0);
  std::vector<int> is_base(A, 0);
  for (int i = 0; i + 1 < A; ++i)
    is_base[i] = atoms[i].kind == KIND_LUT && !atoms[i].negated && atoms[i + 1].negated && same_lut(atoms[i], atoms[i + 1]);
  std::vector<float> cs(A), er(A);
  for (long long m = 0; m < M; ++m)
    for (long long j = 0; j < nbk; ++j) {
      float w[G];
      load_block(W, ldw, m, j, w);
      const long long b = m * nbk + j;
      for (int a = 0; a < A; ++a) {
        const BlockEval r = eval_block(w, c + j * G, atoms[a], *f, k_out[a], pot[a]);
        cs[a] = r.cos; er[a] = r.sse;
        if (block_cos) block_cos[(long long)a * NB + b] = r.cos;
        if (block_sse) block_sse[(long long)a * NB + b] = r.sse;
      }
      for (int a = 0; a < A; ++a) {
        S[a * A + a] += (double)cs[a];
        E[a * A + a] += (double)er[a];
        if (atoms[a].kind != KIND_LUT) continue;
        for (int a2 = a + 1; a2 < A; ++a2) {
          if (atoms[a2].kind != KIND_LUT || atoms[a2].n_bits != atoms[a].n_bits) continue;
          const bool mu = select_metric ? er[a2] < er[a] : cs[a2] > cs[a];
          S[a * A + a2] += (double)(mu ? cs[a2] : cs[a]);
          E[a * A + a2] += (double)(mu ? er[a2] : er[a]);
          N1[a * A + a2] += mu ? 1 : 0;
        }
      }
      if (f->sign_bits)
        for (int i = 0; i < A; ++i) {
          if (!is_base[i]) continue;
          for (int j2 = i; j2 < A; ++j2) {
            if (!is_base[j2] || atoms[j2].n_bits != atoms[i].n_bits) continue;
            const int cand[4] = {i, i + 1, j2, j2 + 1};
            int pick = 0;
            for (int t = 1; t < (j2 == i ? 2 : 4); ++t)
              if (select_metric ? er[cand[t]] < er[cand[pick]] : cs[cand[t]] > cs[cand[pick]]) pick = t;
            SS[i * A + j2] += (double)cs[cand[pick]];
            ES[i * A + j2] += (double)er[cand[pick]];
            NS1[i * A + j2] += pick >= 2 ? 1 : 0;
            NSN[i * A + j2] += (pick & 1) ? 1 : 0;
          }
        }
    }
  const double nb = (double)NB, ne = (double)M * (double)K;
  for (int a = 0; a < A; ++a)
    for (int a2 = 0; a2 < A; ++a2) {
      PairStat& p = pair_table[a * A + a2];
      PairStat& s = signed_table[a * A + a2];
      p = PairStat{0.0, 0.0, -1, -1};
      s = PairStat{0.0, 0.0, -1, -1};
      const bool lut_pair = a2 > a && atoms[a].kind == KIND_LUT && atoms[a2].kind == KIND_LUT && atoms[a].n_bits == atoms[a2].n_bits;
      if (a2 == a || lut_pair) p = PairStat{S[a * A + a2] / nb, E[a * A + a2] / ne, N1[a * A + a2], 0};
      if (f->sign_bits && a2 >= a && is_base[a] && is_base[a2] && atoms[a].n_bits == atoms[a2].n_bits)
        s = PairStat{SS[a * A + a2] / nb, ES[a * A + a2] / ne, NS1[a * A + a2], NSN[a * A + a2]};
    }
  for (int t = 0; t < 5; ++t) best[t] = -1;
  double bp = -2.0, bs = -2.0, bsp = -2.0;
  for (int a = 0; a < A; ++a) {
    if (atoms[a].kind == KIND_LUT && pair_table[a * A + a].acos > bs) { bs = pair_table[a * A + a].acos; best[2] = a; }
    for (int a2 = a + 1; a2 < A; ++a2) {
      if (pair_table[a * A + a2].n_sel1 >= 0 && pair_table[a * A + a2].acos > bp) { bp = pair_table[a * A + a2].acos; best[0] = a; best[1] = a2; }
      if (signed_table[a * A + a2].n_sel1 >= 0 && signed_table[a * A + a2].acos > bsp) { bsp = signed_table[a * A + a2].acos; best[3] = a; best[4] = a2; }
    }
  }
}

void osop_pair_search(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f,
                      int k_mode, const Atom* atoms, int n_atoms, PairStat* pair_table, PairStat* signed_table,
                      int* k_out, int* best, float* block_cos, float* block_sse) {
  osop_pair_search_axes(W, M, K, ldw, c, f, k_mode, atoms, n_atoms, 0, pair_table, signed_table, k_out, best, block_cos, block_sse);
}

// Data-derived DD-n codebook: Lloyd iteration on the pool of blocks that the primary codebook
// reconstructs worst (pair-search steps 2-3).
//   pool      = blocks whose cosine under the primary codebook is <= the pool_rank-th smallest
//               cosine of the layer (ties all in); pool_rank in [1, N_b].
//   domain    = u = w / s_hat with the scale taken against tmax = 1 and the given shift k.
//   weights   = omega_r = c_r / max_k c_k (channel-norm weighted Lloyd, design axis iii).
//   update    = per code j: centroid = S_j / N_j with N_j = sum fix(omega), S_j = sum fix(omega u),
//               fix(v) = llrint(clamp(v, -256, 256) * 2^24) accumulated in int64 (exactly associative);
//               an empty code keeps its entry; every centroid is snapped to bf16; entries re-sorted.
//   distortion[i] = sum omega (u - q)^2 (FP64) under the table used in iteration i; distortion[iters]
//               under the final table.
// Design axes (paragraph "Pair-search design axes"):
//   (i)   pool_by_error = 0: block_metric holds block cosines, the worst blocks are the smallest;
//         pool_by_error = 1: block_metric holds block squared errors (unweighted), the worst are the largest.
//   (iii) uniform_weights = 1: omega = 1 for every channel instead of c / max c.
//   (iv)  pool_rank >= 1: the pool is every block at least as bad as the pool_rank-th worst (the p %
//         rule and top-k are both a rank); pool_rank = 0: the pool is every block at least as bad as
//         the given pool_threshold on the metric (quantile threshold fixed by the caller).
void osop_dd_lloyd_axes(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f, int k,
                        const float* block_metric, int pool_by_error, long long pool_rank, float pool_threshold,
                        int uniform_weights, const float* init_lut, int n_entries, int iters,
                        float* out_lut, double* distortion, long long* pool_count) {
  const long long nbk = K / G, NB = M * nbk;
  const float* block_cos = block_metric;
  float tau = pool_threshold;
  if (pool_rank >= 1) {
    std::vector<float> sorted(block_metric, block_metric + NB);
    if (pool_by_error) {
      std::nth_element(sorted.begin(), sorted.begin() + (pool_rank - 1), sorted.end(), [](float x, float y) { return x > y; });
    } else {
      std::nth_element(sorted.begin(), sorted.begin() + (pool_rank - 1), sorted.end());
    }
    tau = sorted[pool_rank - 1];
  }
  float cmax = 0.0f;
  for (long long i = 0; i < K; ++i) cmax = std::max(cmax, c[i]);
  std::vector<float> omega(K);
  for (long long i = 0; i < K; ++i) omega[i] = uniform_weights ? 1.0f : (cmax > 0.0f ? c[i] / cmax : 0.0f);
  std::vector<float> lut(init_lut, init_lut + n_entries);
  long long cnt = 0;
  for (int it = 0; it <= iters; ++it) {
    std::vector<long long> N(n_entries, 0), S(n_entries, 0);
    double D = 0.0;
    cnt = 0;
    for (long long m = 0; m < M; ++m)
      for (long long j = 0; j < nbk; ++j) {
        const float metric = block_cos[m * nbk + j];
        if (!(pool_by_error ? metric >= tau : metric <= tau)) continue;
        ++cnt;
        float w[G], absmax = 0.0f;
        load_block(W, ldw, m, j, w);
        for (int i = 0; i < G; ++i) absmax = std::max(absmax, std::fabs(w[i]));
        const QScale qs = scale_quantize(*f, absmax, k);   // tmax of a DD atom is declared 1
        const float rcp = qs.s_hat > 0.0f ? 1.0f / qs.s_hat : 0.0f;
        for (int i = 0; i < G; ++i) {
          const float u = w[i] * rcp;
          const float om = omega[j * G + i];
          const int code = encode_lut(lut.data(), n_entries, u);
          const double d = (double)u - (double)lut[code];
          D += (double)om * d * d;
          const float ou = om * u;
          const double ouc = std::min(256.0, std::max(-256.0, (double)ou));
          N[code] += std::llrint((double)om * 16777216.0);
          S[code] += std::llrint(ouc * 16777216.0);
        }
      }
    distortion[it] = D;
    if (it == iters) break;
    for (int jn = 0; jn < n_entries; ++jn)
      if (N[jn] != 0) lut[jn] = snap_bf16((float)((double)S[jn] / (double)N[jn]));
    std::sort(lut.begin(), lut.end());
  }
  for (int jn = 0; jn < n_entries; ++jn) out_lut[jn] = lut[jn];
  *pool_count = cnt;
}

// Grid-constrained DD-n (Section "Per-Layer Pair Search", steps 1 and 3: "histogram-DP cluster selection on the
// deployed LUT value format's grid points", the construction that has no snap-displacement cost).  The paper names
// the construction and prints no recurrence; the reading taken here, step by step:
//   pool, scale, u = w / s_hat and weights omega: exactly those of the Lloyd construction above (same axes);
//   histogram: element u falls into cell t = rint(256 u) (ties to even), clamped to [-320, 320]: cells of width 2^-8
//     over [-1.25, 1.25].  Per cell the fixed-point sums H = sum fix(omega), S = sum fix(omega u) (the product
//     clamped to +-256 as in the Lloyd sums) and Q = sum fix((omega u) u), with fix(v) = llrint(v 2^24) on the fp32
//     products: integer sums, so the histogram does not depend on the order of the elements;
//   clusters: the cells with H > 0, in ascending order, are cut into runs of neighbours; the code point of a run is
//     the grid point of the LUT value format (bf16) nearest to the run's weighted mean S / H -- the quotient in
//     double, rounded to fp32, then to bf16 (nearest even), clamped to [-1.25, 1.25] -- and the run costs
//     Q - 2 q S + q^2 H in double, every product and sum rounded once, in that order;
//   dynamic programme: best[r][j] = the least total cost of cutting cells 0..j into r + 1 runs, a tie between cuts
//     goes to the earliest cut; exactly min(n_entries, cells) runs are used; the table is the runs' code points in
//     ascending order, padded with its last entry when there are fewer cells than entries.
// Returns the table, the least total cost (in units of 2^-24, divided out) and the pool size.
void osop_dd_grid_dp(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f, int k,
                     const float* block_metric, int pool_by_error, long long pool_rank, float pool_threshold,
                     int uniform_weights, int n_entries, float* out_lut, double* cost_out, long long* pool_count) {
  const long long nbk = K / G, NB = M * nbk;
  float tau = pool_threshold;
  if (pool_rank >= 1) {
    std::vector<float> sorted(block_metric, block_metric + NB);
    if (pool_by_error) std::nth_element(sorted.begin(), sorted.begin() + (pool_rank - 1), sorted.end(), [](float x, float y) { return x > y; });
    else std::nth_element(sorted.begin(), sorted.begin() + (pool_rank - 1), sorted.end());
    tau = sorted[pool_rank - 1];
  }
  float cmax = 0.0f;
  for (long long i = 0; i < K; ++i) cmax = std::max(cmax, c[i]);
  std::vector<float> omega(K);
  for (long long i = 0; i < K; ++i) omega[i] = uniform_weights ? 1.0f : (cmax > 0.0f ? c[i] / cmax : 0.0f);
  const int HALF = 320, CELLS = 2 * HALF + 1;
  std::vector<long long> H(CELLS, 0), S(CELLS, 0), Q(CELLS, 0);
  long long cnt = 0;
  for (long long m = 0; m < M; ++m)
    for (long long j = 0; j < nbk; ++j) {
      const float metric = block_metric[m * nbk + j];
      if (!(pool_by_error ? metric >= tau : metric <= tau)) continue;
      ++cnt;
      float w[G], absmax = 0.0f;
      load_block(W, ldw, m, j, w);
      for (int i = 0; i < G; ++i) absmax = std::max(absmax, std::fabs(w[i]));
      const QScale qs = scale_quantize(*f, absmax, k);
      const float rcp = qs.s_hat > 0.0f ? 1.0f / qs.s_hat : 0.0f;
      for (int i = 0; i < G; ++i) {
        const float u = w[i] * rcp;
        const float om = omega[j * G + i];
        const double t = std::nearbyint((double)u * 256.0);          // default rounding mode: ties to even
        const int cell = (int)std::min((double)HALF, std::max((double)-HALF, t)) + HALF;
        const float ou = std::min(256.0f, std::max(-256.0f, om * u));
        const float ouu = ou * u;
        H[cell] += std::llrint((double)om * 16777216.0);
        S[cell] += std::llrint((double)ou * 16777216.0);
        Q[cell] += std::llrint((double)ouu * 16777216.0);
      }
    }
  *pool_count = cnt;
  // the non-empty cells and their prefix sums
  std::vector<long long> pH(1, 0), pS(1, 0), pQ(1, 0);
  for (int t = 0; t < CELLS; ++t)
    if (H[t] > 0) { pH.push_back(pH.back() + H[t]); pS.push_back(pS.back() + S[t]); pQ.push_back(pQ.back() + Q[t]); }
  const int B = (int)pH.size() - 1;
  if (B == 0) {                                   // an empty pool (or all weights zero): nothing to place
    for (int e = 0; e < n_entries; ++e) out_lut[e] = 0.0f;
    *cost_out = 0.0;
    return;
  }
  auto run = [&](int i, int j, float* q_out) {     // cells i..j (inclusive) as one run: its code point and cost
    const double h = (double)(pH[j + 1] - pH[i]), sm = (double)(pS[j + 1] - pS[i]), qq = (double)(pQ[j + 1] - pQ[i]);
    float q = snap_bf16((float)(sm / h));
    q = std::min(1.25f, std::max(-1.25f, q));
    if (q_out) *q_out = q;
    const double qd = (double)q;
    const double a = (2.0 * qd) * sm;
    const double b = (qd * qd) * h;
    return (qq - a) + b;
  };
  const int R = std::min(n_entries, B);
  std::vector<std::vector<double>> best(R, std::vector<double>(B, 0.0));
  std::vector<std::vector<int>> cut(R, std::vector<int>(B, 0));     // first cell of the last run
  for (int j = 0; j < B; ++j) best[0][j] = run(0, j, nullptr);
  for (int r = 1; r < R; ++r)
    for (int j = r; j < B; ++j) {
      double bv = 0.0;
      int bi = -1;
      for (int i = r; i <= j; ++i) {               // the last run is cells i..j, the r runs before it cover 0..i-1
        const double v = best[r - 1][i - 1] + run(i, j, nullptr);
        if (bi < 0 || v < bv) { bv = v; bi = i; }
      }
      best[r][j] = bv;
      cut[r][j] = bi;
    }
  std::vector<float> lut;
  int j = B - 1;
  for (int r = R - 1; r >= 0; --r) {
    const int i = r == 0 ? 0 : cut[r][j];
    float q;
    run(i, j, &q);
    lut.push_back(q);
    j = i - 1;
  }
  std::sort(lut.begin(), lut.end());
  while ((int)lut.size() < n_entries) lut.push_back(lut.back());
  for (int e = 0; e < n_entries; ++e) out_lut[e] = lut[e];
  *cost_out = best[R - 1][B - 1] / 16777216.0;
}

void osop_dd_lloyd(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f, int k,
                   const float* block_cos, long long pool_rank, const float* init_lut, int n_entries, int iters,
                   float* out_lut, double* distortion, long long* pool_count) {
  osop_dd_lloyd_axes(W, M, K, ldw, c, f, k, block_cos, 0, pool_rank, 0.0f, 0, init_lut, n_entries, iters, out_lut, distortion, pool_count);
}

// Materialise: codes and scale words for the chosen codebook(s).
//   candidates per block, in priority order: a, (-a if use_sign), b, (-b if use_sign); the one with the
//   largest block cosine wins, ties keep the earlier.  selector = winner is b or -b; sign = winner is a
//   "-" variant.  The scale word carries the winner's (E, M).
//   codes: 16 n-bit codes per block as one little-endian 16n-bit integer (element r in bits [rn, rn+n)),
//   2n bytes per block.  For LUT atoms the code indexes the atom's table (for a negated table: the
//   index found on -u); for FP atoms it is the format's bit pattern.
//   words: b-bit scale words, block index ascending, as one little-endian bit stream
//   (b = 12: two words per three bytes).  Returns 0, or -1 when a needed sign/selector bit does not exist.
//   select_metric: 0 = the largest block cosine wins, 1 = the smallest block squared error wins (design axis ii).
int osop_pack_axes(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f,
                   const Atom* a, int k_a, const Atom* b, int k_b, int use_sign, int container_bits, int word_sign_bits,
                   int select_metric, unsigned char* codes, unsigned char* words, long long* n_sel1, long long* n_neg) {
  const long long nbk = K / G, NB = M * nbk;
  const int n = a->n_bits;
  const int x = f->exp_bits, y = f->man_bits;
  const int meta = container_bits - word_sign_bits - x - y;
  if (meta < 0 || (use_sign && !word_sign_bits) || (b && meta < 1)) return -1;
  std::memset(codes, 0, (size_t)(NB * 2 * n));
  std::memset(words, 0, (size_t)((NB * container_bits + 7) / 8));
  float wmax = 0.0f;
  for (long long m = 0; m < M; ++m)
    for (long long i = 0; i < K; ++i) wmax = std::max(wmax, std::fabs(bf16_to_float(W[m * ldw + i])));
  *n_sel1 = 0; *n_neg = 0;
  for (long long m = 0; m < M; ++m)
    for (long long j = 0; j < nbk; ++j) {
      float w[G];
      load_block(W, ldw, m, j, w);
      BlockEval bestr{};
      int pick = -1, t = 0;
      for (int which = 0; which < (b ? 2 : 1); ++which) {
        const Atom& base = which ? *b : *a;
        for (int sg = 0; sg < (use_sign ? 2 : 1); ++sg, ++t) {
          Atom cand = base;
          if (sg) cand.negated = 1 - cand.negated;
          const BlockEval r = eval_block(w, c + j * G, cand, *f, which ? k_b : k_a, layer_pot_scale(wmax, cand.tmax));
          if (pick < 0 || (select_metric ? r.sse < bestr.sse : r.cos > bestr.cos)) { bestr = r; pick = which * 2 + sg; }
        }
      }
      const uint32_t sel = pick >= 2, sgn = pick & 1;
      *n_sel1 += sel; *n_neg += sgn;
      const long long blk = m * nbk + j;
      for (int r = 0; r < G; ++r)
        for (int bit = 0; bit < n; ++bit)
          if ((bestr.code[r] >> bit) & 1) {
            const long long pos = (long long)r * n + bit;
            codes[blk * 2 * n + pos / 8] |= (unsigned char)(1u << (pos % 8));
          }
      const uint32_t word = scale_word(*f, container_bits, word_sign_bits, sgn, bestr.E, bestr.M, sel);
      for (int bit = 0; bit < container_bits; ++bit)
        if ((word >> bit) & 1) {
          const long long pos = blk * container_bits + bit;
          words[pos / 8] |= (unsigned char)(1u << (pos % 8));
        }
    }
  return 0;
}

int osop_pack(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f,
              const Atom* a, int k_a, const Atom* b, int k_b, int use_sign, int container_bits, int word_sign_bits,
              unsigned char* codes, unsigned char* words, long long* n_sel1, long long* n_neg) {
  return osop_pack_axes(W, M, K, ldw, c, f, a, k_a, b, k_b, use_sign, container_bits, word_sign_bits, 0, codes, words, n_sel1, n_neg);
}

// ---------------------------------------------------------------------------------------------
// OPQ (Section "Outlier Per-Quantum Extraction (OPQ)").
// Threshold: the m with F_M(m) = (2 Phi(m) - 1)^M = q.  2 Phi(m) - 1 = erf(m / sqrt 2), so m solves
// erf(m / sqrt 2) = q^(1/M); erf is increasing, bisection on [0, 16].
// ---------------------------------------------------------------------------------------------
double osop_opq_threshold(double q, int max_order) {
  const double target = std::pow(q, 1.0 / (double)max_order);
  double lo = 0.0, hi = 16.0;
  for (int it = 0; it < 200; ++it) {
    const double mid = 0.5 * (lo + hi);
    if (std::erf(mid / std::sqrt(2.0)) < target) lo = mid; else hi = mid;
  }
  return 0.5 * (lo + hi);
}

// Extraction.  Element i of block b is an outlier when |w_i| / sigma_b > m.  Readings (the paper does not
// define sigma_b or the record layout beyond "16-bit element index + BF16 value"):
//   sigma_b = sqrt(mean_j w_j^2) over the block's g = 16 elements (root mean square: weights are centred), so the
//   test is w_i^2 g > m^2 sum_j w_j^2, taken in binary64: the squares of bf16 values are exact, the sum runs over
//   j = 0..15 in order, one product m^2 * sum on the right.  A zero block has no outlier.
//   W_out = W with the outliers set to +0 (the codebook input); an outlier keeps its exact bf16 value in the stream.
//   Stream: records ascending by (row m, column k); record = k | bf16 bits << 16 (the 16-bit index is the column:
//   K <= 65536); row_start[m] = first record of row m, row_start[M] = number of records.
//   Records beyond `capacity` are counted, not written.  Returns the number of records.
long long osop_opq_extract(const uint16_t* W, long long M, long long K, long long ldw, double m_thr,
                           uint16_t* W_out, long long ldo, unsigned* row_start, unsigned* records, long long capacity) {
  const long long nbk = K / G;
  const double m2 = m_thr * m_thr;
  long long n = 0;
  for (long long m = 0; m < M; ++m) {
    row_start[m] = (unsigned)n;
    for (long long j = 0; j < nbk; ++j) {
      double w[G], s2 = 0.0;
      for (int i = 0; i < G; ++i) { w[i] = (double)bf16_to_float(W[m * ldw + j * G + i]); s2 = s2 + w[i] * w[i]; }
      const double rhs = m2 * s2;
      for (int i = 0; i < G; ++i) {
        const long long k = j * G + i;
        const uint16_t bits = W[m * ldw + k];
        const bool out = w[i] * w[i] * (double)G > rhs;
        W_out[m * ldo + k] = out ? (uint16_t)0 : bits;
        if (out) {
          if (n < capacity) records[n] = (unsigned)k | ((unsigned)bits << 16);
          ++n;
        }
      }
    }
  }
  row_start[M] = (unsigned)n;
  return n;
}

// ---------------------------------------------------------------------------------------------
// Wr (Section "Sparse Residual Correction (Wr)").  E = W - W_hat for the reconstruction of the chosen codebook(s)
// (per block the winner among a, (-a), b, (-b) exactly as the packer chooses it; W_hat = s_hat q, E_i = w_i - s_hat q_i
// with one rounding, as the block error forms it).  The entries with the largest |E_mk| c_k are kept.  Readings:
//   metric = |E| c_k as one binary32 product; "top sigma" is a rank n_keep given by the caller: tau = the n_keep-th
//   largest metric of the layer, an entry is kept when metric >= tau (ties all in) and metric > 0 (a zero residual
//   corrects nothing);
//   values are E3M4 (sign, 3 exponent bits with bias 3 and the all-ones exponent left out, 4 mantissa bits: largest
//   15.5) of E / 2^e with one exponent e per layer (the "header"): 2^e = the smallest power of two with
//   max|E_kept| / 2^e <= 15.5; nearest, ties to the even magnitude number;
//   stream as for OPQ: record = k | code << 16, ascending by (m, k), row_start[M + 1].
// Returns the number of records; *scale_exp = e (0 when nothing is kept), *tau_out = tau.
// ---------------------------------------------------------------------------------------------
long long osop_wr_extract(const uint16_t* W, long long M, long long K, long long ldw, const float* c, const ScaleFmt* f,
                          const Atom* a, int k_a, const Atom* b, int k_b, int use_sign, int select_metric, long long n_keep,
                          unsigned* row_start, unsigned* records, long long capacity, int* scale_exp, float* tau_out,
                          float* resid_out) {
  const long long nbk = K / G;
  float wmax = 0.0f;
  for (long long m = 0; m < M; ++m)
    for (long long i = 0; i < K; ++i) wmax = std::max(wmax, std::fabs(bf16_to_float(W[m * ldw + i])));
  std::vector<float> E((size_t)(M * K)), metric((size_t)(M * K));
  for (long long m = 0; m < M; ++m)
    for (long long j = 0; j < nbk; ++j) {
      float w[G];
      load_block(W, ldw, m, j, w);
      BlockEval bestr{};
      int pick = -1;
      for (int which = 0; which < (b ? 2 : 1); ++which) {
        const Atom& base = which ? *b : *a;
        for (int sg = 0; sg < (use_sign ? 2 : 1); ++sg) {
          Atom cand = base;
          if (sg) cand.negated = 1 - cand.negated;
          const BlockEval r = eval_block(w, c + j * G, cand, *f, which ? k_b : k_a, layer_pot_scale(wmax, cand.tmax));
          if (pick < 0 || (select_metric ? r.sse < bestr.sse : r.cos > bestr.cos)) { bestr = r; pick = which * 2 + sg; }
        }
      }
      for (int i = 0; i < G; ++i) {
        const long long at = m * K + j * G + i;
        E[(size_t)at] = std::fmaf(-bestr.s_hat, bestr.q[i], w[i]);
        metric[(size_t)at] = std::fabs(E[(size_t)at]) * c[j * G + i];
        if (resid_out) resid_out[at] = E[(size_t)at];
      }
    }
  std::vector<float> sorted(metric);
  std::sort(sorted.begin(), sorted.end(), [](float x, float y) { return x > y; });
  const float tau = sorted[(size_t)(n_keep - 1)];
  float emax = 0.0f;
  for (size_t i = 0; i < E.size(); ++i)
    if (metric[i] >= tau && metric[i] > 0.0f) emax = std::max(emax, std::fabs(E[i]));
  Atom e3m4{};
  e3m4.n_bits = 8; e3m4.kind = KIND_FP_GRID; e3m4.scope = 0; e3m4.tmax = 15.5f; e3m4.grid_neg_max = 15.5f;
  e3m4.grid_exp_bits = 3; e3m4.grid_man_bits = 4; e3m4.grid_bias = 3;
  int e = 0;
  if (emax > 0.0f) e = std::ilogb(layer_pot_scale(emax, 15.5f));
  long long n = 0;
  for (long long m = 0; m < M; ++m) {
    row_start[m] = (unsigned)n;
    for (long long k = 0; k < K; ++k) {
      const size_t at = (size_t)(m * K + k);
      if (!(metric[at] >= tau && metric[at] > 0.0f)) continue;
      int code = 0;
      grid_quantize(e3m4, std::ldexp(E[at], -e), &code);
      if (n < capacity) records[n] = (unsigned)k | ((unsigned)code << 16);
      ++n;
    }
  }
  row_start[M] = (unsigned)n;
  *scale_exp = e;
  *tau_out = tau;
  return n;
}

}  // extern "C"
