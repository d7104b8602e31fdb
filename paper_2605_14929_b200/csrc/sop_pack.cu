// sop_pack: materialise the chosen codebook(s): per block the best of the (up to four) candidates -- read off
// the per-block cosines of the sweep where they are given, else re-evaluated with the same arithmetic -- is
// encoded: 2n bytes of codes plus one b-bit scale word (sign, exponent, mantissa, selector).  Reads W once,
// writes ~n/8 + b/128 bytes per element; bound by instruction issue (the encode), not by bytes.  Table codes
// come from a uniform cell grid on u where the table allows it, else from a binary search over the thresholds.
#include <string.h>

#include "sop_device.cuh"

namespace sop {

constexpr int PTB = 256;

struct PackArgs {
  const uint16_t* W;
  const float* c;
  long long M, K, ldw, nbk, NB;
  int index_a, index_b, k_mode, use_sign;
  int container_bits, word_sign_bits, meta_bits;
  unsigned char* codes;
  unsigned* words;       // zeroed before the kernel; filled with atomicOr
  unsigned long long* counts;
  const float* block_cos;   // optional [n_atoms x NB]: per-block cosines (or errors, with select_err) of an earlier sweep
  int select_err;           // 1: the smallest block error wins instead of the largest block cosine
  int cos_neg_a, cos_neg_b; // rows of the negated variants of index_a / index_b (-1: unknown, evaluate instead)
};

constexpr int KIND_LUT16 = 100;   // inside this file: a LUT of at most 16 entries (a four-step search is enough)
constexpr int KIND_LUT_CELL = 101; // inside this file: a LUT whose codes come from a uniform cell grid on u (one look-up, one compare)
constexpr int CELL_ROWS_MAX = 1025;
constexpr float CELL_MAGIC = 12582912.0f;   // 1.5 * 2^23: adding it leaves rint(x) in the low mantissa bits

// cell grid of a table: cell = rint(u * invh) + c_half, clamped to [0, 2 c_half]
struct PackCand { int table; int kind; int neg; int scope; int k; float tmax; GridDev grid; int sign_pos; float invh; int c_half; };

// One candidate on one block, everything in registers; same operation order as the sweep kernel.
// The 16 codes come back as bytes, four per word (element i in byte i % 4 of word i / 4).
// METRIC: 0 = codes only, 1 = also the block cosine, 2 = also the block squared error (in cos_out).
template <int METRIC, int KIND>
__device__ __forceinline__ void eval_block_kind(const float (&w)[16], const float (&c)[16], const float* __restrict__ tau,
                                                const float* __restrict__ lutv, int neg, float rcp, float s_hat,
                                                float& cos_out, uint32_t (&code4)[4], const GridDev grid = GridDev(), int sign_pos = 0,
                                                const uint2* __restrict__ cells = nullptr, float invh = 0.0f, int c_half = 0) {
  float qn[4], qd[4], qw[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    float an = 0.0f, ad = 0.0f, aw = 0.0f;
    uint32_t packed = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = 4 * h + r;
      const float u = __fmul_rn(w[i], rcp);
      float q;
      uint32_t code;
      if (KIND == KIND_LUT_CELL) {
        // the cell holds at most one decision threshold: the code is the number of thresholds below the cell, plus one
        // when u lies above the cell's own threshold (+inf when it has none)
        const float uu = neg ? -u : u;
        const float t = fminf(fmaxf(__fmaf_rn(uu, invh, CELL_MAGIC + (float)c_half), CELL_MAGIC), CELL_MAGIC + (float)(2 * c_half));
        const uint2 e = cells[__float_as_uint(t) - __float_as_uint(CELL_MAGIC)];
        code = e.y + (uu > __uint_as_float(e.x) ? 1u : 0u);
        q = neg ? -lutv[code] : lutv[code];
      } else if (KIND == SOP_KIND_LUT || KIND == KIND_LUT16) {
        code = (uint32_t)(KIND == KIND_LUT16 ? count_below<4>(tau, neg ? -u : u) : count_below<5>(tau, neg ? -u : u));
        q = neg ? -lutv[code] : lutv[code];
      } else if (KIND == SOP_KIND_FP_E2M3) {
        q = fp_quantize<SOP_KIND_FP_E2M3>(u);
        code = fp_code<SOP_KIND_FP_E2M3>(q);
      } else if (KIND == SOP_KIND_FP_GRID) {
        q = grid_quantize(u, grid);
        code = grid_code(q, grid, sign_pos);      // at most 8 bits: the host refuses wider grids here
      } else {
        q = fp_quantize<SOP_KIND_FP_E4M3>(u);
        code = fp_code<SOP_KIND_FP_E4M3>(q);
      }
      packed |= code << (8 * r);
      if (METRIC == 1) {
        const float cw = __fmul_rn(c[i], w[i]);
        const float cq = __fmul_rn(c[i], q);
        aw = __fmaf_rn(cw, w[i], aw);
        ad = __fmaf_rn(cq, w[i], ad);
        an = __fmaf_rn(cq, q, an);
      } else if (METRIC == 2) {
        const float e = __fmaf_rn(-s_hat, q, w[i]);     // w - s q with one rounding, as the sweep forms it
        an = __fmaf_rn(e, e, an);
      }
    }
    qn[h] = an; qd[h] = ad; qw[h] = aw;
    code4[h] = packed;
  }
  cos_out = METRIC == 1 ? block_cosine(quad_tree(qw), quad_tree(qn), quad_tree(qd)) : (METRIC == 2 ? quad_tree(qn) : 0.0f);
}

// the quantiser kind is decided once per block, outside the element loops: a kind test inside them lets
// the compiler hoist the FP-grid arithmetic into the table path
template <int METRIC>
__device__ __forceinline__ void eval_block_regs(const float (&w)[16], const float (&c)[16], const float* __restrict__ tau,
                                                const float* __restrict__ lutv, int kind, int neg, float rcp, float s_hat,
                                                float& cos_out, uint32_t (&code4)[4], const GridDev grid, int sign_pos,
                                                const uint2* __restrict__ cells, float invh, int c_half) {
  if (kind == KIND_LUT_CELL) eval_block_kind<METRIC, KIND_LUT_CELL>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4, grid, sign_pos, cells, invh, c_half);
  else if (kind == KIND_LUT16) eval_block_kind<METRIC, KIND_LUT16>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4);
  else if (kind == SOP_KIND_LUT) eval_block_kind<METRIC, SOP_KIND_LUT>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4);
  else if (kind == SOP_KIND_FP_GRID) eval_block_kind<METRIC, SOP_KIND_FP_GRID>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4, grid, sign_pos);
  else if (kind == SOP_KIND_FP_E2M3) eval_block_kind<METRIC, SOP_KIND_FP_E2M3>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4);
  else eval_block_kind<METRIC, SOP_KIND_FP_E4M3>(w, c, tau, lutv, neg, rcp, s_hat, cos_out, code4);
}

// USE_COS: the winner of each block is read off the per-block cosines of a sweep and only it is encoded
// (no channel norms needed); otherwise every candidate of the choice is evaluated here.
template <bool USE_COS>
__global__ void __launch_bounds__(PTB, USE_COS ? 4 : 1) pack_kernel(PackArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res) {
  __shared__ float lutv[2][32], tau[2][32];
  __shared__ uint2 cells[2][CELL_ROWS_MAX];       // per table and cell: {the cell's threshold (+inf: none), thresholds below the cell}
  __shared__ PackCand base[2];
  __shared__ int s_nb, s_nbits;
  __shared__ float s_pot[2];
  __shared__ unsigned s_cnt[2];
  __shared__ int s_row[4];   // rows of block_cos for the candidates a, -a, b, -b (-1: none)
  __shared__ int s_idx[2];   // the two atoms
  __shared__ int s_no_pair;  // the search result holds no pair to pack
  const int tid = threadIdx.x;
  if (tid == 0) {
    int ia = a.index_a, ib = a.index_b;
    const bool from_result = ia == SOP_PAIR_FROM_RESULT;
    if (ia == SOP_PAIR_FROM_RESULT) {
      ia = a.use_sign ? res->best_sa : res->best_a;
      ib = a.use_sign ? res->best_sb : res->best_b;
    }
    // a result without a pair (singles-only search, no signed table, one base atom): nothing is packed and the
    // counts say so; with use_sign the second atom of each must exist too (the negation follows its atom)
    s_no_pair = from_result && (ia < 0 || ib < 0 || ia >= A.n_atoms || ib >= A.n_atoms ||
                                (a.use_sign && (ia + 1 >= A.n_atoms || ib + 1 >= A.n_atoms))) ? 1 : 0;
    ia = max(0, min(A.n_atoms - 1, ia));
    int nb = 1;
    if (ib != SOP_NO_ATOM) { ib = max(0, min(A.n_atoms - 1, ib)); nb = 2; }
    s_nb = nb;
    s_nbits = A.atoms[ia].n_bits;
    const float wmax = res ? res->layer_absmax : 0.0f;
    for (int t = 0; t < nb; ++t) {
      const int idx = t ? ib : ia;
      const sop_atom& at = A.atoms[idx];
      base[t].table = t; base[t].kind = (at.kind == SOP_KIND_LUT && at.n_entries <= 16) ? KIND_LUT16 : at.kind; base[t].neg = at.negated; base[t].scope = at.scope; base[t].tmax = at.tmax;
      base[t].k = a.k_mode == SOP_K_FROM_RESULT ? res->k[idx] : a.k_mode;
      base[t].grid.min_eb = 128 - at.grid_bias; base[t].grid.sh = 23 - at.grid_man_bits;
      base[t].grid.vpos = at.tmax; base[t].grid.vneg = at.grid_neg_max;
      base[t].sign_pos = at.grid_exp_bits + at.grid_man_bits;
      base[t].invh = 0.0f; base[t].c_half = 0;
      s_pot[t] = at.scope == 0 ? layer_pot_scale(wmax, at.tmax) : 0.0f;
      s_idx[t] = idx;
    }
    // from a search result with signs, a and b are base atoms and each is followed by its negation
    s_row[0] = ia;
    s_row[1] = from_result ? ia + 1 : a.cos_neg_a;
    s_row[2] = nb == 2 ? ib : -1;
    s_row[3] = nb == 2 ? (from_result ? ib + 1 : a.cos_neg_b) : -1;
    s_cnt[0] = s_cnt[1] = 0;
  }
  __syncthreads();
  if (s_no_pair) {
    if (a.counts && blockIdx.x == 0 && tid < 2) a.counts[tid] = ~0ull;     // {-1, -1}
    return;
  }
  const int nb = s_nb, n = s_nbits, b = a.container_bits;
  // table values and decision thresholds of the (up to two) tables: one thread per entry (the same rule as
  // build_thresholds: the largest fp32 <= the midpoint, a repeated entry takes the threshold above it)
  if (tid < 32 * nb) {
    const int t = tid >> 5, j = tid & 31, idx = s_idx[t];
    const sop_atom& at = A.atoms[idx];
    const bool dd = (A.dd_mask >> idx) & 1u;
    const int ne = at.kind == SOP_KIND_LUT ? at.n_entries : 2;
    lutv[t][j] = at.kind == SOP_KIND_LUT ? (dd ? A.dd_lut[min(j, ne - 1)] : at.lut[min(j, ne - 1)]) : 0.0f;
    __syncwarp();
    int jj = j;
    while (jj < ne - 1 && lutv[t][jj] == lutv[t][jj + 1]) ++jj;
    tau[t][j] = jj < ne - 1 ? __double2float_rd(0.5 * ((double)lutv[t][jj] + (double)lutv[t][jj + 1])) : __int_as_float(0x7F800000);
  }
  __syncthreads();
  // Cell grids of the tables.  A grid of width h <= (smallest gap between two thresholds) / 2 puts at most one threshold
  // into a cell's closed interval [(k - 1/2) h, (k + 1/2) h]; the first and last cells lie beyond every threshold.  A
  // table with repeated thresholds, or one that would need more than CELL_ROWS_MAX cells, keeps the binary search.
  if (tid < nb) {
    const int t = tid;
    PackCand cd = base[t];
    const int ne = A.atoms[s_idx[t]].kind == SOP_KIND_LUT ? A.atoms[s_idx[t]].n_entries : 0;
    if (ne >= 2) {
      float gap = __int_as_float(0x7F800000), reach = 0.0f;
      bool ok = true;
      for (int j = 0; j < ne - 1; ++j) {
        reach = fmaxf(reach, fabsf(tau[t][j]));
        if (j + 1 < ne - 1) {
          const float g = __fsub_rn(tau[t][j + 1], tau[t][j]);
          if (!(g > 0.0f)) ok = false;
          gap = fminf(gap, g);
        }
      }
      if (ne == 2) gap = 1.0f;
      if (ok && gap > 0.0f && reach < 1.0e6f) {
        const int eh = ilogb_pos(gap) - 1;                       // h = 2^eh <= gap / 2
        if (eh >= -20 && eh <= 20) {
          const float h = pow2f_int(eh);
          const float rows_half = ceilf(__fdiv_rn(reach, h)) + 1.0f;
          if (2.0f * rows_half + 1.0f <= (float)CELL_ROWS_MAX) {
            cd.invh = pow2f_int(-eh);
            cd.c_half = (int)rows_half;
            cd.kind = KIND_LUT_CELL;
          }
        }
      }
    }
    base[t] = cd;
  }
  __syncthreads();
  for (int t = 0; t < nb; ++t) {
    if (base[t].kind != KIND_LUT_CELL) continue;
    const int ch = base[t].c_half, ne = A.atoms[s_idx[t]].n_entries;
    const float h = __fdiv_rn(1.0f, base[t].invh);
    for (int r = tid; r <= 2 * ch; r += PTB) {
      const float lo = __fmul_rn((float)(r - ch) - 0.5f, h), hi = __fmul_rn((float)(r - ch) + 0.5f, h);   // exact: small integers and halves times a power of two
      unsigned below = 0;
      float thr = __int_as_float(0x7F800000);
      for (int j = 0; j < ne - 1; ++j) {
        const float tj = tau[t][j];
        if (r > 0 && tj < lo) ++below;
        else if (r == 2 * ch || tj <= hi) thr = fminf(thr, tj);
      }
      cells[t][r] = make_uint2(__float_as_uint(thr), below);
    }
  }
  __syncthreads();

  const int n_sign = a.use_sign ? 2 : 1;
  unsigned my_sel = 0, my_neg = 0;
  const unsigned nbk32 = (unsigned)a.nbk, NB32 = (unsigned)a.NB;       // the block count fits 31 bits
  const int n_cand = nb * n_sign;
  // the loads of a block (its weights and, when the winner is read off a sweep, the candidates' values) are
  // issued one iteration ahead
  auto fetch = [&](unsigned blk, uint4& v0, uint4& v1, float (&cs4)[4]) {
    const unsigned m = blk / nbk32, j = blk - m * nbk32;
    const uint4* p = reinterpret_cast<const uint4*>(a.W + (long long)m * a.ldw + (long long)j * SOP_G);
    v0 = __ldg(p); v1 = __ldg(p + 1);
    if (USE_COS) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int slot = n_sign == 2 ? q : 2 * q;          // candidate q of the order a, (-a), b, (-b)
        cs4[q] = q < n_cand ? __ldg(a.block_cos + (size_t)s_row[slot] * a.NB + blk) : 0.0f;
      }
    }
  };
  const unsigned stride = gridDim.x * PTB;
  uint4 nv0 = make_uint4(0u, 0u, 0u, 0u), nv1 = nv0;
  float ncs4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  if (blockIdx.x * PTB + tid < NB32) fetch(blockIdx.x * PTB + tid, nv0, nv1, ncs4);
  for (unsigned blk = blockIdx.x * PTB + tid; blk < NB32; blk += stride) {
    const unsigned j = blk % nbk32;
    const uint4 v0 = nv0, v1 = nv1;
    float cs4[4] = {ncs4[0], ncs4[1], ncs4[2], ncs4[3]};
    if (blk + stride < NB32) fetch(blk + stride, nv0, nv1, ncs4);
    const uint32_t wb[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    float w[16], c[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) { w[2 * i] = bf16lo(wb[i]); w[2 * i + 1] = bf16hi(wb[i]); }
    if (USE_COS) {
#pragma unroll
      for (int i = 0; i < 16; ++i) c[i] = 0.0f;
    } else {
      const float4* cp = reinterpret_cast<const float4*>(a.c + j * SOP_G);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = __ldg(cp + q);
        c[4 * q] = v.x; c[4 * q + 1] = v.y; c[4 * q + 2] = v.z; c[4 * q + 3] = v.w;
      }
    }
    // bf16 magnitudes order like their bit patterns: the maximum of the sixteen 15-bit patterns, two per word at a time
    uint32_t mb = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) mb = __vmaxu2(mb, wb[q] & 0x7FFF7FFFu);
    mb = max(mb & 0xFFFFu, mb >> 16);
    const float amax = __uint_as_float(mb << 16);
    float best_cos = 0.0f;
    uint32_t best_scode = 0, best4[4] = {0u, 0u, 0u, 0u};
    int pick = -1;
    if (USE_COS) {
      // the winner follows from the cosines of the sweep (same arithmetic, bit for bit): only it is encoded
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (q >= n_cand) break;
        const float cs = cs4[q];
        const int slot = n_sign == 2 ? q : 2 * q;
        if (pick < 0 || (a.select_err ? cs < best_cos : cs > best_cos)) { best_cos = cs; pick = slot; }
      }
      const int t = pick >> 1, sg = pick & 1;
      const PackCand cd = base[t];
      float s_hat;
      if (cd.scope == 0) {
        s_hat = amax > 0.0f ? s_pot[t] : 0.0f;
      } else {
        const float sigma = cd.tmax == 1.0f ? amax : __fdiv_rn(amax, cd.tmax);
        const QScale qs = scale_quantize(sigma, cd.k, F);
        s_hat = qs.s_hat;
        best_scode = qs.code;
      }
      const float rcp = s_hat > 0.0f ? __frcp_rn(s_hat) : 0.0f;
      float unused;
      eval_block_regs<0>(w, c, tau[t], lutv[t], cd.kind, sg ? 1 - cd.neg : cd.neg, rcp, s_hat, unused, best4, cd.grid, cd.sign_pos, cells[t], cd.invh, cd.c_half);
    } else {
      for (int t = 0; t < nb; ++t) {
        const PackCand cd = base[t];
        float s_hat;
        uint32_t sc = 0;
        if (cd.scope == 0) {
          s_hat = amax > 0.0f ? s_pot[t] : 0.0f;
        } else {
          const float sigma = cd.tmax == 1.0f ? amax : __fdiv_rn(amax, cd.tmax);
          const QScale qs = scale_quantize(sigma, cd.k, F);
          s_hat = qs.s_hat;
          sc = qs.code;
        }
        const float rcp = s_hat > 0.0f ? __frcp_rn(s_hat) : 0.0f;
        for (int sg = 0; sg < n_sign; ++sg) {
          float cs;
          uint32_t c4[4];
          if (a.select_err) eval_block_regs<2>(w, c, tau[t], lutv[t], cd.kind, sg ? 1 - cd.neg : cd.neg, rcp, s_hat, cs, c4, cd.grid, cd.sign_pos, cells[t], cd.invh, cd.c_half);
          else eval_block_regs<1>(w, c, tau[t], lutv[t], cd.kind, sg ? 1 - cd.neg : cd.neg, rcp, s_hat, cs, c4, cd.grid, cd.sign_pos, cells[t], cd.invh, cd.c_half);
          if (pick < 0 || (a.select_err ? cs < best_cos : cs > best_cos)) {
            best_cos = cs; best_scode = sc; pick = 2 * t + sg;
#pragma unroll
            for (int h = 0; h < 4; ++h) best4[h] = c4[h];
          }
        }
      }
    }
    const unsigned sel = pick >> 1, sgn = pick & 1;
    my_sel += sel; my_neg += sgn;
    // codes: 16 n-bit fields, little-endian, 2n bytes
    unsigned long long lo = 0, hi = 0;   // 128-bit accumulator
    if (n == 4) {
      uint32_t h16[4];
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const uint32_t y = (best4[h] | (best4[h] >> 4)) & 0x00FF00FFu;   // bytes 0 and 2 hold two codes each
        h16[h] = (y | (y >> 8)) & 0xFFFFu;
      }
      lo = (unsigned long long)(h16[0] | (h16[1] << 16)) | ((unsigned long long)(h16[2] | (h16[3] << 16)) << 32);
    } else
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int pos = i * n;
      const unsigned long long v = (unsigned long long)((best4[i >> 2] >> (8 * (i & 3))) & 0xFFu);
      if (pos < 64) {
        lo |= v << pos;
        if (pos + n > 64) hi |= v >> (64 - pos);
      } else {
        hi |= v << (pos - 64);
      }
    }
    unsigned short* dst = reinterpret_cast<unsigned short*>(a.codes + (size_t)blk * 2 * n);
    if (n == 4) {
      *reinterpret_cast<uint2*>(dst) = make_uint2((unsigned)lo, (unsigned)(lo >> 32));
    } else if (n == 8) {
      *reinterpret_cast<uint4*>(dst) = make_uint4((unsigned)lo, (unsigned)(lo >> 32), (unsigned)hi, (unsigned)(hi >> 32));
    } else {
      for (int i = 0; i < n; ++i) dst[i] = (unsigned short)((i < 4 ? lo >> (16 * i) : hi >> (16 * (i - 4))) & 0xFFFFu);
    }
    // scale word
    unsigned word;
    if (a.word_sign_bits) word = (sgn << (b - 1)) | (best_scode << a.meta_bits) | (a.meta_bits >= 1 ? sel : 0u);
    else if (a.meta_bits >= 1) word = (sel << (b - 1)) | (best_scode << (a.meta_bits - 1));
    else word = best_scode;
    const long long bit = (long long)blk * b;
    const long long wi = bit >> 5;
    const int sh = (int)(bit & 31);
    if (b == 16) {
      reinterpret_cast<unsigned short*>(a.words)[blk] = (unsigned short)word;
    } else if (b == 8) {
      reinterpret_cast<unsigned char*>(a.words)[blk] = (unsigned char)word;
    } else if (word) {
      atomicOr(&a.words[wi], word << sh);
      if (sh + b > 32) atomicOr(&a.words[wi + 1], word >> (32 - sh));
    }
  }
  if (a.counts) {
    atomicAdd(&s_cnt[0], my_sel);
    atomicAdd(&s_cnt[1], my_neg);
    __syncthreads();
    if (tid < 2 && s_cnt[tid]) atomicAdd(&a.counts[tid], (unsigned long long)s_cnt[tid]);
  }
}

int num_sms();

}  // namespace sop

extern "C" {

int sop_pack(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
             const sop_scale_fmt* fmt, const sop_atom* atoms, int n_atoms, const float* dd_lut_dev,
             unsigned dd_mask, int index_a, int index_b, int k_mode, const sop_search_result* search_dev,
             int use_sign, int container_bits, int word_sign_bits, unsigned char* codes_dev,
             unsigned char* words_dev, long long* counts_dev, const float* block_metric_dev, int flags, void* stream) {
  using namespace sop;
  const float* block_cos_dev = block_metric_dev;
  if (flags & ~SOP_PACK_SELECT_MSE) return SOP_ERR_RANGE;
  int rc = validate_layer(W_dev, M, K, ldw, c_dev, g);
  if (rc) return rc;
  if (!codes_dev || !words_dev) return SOP_ERR_NULL;
  FmtDev F;
  if ((rc = validate_fmt(fmt, &F))) return rc;
  AtomsDev A;
  if ((rc = validate_atoms(atoms, n_atoms, dd_mask, dd_lut_dev, &A))) return rc;
  if (use_sign != 0 && use_sign != 1) return SOP_ERR_FORMAT;
  if (word_sign_bits != 0 && word_sign_bits != 1) return SOP_ERR_FORMAT;
  if (container_bits != 8 && container_bits != 12 && container_bits != 16) return SOP_ERR_FORMAT;
  const int meta = container_bits - word_sign_bits - fmt->exp_bits - fmt->man_bits;
  if (meta < 0 || (use_sign && !word_sign_bits)) return SOP_ERR_FORMAT;
  const bool from_result = index_a == SOP_PAIR_FROM_RESULT;
  if (from_result) {
    if (!search_dev) return SOP_ERR_NULL;
    if (index_b == SOP_NO_ATOM) return SOP_ERR_RANGE;
  } else {
    if (index_a < 0 || index_a >= n_atoms) return SOP_ERR_RANGE;
    if (index_b != SOP_NO_ATOM && (index_b < 0 || index_b >= n_atoms)) return SOP_ERR_RANGE;
    if (index_b != SOP_NO_ATOM && (atoms[index_a].n_bits != atoms[index_b].n_bits || atoms[index_a].kind != SOP_KIND_LUT ||
                                   atoms[index_b].kind != SOP_KIND_LUT)) return SOP_ERR_ALPHABET;
    if (use_sign && atoms[index_a].kind != SOP_KIND_LUT) return SOP_ERR_ALPHABET;
  }
  const bool pair = index_b != SOP_NO_ATOM;
  if (pair && meta < 1) return SOP_ERR_FORMAT;     // the selector needs a metabit
  // a parametric grid is packed as sign | E | M in at most 8 bits; wider grids and grids without such a code are swept only
  if (!from_result && atoms[index_a].kind == SOP_KIND_FP_GRID &&
      (atoms[index_a].grid_exp_bits < 1 || atoms[index_a].n_bits > 8)) return SOP_ERR_ALPHABET;
  if (k_mode == SOP_K_FROM_RESULT) { if (!search_dev) return SOP_ERR_NULL; }
  else if (k_mode < -64 || k_mode > 64) return SOP_ERR_RANGE;
  bool need_wmax = false;
  for (int i = 0; i < n_atoms; ++i) need_wmax |= atoms[i].scope == 0;
  if (need_wmax && !search_dev) return SOP_ERR_NULL;  // the layer power-of-two scale comes from a previous search
  if (((uintptr_t)codes_dev & 15u) || ((uintptr_t)words_dev & 3u)) return SOP_ERR_SHAPE;
  // every atom that can be picked must share n_bits with the first LUT atom when the pair comes from the device
  int n_bits = from_result ? 0 : atoms[index_a].n_bits;
  if (from_result) {
    for (int i = 0; i < n_atoms; ++i)
      if (atoms[i].kind == SOP_KIND_LUT) { if (!n_bits) n_bits = atoms[i].n_bits; else if (atoms[i].n_bits != n_bits) return SOP_ERR_ALPHABET; }
    if (!n_bits) return SOP_ERR_ALPHABET;
  }

  PackArgs a;
  a.W = (const uint16_t*)W_dev; a.c = c_dev; a.M = M; a.K = K; a.ldw = ldw; a.nbk = K / SOP_G; a.NB = M * a.nbk;
  a.index_a = index_a; a.index_b = index_b; a.k_mode = k_mode; a.use_sign = use_sign;
  a.container_bits = container_bits; a.word_sign_bits = word_sign_bits; a.meta_bits = meta;
  a.codes = codes_dev; a.words = (unsigned*)words_dev; a.counts = (unsigned long long*)counts_dev;
  a.block_cos = block_cos_dev;
  a.select_err = (flags & SOP_PACK_SELECT_MSE) ? 1 : 0;
  a.cos_neg_a = a.cos_neg_b = -1;
  if (block_cos_dev && use_sign && !from_result) {
    // row of the negated variant of an explicitly given atom: same table and scale reference, opposite sign
    auto find_neg = [&](int i) {
      for (int j = 0; j < n_atoms; ++j)
        if (j != i && atoms[j].kind == atoms[i].kind && atoms[j].negated != atoms[i].negated && atoms[j].tmax == atoms[i].tmax &&
            atoms[j].n_entries == atoms[i].n_entries && ((dd_mask >> j) & 1u) == ((dd_mask >> i) & 1u) &&
            (((dd_mask >> i) & 1u) || memcmp(atoms[j].lut, atoms[i].lut, sizeof(float) * atoms[i].n_entries) == 0))
          return j;
      return -1;
    };
    a.cos_neg_a = find_neg(index_a);
    if (index_b != SOP_NO_ATOM) a.cos_neg_b = find_neg(index_b);
  }
  cudaStream_t st = (cudaStream_t)stream;
  const size_t word_bytes = (size_t)((a.NB * container_bits + 7) / 8);
  // 12-bit words are merged into the stream with 32-bit atomicOr (the caller's buffer holds whole 32-bit
  // words and starts from zero); 8- and 16-bit words are stored directly, only the padding is cleared
  const size_t padded = (word_bytes + 3) & ~(size_t)3;
  if (container_bits == 12) SOP_CUDA_TRY(cudaMemsetAsync(words_dev, 0, padded, st));
  else SOP_CUDA_TRY(cudaMemsetAsync(words_dev + padded - 4, 0, 4, st));
  if (counts_dev) SOP_CUDA_TRY(cudaMemsetAsync(counts_dev, 0, 2 * sizeof(long long), st));
  long long grid = (a.NB + PTB - 1) / PTB;
  const int sms = num_sms();
  if (grid > (long long)sms * 4) grid = (long long)sms * 4;      // one wave of resident CTAs: the table set-up runs once per CTA
  if ((rc = profile_mark(SOP_PROFILE_PACK, 0, st))) return rc;
  const bool negs_known = !use_sign || from_result || (a.cos_neg_a >= 0 && (!pair || a.cos_neg_b >= 0));
  if (block_cos_dev && negs_known) pack_kernel<true><<<(int)grid, PTB, 0, st>>>(a, A, F, search_dev);
  else pack_kernel<false><<<(int)grid, PTB, 0, st>>>(a, A, F, search_dev);
  if ((rc = profile_mark(SOP_PROFILE_PACK, 1, st))) return rc;
  SOP_CUDA_TRY(cudaGetLastError());
  return SOP_OK;
}

}  // extern "C"
