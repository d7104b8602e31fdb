// sop_opq_extract and sop_wr_extract: the two sparse side streams on either side of the search.
//
// Both are scans with an ordered compaction: a thread owns one 16-element block, a CTA pass ("tile") 256
// consecutive blocks.  The records of a stream ascend by (row, column), which is the order of the blocks and of
// the elements inside a block, so the place of a block's first record is the exclusive prefix sum of the
// per-block record counts:
//   count kernel    per-tile record counts (one 32-bit sum per tile)
//   tile_scan       one CTA turns them into exclusive offsets, writes the total
//   write kernel    recomputes the per-block counts, scans them inside the CTA and writes records and row starts
// Nothing waits on another CTA.
//
//   opq_mask_kernel     reads W once: per block the outlier mask (binary64 test w_i^2 g > m^2 sum w^2), W_out with
//                       the outliers zeroed, the 16-bit mask, the tile count
//   opq_write_kernel    reads the masks, and W only where a mask is set: records (column | bf16 bits << 16)
//   wr_hist_kernel<-1>  first decode pass of the packed stream (scale word -> s_hat, codes -> table values, residual
//                       E = w - s_hat q with one rounding, metric |E| c_k): histogram of one value per block, the
//                       block's largest metric (top 11 bits of the inverted metric bits).  At least n_keep elements
//                       are as large as the n_keep-th largest block maximum, so the threshold lies in that value's
//                       bin or an earlier one
//   wr_pick_kernel      after each histogram: the bin that holds the rank, the prefix for the next pass
//   wr_collect_kernel   second decode pass: every element whose bin is not later than that bound goes to a candidate
//                       list (position, residual, metric): a fraction of a per cent of the layer
//   wr_cand_hist_kernel<0,1,2>, wr_mark_kernel
//                       over the list: three-pass radix select (11 / 11 / 10 bits) of the n_keep-th largest metric,
//                       then the kept set as one 16-bit mask per block, the per-tile counts and the largest kept |E|
//   wr_map_write_kernel E3M4 codes of E / 2^e, records (column | code << 16): decodes only the blocks with a kept entry
//   wr_hist_kernel<0,1,2>, wr_count_kernel, wr_write_kernel
//                       the same steps as full decode passes: taken when the candidates do not fit their list (a
//                       layer whose metrics are nearly all alike).  Both sets of launches are enqueued; the set
//                       that is not needed returns at once (wr_mode_kernel sets the flag on the device).
// The residual is never stored: decoding a block (2.6 bytes per element read) is cheaper than reading 4 bytes.
#include <math.h>
#include <string.h>

#include "sop_device.cuh"

namespace sop {

constexpr int STB = 256;          // threads per CTA = blocks per tile

int num_sms();

struct SparseWs {
  unsigned hist[3][2048];
  unsigned hist_bm[2048];         // histogram of the per-block maxima of the metric (top 11 bits of the inverted key)
  unsigned bm_bin;                // bin of the n_keep-th largest block maximum: the threshold cannot lie in a later bin
  unsigned prefix;                // inverted-key prefix fixed by the selection passes so far
  unsigned tau_bits;              // the threshold metric as fp32 bits (a NaN pattern: nothing is kept)
  unsigned long long rank;        // rank still to find among the keys with that prefix
  unsigned emax_bits;             // max |E| over the kept entries, fp32 bits
  int scale_exp;
  int no_pair;                    // the search result holds no pair: nothing was packed, nothing is corrected
  unsigned n_cand;                // candidates found (may exceed the list's capacity: then the list is not used)
  unsigned overflow;              // 1: the candidates did not fit, the full decode passes do the work
  unsigned pad[3];
};

static size_t sparse_tiles_off() { return (sizeof(SparseWs) + 255) & ~(size_t)255; }
static long long sparse_tiles(long long NB) { return (NB + STB - 1) / STB; }
static size_t sparse_masks_off(long long NB) { return sparse_tiles_off() + (((size_t)sparse_tiles(NB) * 4 + 255) & ~(size_t)255); }
// Wr: behind the per-block masks the candidate list, three 32-bit arrays of wr_cand_cap entries
static size_t wr_cand_off(long long NB) { return sparse_masks_off(NB) + (((size_t)NB * 2 + 255) & ~(size_t)255); }
static unsigned wr_cand_cap(long long NB) { const long long c = NB / 4; return (unsigned)(c > 65536 ? c : 65536); }   // 1/64 of the elements

// exclusive prefix sum of one value per thread over the CTA (STB threads); *total = the CTA's sum
__device__ __forceinline__ unsigned cta_excl_scan(unsigned v, unsigned* s_warp, unsigned* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();                 // s_warp may still be read from the previous tile
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  unsigned base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < STB / 32; ++w) { const unsigned c = s_warp[w]; tot += c; if (w < warp) base += c; }
  *total = tot;
  return base + incl - v;
}

// In place: tile_sums[t] becomes the number of records before tile t.  One CTA of 32 warps: a warp takes a contiguous
// share of the tiles and sums it with coalesced loads, the 32 sums are scanned, the warp then walks its share again
// 32 tiles at a time (a warp scan plus the running sum).  The total goes to row_start[M] and *count.  With `wr` the
// kernel also turns the largest kept |E| into the layer exponent of the Wr values.
__global__ void __launch_bounds__(1024) tile_scan_kernel(unsigned* __restrict__ tile_sums, long long n_tiles, unsigned* __restrict__ row_start,
                                                         long long M, long long* __restrict__ count, SparseWs* __restrict__ ws, int wr,
                                                         int* __restrict__ scale_exp_out, float* __restrict__ tau_out) {
  __shared__ unsigned s_warp[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long per = ((n_tiles + 31) / 32 + 31) / 32 * 32;            // tiles per warp, a multiple of 32
  const long long t0 = (long long)warp * per, t1 = t0 + per < n_tiles ? t0 + per : n_tiles;
  unsigned local = 0;
  for (long long i = t0 + lane; i < t1; i += 32) local += tile_sums[i];
#pragma unroll
  for (int o = 16; o; o >>= 1) local += __shfl_xor_sync(0xFFFFFFFFu, local, o);
  if (lane == 0) s_warp[warp] = local;
  __syncthreads();
  unsigned run = 0, total = 0;
#pragma unroll
  for (int w = 0; w < 32; ++w) { const unsigned c = s_warp[w]; total += c; if (w < warp) run += c; }
  for (long long i0 = t0; i0 < t1; i0 += 32) {
    const long long i = i0 + lane;
    const unsigned v = i < t1 ? tile_sums[i] : 0u;
    unsigned incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    if (i < t1) tile_sums[i] = run + incl - v;
    run += __shfl_sync(0xFFFFFFFFu, incl, 31);
  }
  if (tid == 0) {
    row_start[M] = total;
    if (count) *count = wr && ws->no_pair ? -1ll : (long long)total;
    if (wr) {
      const float emax = __uint_as_float(ws->emax_bits);
      const int e = emax > 0.0f ? ilogb_pos(layer_pot_scale(emax, 15.5f)) : 0;
      ws->scale_exp = e;
      if (scale_exp_out) *scale_exp_out = e;
      if (tau_out) *tau_out = __uint_as_float(ws->tau_bits);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// OPQ
// ---------------------------------------------------------------------------------------------
struct OpqArgs {
  const uint16_t* W;
  uint16_t* W_out;
  long long M, K, ldw, ldo, nbk, NB;
  double m2;                      // the threshold squared
  unsigned short* masks;          // workspace: one 16-bit outlier mask per block
  unsigned* tile_sums;            // workspace
  unsigned* row_start;
  unsigned* records;
  long long capacity;
};

__global__ void __launch_bounds__(STB) opq_mask_kernel(OpqArgs a) {
  __shared__ unsigned s_cnt;
  const int tid = threadIdx.x;
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    const long long blk = tile * STB + tid;
    unsigned mask = 0;
    if (blk < a.NB) {
      const long long m = (long long)((unsigned)blk / (unsigned)a.nbk), j = blk - m * a.nbk;   // the block count fits 31 bits
      const uint4* p = reinterpret_cast<const uint4*>(a.W + m * a.ldw + j * SOP_G);
      const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
      uint32_t wb[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      double sq[16], s2 = 0.0;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const double w = (double)((i & 1) ? bf16hi(wb[i >> 1]) : bf16lo(wb[i >> 1]));
        sq[i] = __dmul_rn(w, w);                 // exact: a bf16 value has 8 significant bits
        s2 = __dadd_rn(s2, sq[i]);               // element order
      }
      const double rhs = __dmul_rn(a.m2, s2);
#pragma unroll
      for (int i = 0; i < 16; ++i)
        if (__dmul_rn(sq[i], 16.0) > rhs) {
          mask |= 1u << i;
          wb[i >> 1] &= (i & 1) ? 0x0000FFFFu : 0xFFFF0000u;
        }
      uint4* q = reinterpret_cast<uint4*>(a.W_out + m * a.ldo + j * SOP_G);
      q[0] = make_uint4(wb[0], wb[1], wb[2], wb[3]);
      q[1] = make_uint4(wb[4], wb[5], wb[6], wb[7]);
      a.masks[blk] = (unsigned short)mask;
    }
    unsigned cnt = (unsigned)__popc(mask);
#pragma unroll
    for (int o = 16; o; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
    if ((tid & 31) == 0 && cnt) atomicAdd(&s_cnt, cnt);
    __syncthreads();
    if (tid == 0) a.tile_sums[tile] = s_cnt;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(STB) opq_write_kernel(OpqArgs a) {
  __shared__ unsigned s_warp[STB / 32];
  const int tid = threadIdx.x;
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long blk = tile * STB + tid;
    const unsigned mask = blk < a.NB ? (unsigned)a.masks[blk] : 0u;
    unsigned tot;
    const unsigned excl = cta_excl_scan((unsigned)__popc(mask), s_warp, &tot);
    if (blk >= a.NB) continue;
    unsigned pos = a.tile_sums[tile] + excl;
    const long long m = (long long)((unsigned)blk / (unsigned)a.nbk), j = blk - m * a.nbk;   // the block count fits 31 bits
    if (j == 0) a.row_start[m] = pos;
    if (mask) {
      const uint16_t* p = a.W + m * a.ldw + j * SOP_G;
      for (unsigned rest = mask; rest; rest &= rest - 1u) {
        const int i = __ffs((int)rest) - 1;
        if ((long long)pos < a.capacity) a.records[pos] = (unsigned)(j * SOP_G + i) | ((unsigned)p[i] << 16);
        ++pos;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Wr
// ---------------------------------------------------------------------------------------------
struct WrArgs {
  const uint16_t* W;
  const float* c;
  long long M, K, ldw, nbk, NB;
  int index_a, index_b, k_mode, use_sign;
  int container_bits, word_sign_bits, meta_bits;
  const unsigned char* codes;
  const unsigned* words;
  long long n_keep;
  unsigned* tile_sums;
  unsigned* row_start;
  unsigned* records;
  long long capacity;
  unsigned short* kept;           // workspace: per block the 16-bit mask of kept entries (candidate path)
  unsigned* cand_pos;             // workspace: candidate list: element position blk * 16 + i,
  unsigned* cand_e;               //   residual bits,
  unsigned* cand_m;               //   metric bits
  unsigned cand_cap;
};

struct WrCand { int kind, neg, scope, k, sign_pos, y, bias; float tmax; };

// what a CTA needs to decode the stream: the (up to two) tables and their atoms' parameters
struct WrShared {
  float lutv[2][32];
  WrCand cand[2];
  float pot[2];
  int n_bits;
  int no_pair;
};

// value of the code sign | E | M of a floating-point element grid with y mantissa bits and the given bias
__device__ __forceinline__ float fp_grid_decode(uint32_t code, int sign_pos, int y, int bias) {
  const uint32_t mag = code & ((1u << sign_pos) - 1u);
  const uint32_t E = mag >> y, Mm = mag & ((1u << y) - 1u);
  const float v = ldexp_once(E ? ((1u << y) + Mm) : Mm, (int)(E ? E : 1u) - bias - y);
  return ((code >> sign_pos) & 1u) ? -v : v;
}

// the scale a scale code stands for: the tail of scale_quantize
__device__ __forceinline__ float scale_decode(uint32_t code, int k, const FmtDev& f) {
  const int E = (int)(code >> f.y);
  const uint32_t Mm = code & ((1u << f.y) - 1u);
  const uint32_t mant = E ? ((1u << f.y) + Mm) : Mm;
  return mant ? ldexp_once(mant, (E ? E : 1) - f.bias - f.y - k) : 0.0f;
}

// thread 0 of every CTA; the caller synchronises afterwards
__device__ void wr_setup(const WrArgs& a, const AtomsDev& A, const sop_search_result* __restrict__ res, WrShared& sh) {
  int ia = a.index_a, ib = a.index_b;
  const bool from_result = ia == SOP_PAIR_FROM_RESULT;
  if (from_result) {
    ia = a.use_sign ? res->best_sa : res->best_a;
    ib = a.use_sign ? res->best_sb : res->best_b;
  }
  // a result without a pair: the packer wrote nothing, so there is nothing to correct
  sh.no_pair = from_result && (ia < 0 || ib < 0 || ia >= A.n_atoms || ib >= A.n_atoms ||
                               (a.use_sign && (ia + 1 >= A.n_atoms || ib + 1 >= A.n_atoms))) ? 1 : 0;
  ia = max(0, min(A.n_atoms - 1, ia));
  int nb = 1;
  if (ib != SOP_NO_ATOM) { ib = max(0, min(A.n_atoms - 1, ib)); nb = 2; }
  sh.n_bits = A.atoms[ia].n_bits;
  const float wmax = res ? res->layer_absmax : 0.0f;
  for (int t = 0; t < nb; ++t) {
    const int idx = t ? ib : ia;
    const sop_atom& at = A.atoms[idx];
    WrCand cd;
    cd.kind = at.kind; cd.neg = at.negated; cd.scope = at.scope; cd.tmax = at.tmax;
    cd.k = a.k_mode == SOP_K_FROM_RESULT ? res->k[idx] : a.k_mode;
    if (at.kind == SOP_KIND_FP_E2M3) { cd.sign_pos = 5; cd.y = 3; cd.bias = 1; }
    else if (at.kind == SOP_KIND_FP_E4M3) { cd.sign_pos = 7; cd.y = 3; cd.bias = 7; }
    else { cd.sign_pos = at.grid_exp_bits + at.grid_man_bits; cd.y = at.grid_man_bits; cd.bias = at.grid_bias; }
    sh.cand[t] = cd;
    sh.pot[t] = at.scope == 0 ? layer_pot_scale(wmax, at.tmax) : 0.0f;
    const bool dd = (A.dd_mask >> idx) & 1u;
    const int ne = at.kind == SOP_KIND_LUT ? at.n_entries : 1;
    for (int j = 0; j < 32; ++j) sh.lutv[t][j] = at.kind == SOP_KIND_LUT ? (dd ? A.dd_lut[min(j, ne - 1)] : at.lut[min(j, ne - 1)]) : 0.0f;
  }
}

// One block of the packed layer: the residual E_i = w_i - s_hat q_i (one rounding) and the metric |E_i| c_k.
// LUT4: both codebooks are tables of at most 16 entries (the common case): constant shifts, no kind test per element.
template <bool LUT4>
__device__ __forceinline__ void wr_block(const WrArgs& a, const FmtDev& F, const WrShared& sh, long long blk, long long j,
                                         const uint16_t* __restrict__ wrow, float (&E)[16], float (&met)[16]) {
  const uint4* p = reinterpret_cast<const uint4*>(wrow);
  const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
  const uint32_t wb[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
  const int n = LUT4 ? 4 : sh.n_bits, b = a.container_bits;
  // the 16n-bit payload as one little-endian integer
  unsigned long long lo = 0, hi = 0;
  const unsigned char* cp = a.codes + (size_t)blk * 2 * n;
  if (n == 4) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(cp));
    lo = (unsigned long long)t.x | ((unsigned long long)t.y << 32);
  } else if (n == 8) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(cp));
    lo = (unsigned long long)t.x | ((unsigned long long)t.y << 32);
    hi = (unsigned long long)t.z | ((unsigned long long)t.w << 32);
  } else {
    const unsigned short* sp = reinterpret_cast<const unsigned short*>(cp);
    for (int i = 0; i < n; ++i) {
      const unsigned long long v = (unsigned long long)__ldg(sp + i);
      if (i < 4) lo |= v << (16 * i); else hi |= v << (16 * (i - 4));
    }
  }
  // the scale word: sign, scale code, selector
  unsigned word;
  if (b == 16) word = (unsigned)__ldg(reinterpret_cast<const unsigned short*>(a.words) + blk);
  else if (b == 8) word = (unsigned)__ldg(reinterpret_cast<const unsigned char*>(a.words) + blk);
  else {
    const long long bit = blk * b;
    const long long wi = bit >> 5;
    const int s = (int)(bit & 31);
    word = __ldg(a.words + wi) >> s;
    if (s + b > 32) word |= __ldg(a.words + wi + 1) << (32 - s);
    word &= (1u << b) - 1u;
  }
  unsigned sgn = 0, sel = 0, scode;
  const unsigned cmask = (1u << (b - a.word_sign_bits - a.meta_bits)) - 1u;
  if (a.word_sign_bits) { sgn = word >> (b - 1); scode = (word >> a.meta_bits) & cmask; sel = a.meta_bits >= 1 ? (word & 1u) : 0u; }
  else if (a.meta_bits >= 1) { sel = word >> (b - 1); scode = (word >> (a.meta_bits - 1)) & cmask; }
  else scode = word & cmask;
  if (a.index_b == SOP_NO_ATOM) sel = 0;
  const WrCand cd = sh.cand[sel];
  float s_hat;
  if (cd.scope == 0) {
    uint32_t mb = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) { mb = max(mb, wb[q] & 0x7FFFu); mb = max(mb, (wb[q] >> 16) & 0x7FFFu); }
    s_hat = mb ? sh.pot[sel] : 0.0f;
  } else {
    s_hat = scale_decode(scode, cd.k, F);
  }
  const int neg = sgn ? 1 - cd.neg : cd.neg;
  const unsigned emask = (1u << n) - 1u;
  const float4* cq = reinterpret_cast<const float4*>(a.c + j * SOP_G);
  float c[16];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = __ldg(cq + q);
    c[4 * q] = v.x; c[4 * q + 1] = v.y; c[4 * q + 2] = v.z; c[4 * q + 3] = v.w;
  }
  const uint32_t lo32[2] = {(uint32_t)lo, (uint32_t)(lo >> 32)};
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    uint32_t code;
    if (LUT4 || n == 4) {             // the common width: 32-bit shifts by constants
      code = (lo32[i >> 3] >> (4 * (i & 7))) & 15u;
    } else {
      const int pos = i * n;
      unsigned long long v;
      if (pos < 64) { v = lo >> pos; if (pos + n > 64) v |= hi << (64 - pos); }
      else v = hi >> (pos - 64);
      code = (uint32_t)v & emask;
    }
    float q;
    if (LUT4 || cd.kind == SOP_KIND_LUT) { q = sh.lutv[sel][code & 31u]; q = neg ? -q : q; }
    else q = fp_grid_decode(code, cd.sign_pos, cd.y, cd.bias);
    const float w = (i & 1) ? bf16hi(wb[i >> 1]) : bf16lo(wb[i >> 1]);
    E[i] = __fmaf_rn(-s_hat, q, w);
    met[i] = __fmul_rn(fabsf(E[i]), c[i]);
  }
}

// the metric as a key whose ascending order is the metric's descending order (the metric is never negative;
// a NaN counts as zero)
__device__ __forceinline__ unsigned wr_key(float met) {
  return ~(met > 0.0f ? __float_as_uint(met) : 0u);
}

template <int PASS, bool LUT4>
__global__ void __launch_bounds__(STB) wr_hist_kernel(WrArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res,
                                                      SparseWs* __restrict__ ws) {
  __shared__ WrShared sh;
  __shared__ unsigned hist[2048];
  const int tid = threadIdx.x;
  if (PASS >= 0 && !ws->overflow) return;          // the candidate list serves the selection
  for (int i = tid; i < 2048; i += STB) hist[i] = 0;
  if (tid == 0) wr_setup(a, A, res, sh);
  __syncthreads();
  if (sh.no_pair) return;
  const unsigned prefix = PASS > 0 ? ws->prefix : 0u;
  const unsigned bm_bin = PASS == 0 ? ws->bm_bin : 2047u;
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long blk = tile * STB + tid;
    if (blk >= a.NB) continue;
    const long long m = (long long)((unsigned)blk / (unsigned)a.nbk), j = blk - m * a.nbk;   // the block count fits 31 bits
    float E[16], met[16];
    wr_block<LUT4>(a, F, sh, blk, j, a.W + m * a.ldw + j * SOP_G, E, met);
    if constexpr (PASS < 0) {
      float bm = 0.0f;
#pragma unroll
      for (int i = 0; i < 16; ++i) bm = fmaxf(bm, met[i]);             // fmaxf drops a NaN
      // most blocks share a handful of bins: one addition per distinct bin of the warp
      const unsigned bin = wr_key(bm) >> 21;
      const unsigned same = __match_any_sync(__activemask(), bin);
      if ((__ffs((int)same) - 1) == (tid & 31)) atomicAdd(&hist[bin], (unsigned)__popc(same));
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const unsigned key = wr_key(met[i]);
        if (PASS == 0) {
          if ((key >> 21) <= bm_bin) atomicAdd(&hist[key >> 21], 1u);
        } else if (PASS == 1) {
          if ((key >> 21) == prefix) atomicAdd(&hist[(key >> 10) & 2047u], 1u);
        } else {
          if ((key >> 10) == prefix) atomicAdd(&hist[key & 1023u], 1u);
        }
      }
    }
  }
  __syncthreads();
  unsigned* out = PASS < 0 ? ws->hist_bm : ws->hist[PASS < 0 ? 0 : PASS];
  for (int i = tid; i < 2048; i += STB)
    if (hist[i]) atomicAdd(&out[i], hist[i]);
}

// One CTA after each histogram pass: the bin that holds the rank, the prefix and the rank inside it for the next
// pass; after the last pass the threshold itself.  Pass -1: the bin of the n_keep-th largest block maximum.  A rank
// beyond the histogram's total (no pair to correct, so the histogram is empty) leaves a NaN threshold: nothing
// compares >= to it.
__global__ void __launch_bounds__(1024) wr_pick_kernel(SparseWs* __restrict__ ws, int pass, long long n_keep) {
  __shared__ unsigned long long s_warp[32];
  __shared__ int s_bin;
  __shared__ unsigned long long s_before;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nb = pass < 2 ? 2048 : 1024;
  const unsigned long long rank = pass <= 0 ? (unsigned long long)n_keep : ws->rank;
  if (tid == 0) { s_bin = -1; s_before = 0; }
  const int b0 = 2 * tid;
  const unsigned* h = pass < 0 ? ws->hist_bm : ws->hist[pass];
  const unsigned long long c0 = b0 < nb ? h[b0] : 0ull, c1 = b0 + 1 < nb ? h[b0 + 1] : 0ull;
  const unsigned long long local = c0 + c1;
  unsigned long long incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  unsigned long long base = 0;
  for (int w = 0; w < warp; ++w) base += s_warp[w];
  const unsigned long long excl = base + incl - local;
  if (local && excl < rank && rank <= excl + local) {
    if (rank <= excl + c0) { s_bin = b0; s_before = excl; }
    else { s_bin = b0 + 1; s_before = excl + c0; }
  }
  __syncthreads();
  if (tid == 0 && pass < 0) {
    // fewer blocks than entries to keep: no bound, every bin counts
    ws->bm_bin = s_bin < 0 ? 2047u : (unsigned)s_bin;
  } else if (tid == 0) {
    const unsigned prev = pass ? ws->prefix : 0u;
    if (s_bin < 0) {
      ws->prefix = 0xFFFFFFFFu; ws->rank = 0; ws->tau_bits = 0x7FC00000u;
    } else {
      const unsigned pre = (prev << (pass < 2 ? 11 : 10)) | (unsigned)s_bin;
      ws->prefix = pre;
      ws->rank = rank - s_before;
      if (pass == 2) ws->tau_bits = ~pre;
    }
  }
}

__device__ __forceinline__ bool wr_kept(float met, float tau) { return met >= tau && met > 0.0f; }

// The stored value of a residual: the E3M4 code (bias 3, 4 mantissa bits, largest 15.5) of E / 2^e.  The quotient is
// formed by two exact multiplications by powers of two (|E| / 2^e <= 15.5; a quotient below the fp32 normal range is
// far below half the smallest E3M4 step and rounds to zero either way).
struct WrValue {
  float f1, f2;
  GridDev g;
  __device__ explicit WrValue(int e) {
    const int e1 = max(-100, min(100, -e));
    f1 = pow2f_int(e1); f2 = pow2f_int(max(-120, min(120, -e - e1)));
    g.min_eb = 125; g.sh = 19; g.vpos = 15.5f; g.vneg = 15.5f;
  }
  __device__ __forceinline__ uint32_t code(float E) const {
    return grid_code(grid_quantize(__fmul_rn(__fmul_rn(E, f1), f2), g), g, 7);
  }
};

// Second decode pass: the candidates.  A thread counts its block's candidates, the warp reserves room for all of them
// with one addition to the list's counter, every thread writes its own.  Beyond the capacity nothing is written; the
// counter keeps counting, which is how the overflow is seen.
template <bool LUT4>
__global__ void __launch_bounds__(STB) wr_collect_kernel(WrArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res,
                                                         SparseWs* __restrict__ ws) {
  __shared__ WrShared sh;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) wr_setup(a, A, res, sh);
  __syncthreads();
  if (blockIdx.x == 0 && tid == 0) ws->no_pair = sh.no_pair;
  if (sh.no_pair) return;
  const unsigned bm_bin = ws->bm_bin;
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long blk = tile * STB + tid;
    float E[16], met[16];
    unsigned in = 0;
    if (blk < a.NB) {
      const long long m = (long long)((unsigned)blk / (unsigned)a.nbk), j = blk - m * a.nbk;
      wr_block<LUT4>(a, F, sh, blk, j, a.W + m * a.ldw + j * SOP_G, E, met);
      float bm = 0.0f;
#pragma unroll
      for (int i = 0; i < 16; ++i) bm = fmaxf(bm, met[i]);
      if ((wr_key(bm) >> 21) <= bm_bin) {            // few blocks reach the bound at all
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if ((wr_key(met[i]) >> 21) <= bm_bin) in |= 1u << i;
      }
    }
    if (!__any_sync(0xFFFFFFFFu, in != 0u)) continue;
    const unsigned mine = (unsigned)__popc(in);
    unsigned incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    const unsigned total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    unsigned base = 0;
    if (lane == 31 && total) base = atomicAdd(&ws->n_cand, total);
    base = __shfl_sync(0xFFFFFFFFu, base, 31);
    unsigned at = base + incl - mine;
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if ((in >> i) & 1u) {
        if (at < a.cand_cap) {
          a.cand_pos[at] = (unsigned)blk * 16u + (unsigned)i;
          a.cand_e[at] = __float_as_uint(E[i]);
          a.cand_m[at] = __float_as_uint(met[i]);
        }
        ++at;
      }
  }
}

__global__ void wr_mode_kernel(SparseWs* __restrict__ ws, unsigned cand_cap) {
  if (threadIdx.x == 0 && blockIdx.x == 0) ws->overflow = ws->n_cand > cand_cap ? 1u : 0u;
}

// The selection passes over the candidate list instead of the layer.
template <int PASS>
__global__ void __launch_bounds__(STB) wr_cand_hist_kernel(WrArgs a, SparseWs* __restrict__ ws) {
  __shared__ unsigned hist[2048];
  if (ws->overflow) return;
  const int tid = threadIdx.x;
  for (int i = tid; i < 2048; i += STB) hist[i] = 0;
  __syncthreads();
  const unsigned n = ws->n_cand, prefix = PASS > 0 ? ws->prefix : 0u;
  for (unsigned i = blockIdx.x * STB + tid; i < n; i += gridDim.x * STB) {
    const unsigned key = wr_key(__uint_as_float(a.cand_m[i]));
    if (PASS == 0) atomicAdd(&hist[key >> 21], 1u);
    else if (PASS == 1) { if ((key >> 21) == prefix) atomicAdd(&hist[(key >> 10) & 2047u], 1u); }
    else { if ((key >> 10) == prefix) atomicAdd(&hist[key & 1023u], 1u); }
  }
  __syncthreads();
  for (int i = tid; i < 2048; i += STB)
    if (hist[i]) atomicAdd(&ws->hist[PASS][i], hist[i]);
}

// The kept candidates: their bit in the per-block masks (two blocks per 32-bit word), their tile's record count (cleared
// by the host call), the largest |E| among them.
__global__ void __launch_bounds__(STB) wr_mark_kernel(WrArgs a, SparseWs* __restrict__ ws) {
  if (ws->overflow) return;
  const float tau = __uint_as_float(ws->tau_bits);
  const unsigned n = ws->n_cand;
  unsigned emax = 0;
  unsigned* map = reinterpret_cast<unsigned*>(a.kept);
  for (unsigned i = blockIdx.x * STB + threadIdx.x; i < n; i += gridDim.x * STB) {
    if (!wr_kept(__uint_as_float(a.cand_m[i]), tau)) continue;
    const unsigned pos = a.cand_pos[i];
    atomicOr(&map[pos >> 5], 1u << (pos & 31u));
    atomicAdd(&a.tile_sums[pos >> 12], 1u);          // a tile is 256 blocks of 16 elements
    emax = max(emax, a.cand_e[i] & 0x7FFFFFFFu);
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, o));
  if ((threadIdx.x & 31) == 0 && emax) atomicMax(&ws->emax_bits, emax);
}

template <bool LUT4>
__global__ void __launch_bounds__(STB) wr_count_kernel(WrArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res,
                                                       SparseWs* __restrict__ ws) {
  __shared__ WrShared sh;
  __shared__ unsigned s_cnt;
  const int tid = threadIdx.x;
  if (!ws->overflow) return;
  if (tid == 0) wr_setup(a, A, res, sh);
  __syncthreads();
  const float tau = __uint_as_float(ws->tau_bits);
  const long long n_tiles = (a.NB + STB - 1) / STB;
  unsigned emax = 0;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    const long long blk = tile * STB + tid;
    unsigned cnt = 0;
    if (blk < a.NB && !sh.no_pair) {
      const long long m = (long long)((unsigned)blk / (unsigned)a.nbk), j = blk - m * a.nbk;   // the block count fits 31 bits
      float E[16], met[16];
      wr_block<LUT4>(a, F, sh, blk, j, a.W + m * a.ldw + j * SOP_G, E, met);
#pragma unroll
      for (int i = 0; i < 16; ++i)
        if (wr_kept(met[i], tau)) { ++cnt; emax = max(emax, __float_as_uint(fabsf(E[i]))); }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
    if ((tid & 31) == 0 && cnt) atomicAdd(&s_cnt, cnt);
    __syncthreads();
    if (tid == 0) a.tile_sums[tile] = s_cnt;
    __syncthreads();
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, o));
  if ((tid & 31) == 0 && emax) atomicMax(&ws->emax_bits, emax);
}

// The full-decode write pass: every block is decoded and its entries are compared with the threshold.
template <bool LUT4>
__global__ void __launch_bounds__(STB) wr_write_kernel(WrArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res,
                                                       const SparseWs* __restrict__ ws) {
  __shared__ WrShared sh;
  __shared__ unsigned s_warp[STB / 32];
  const int tid = threadIdx.x;
  if (!ws->overflow) return;
  if (tid == 0) wr_setup(a, A, res, sh);
  __syncthreads();
  const float tau = __uint_as_float(ws->tau_bits);
  const WrValue V(ws->scale_exp);
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long blk = tile * STB + tid;
    float E[16], met[16];
    unsigned keep = 0;
    long long m = 0, j = 0;
    if (blk < a.NB) {
      m = (long long)((unsigned)blk / (unsigned)a.nbk); j = blk - m * a.nbk;
      if (!sh.no_pair) {
        wr_block<LUT4>(a, F, sh, blk, j, a.W + m * a.ldw + j * SOP_G, E, met);
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (wr_kept(met[i], tau)) keep |= 1u << i;
      }
    }
    unsigned tot;
    const unsigned excl = cta_excl_scan((unsigned)__popc(keep), s_warp, &tot);
    if (blk >= a.NB) continue;
    unsigned pos = a.tile_sums[tile] + excl;
    if (j == 0) a.row_start[m] = pos;
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if ((keep >> i) & 1u) {
        if ((long long)pos < a.capacity) a.records[pos] = (unsigned)(j * SOP_G + i) | (V.code(E[i]) << 16);
        ++pos;
      }
  }
}

// The write pass of the candidate path: the kept entries come from the per-block masks.  Every thread scans its
// block's count; the few blocks of a tile that hold a kept entry are put on a list in shared memory and decoded by the
// first threads of the CTA, so that a warp does not run a decode for one lane.
template <bool LUT4>
__global__ void __launch_bounds__(STB) wr_map_write_kernel(WrArgs a, AtomsDev A, FmtDev F, const sop_search_result* __restrict__ res,
                                                           const SparseWs* __restrict__ ws) {
  __shared__ WrShared sh;
  __shared__ unsigned s_warp[STB / 32];
  __shared__ unsigned s_n;
  __shared__ unsigned s_pos[STB];          // per listed block: its first record
  __shared__ unsigned short s_blk[STB], s_keep[STB];
  const int tid = threadIdx.x;
  if (ws->overflow) return;
  if (tid == 0) { wr_setup(a, A, res, sh); s_n = 0; }
  __syncthreads();
  const WrValue V(ws->scale_exp);
  const long long n_tiles = (a.NB + STB - 1) / STB;
  for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const long long blk = tile * STB + tid;
    const unsigned keep = blk < a.NB && !sh.no_pair ? (unsigned)a.kept[blk] : 0u;
    unsigned tot;
    const unsigned excl = cta_excl_scan((unsigned)__popc(keep), s_warp, &tot);        // (two barriers)
    if (blk < a.NB) {
      const unsigned pos = a.tile_sums[tile] + excl;
      const long long m = (long long)((unsigned)blk / (unsigned)a.nbk);
      if (blk - m * a.nbk == 0) a.row_start[m] = pos;
      if (keep) {
        const unsigned at = atomicAdd(&s_n, 1u);
        s_pos[at] = pos; s_blk[at] = (unsigned short)tid; s_keep[at] = (unsigned short)keep;
      }
    }
    __syncthreads();
    const unsigned n = s_n;
    for (unsigned q = tid; q < n; q += STB) {
      const long long b = tile * STB + s_blk[q];
      const long long m = (long long)((unsigned)b / (unsigned)a.nbk), j = b - m * a.nbk;
      float E[16], met[16];
      wr_block<LUT4>(a, F, sh, b, j, a.W + m * a.ldw + j * SOP_G, E, met);
      unsigned pos = s_pos[q];
      const unsigned k = s_keep[q];
#pragma unroll
      for (int i = 0; i < 16; ++i)
        if ((k >> i) & 1u) {
          if ((long long)pos < a.capacity) a.records[pos] = (unsigned)(j * SOP_G + i) | (V.code(E[i]) << 16);
          ++pos;
        }
    }
    __syncthreads();
    if (tid == 0) s_n = 0;                  // read again only after the next tile's scan barriers
  }
}

}  // namespace sop

extern "C" {

int sop_opq_threshold(double q, int max_order, double* m_out) {
  if (!m_out) return SOP_ERR_NULL;
  if (!(q > 0.0 && q < 1.0) || max_order < 1) return SOP_ERR_RANGE;
  // (2 Phi(m) - 1)^M = q with 2 Phi(m) - 1 = erf(m / sqrt 2): solve erf(m / sqrt 2) = q^(1/M) by bisection
  const double target = exp(log(q) / (double)max_order);
  double lo = 0.0, hi = 16.0;
  for (int it = 0; it < 128; ++it) {
    const double mid = 0.5 * (lo + hi);
    if (erf(mid * 0.70710678118654752440) < target) lo = mid; else hi = mid;
  }
  *m_out = 0.5 * (lo + hi);
  return SOP_OK;
}

int sop_opq_workspace(long long M, long long K, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (M < 1 || K < 1 || (K % SOP_G) != 0 || M > (1ll << 31) / (K / SOP_G)) return SOP_ERR_SHAPE;
  const long long NB = M * (K / SOP_G);
  *bytes = sop::sparse_masks_off(NB) + (((size_t)NB * 2 + 255) & ~(size_t)255);
  return SOP_OK;
}

int sop_opq_extract(const void* W_dev, long long M, long long K, long long ldw, int g, double m,
                    void* W_out_dev, long long ldo, unsigned* row_start_dev, unsigned* records_dev, long long capacity,
                    long long* count_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
  using namespace sop;
  if (!W_dev || !W_out_dev || !row_start_dev || !count_dev) return SOP_ERR_NULL;
  if (g != SOP_G || M < 1 || K < 1 || (K % SOP_G) != 0 || ldw < K || (ldw % 8) != 0 || ldo < K || (ldo % 8) != 0) return SOP_ERR_SHAPE;
  if (((uintptr_t)W_dev & 15u) || ((uintptr_t)W_out_dev & 15u)) return SOP_ERR_SHAPE;
  if (M > (1ll << 31) / (K / SOP_G) || K > 65536) return SOP_ERR_SHAPE;       // the record holds the column in 16 bits
  if (W_out_dev == W_dev) return SOP_ERR_RANGE;                               // the stream is written from the untouched input
  if (!(m > 0.0) || !(m < 1.0e6)) return SOP_ERR_RANGE;
  if (capacity < 0 || (capacity > 0 && !records_dev)) return SOP_ERR_NULL;
  size_t need = 0;
  sop_opq_workspace(M, K, &need);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;
  OpqArgs a;
  a.W = (const uint16_t*)W_dev; a.W_out = (uint16_t*)W_out_dev; a.M = M; a.K = K; a.ldw = ldw; a.ldo = ldo;
  a.nbk = K / SOP_G; a.NB = M * a.nbk; a.m2 = m * m;
  unsigned char* wsb = (unsigned char*)workspace_dev;
  a.tile_sums = (unsigned*)(wsb + sparse_tiles_off());
  a.masks = (unsigned short*)(wsb + sparse_masks_off(a.NB));
  a.row_start = row_start_dev; a.records = records_dev; a.capacity = capacity;
  cudaStream_t st = (cudaStream_t)stream;
  const long long n_tiles = sparse_tiles(a.NB);
  const long long cap = (long long)num_sms() * 8;
  const int grid = (int)(n_tiles < cap ? n_tiles : cap);
  int rc;
  if ((rc = profile_mark(SOP_PROFILE_OPQ, 0, st))) return rc;
  opq_mask_kernel<<<grid, STB, 0, st>>>(a);
  tile_scan_kernel<<<1, 1024, 0, st>>>(a.tile_sums, n_tiles, row_start_dev, M, count_dev, (SparseWs*)workspace_dev, 0, nullptr, nullptr);
  opq_write_kernel<<<grid, STB, 0, st>>>(a);
  SOP_CUDA_TRY(cudaGetLastError());
  if ((rc = profile_mark(SOP_PROFILE_OPQ, 1, st))) return rc;
  return SOP_OK;
}

int sop_wr_workspace(long long M, long long K, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (M < 1 || K < 1 || (K % SOP_G) != 0 || M > (1ll << 31) / (K / SOP_G)) return SOP_ERR_SHAPE;
  const long long NB = M * (K / SOP_G);
  *bytes = sop::wr_cand_off(NB) + 3 * (((size_t)sop::wr_cand_cap(NB) * 4 + 255) & ~(size_t)255);
  return SOP_OK;
}

int sop_wr_extract(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                   const sop_scale_fmt* fmt, const sop_atom* atoms, int n_atoms, const float* dd_lut_dev, unsigned dd_mask,
                   int index_a, int index_b, int k_mode, const sop_search_result* search_dev, int use_sign,
                   int container_bits, int word_sign_bits, const unsigned char* codes_dev, const unsigned char* words_dev,
                   long long n_keep, unsigned* row_start_dev, unsigned* records_dev, long long capacity,
                   long long* count_dev, int* scale_exp_dev, float* tau_dev, void* workspace_dev, size_t workspace_bytes,
                   void* stream) {
  using namespace sop;
  int rc = validate_layer(W_dev, M, K, ldw, c_dev, g);
  if (rc) return rc;
  if (!codes_dev || !words_dev || !row_start_dev || !count_dev || !scale_exp_dev) return SOP_ERR_NULL;
  if (K > 65536) return SOP_ERR_SHAPE;                                        // the record holds the column in 16 bits
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
    if (atoms[index_a].kind == SOP_KIND_FP_GRID && (atoms[index_a].grid_exp_bits < 1 || atoms[index_a].n_bits > 8)) return SOP_ERR_ALPHABET;
  }
  if (index_b != SOP_NO_ATOM && meta < 1) return SOP_ERR_FORMAT;
  if (k_mode == SOP_K_FROM_RESULT) { if (!search_dev) return SOP_ERR_NULL; }
  else if (k_mode < -64 || k_mode > 64) return SOP_ERR_RANGE;
  bool need_wmax = false;
  for (int i = 0; i < n_atoms; ++i) need_wmax |= atoms[i].scope == 0;
  if (need_wmax && !search_dev) return SOP_ERR_NULL;
  if (((uintptr_t)codes_dev & 15u) || ((uintptr_t)words_dev & 3u)) return SOP_ERR_SHAPE;
  if (from_result) {
    int n_bits = 0;
    for (int i = 0; i < n_atoms; ++i)
      if (atoms[i].kind == SOP_KIND_LUT) { if (!n_bits) n_bits = atoms[i].n_bits; else if (atoms[i].n_bits != n_bits) return SOP_ERR_ALPHABET; }
    if (!n_bits) return SOP_ERR_ALPHABET;
  }
  if (n_keep < 1 || n_keep > M * K) return SOP_ERR_RANGE;
  if (capacity < 0 || (capacity > 0 && !records_dev)) return SOP_ERR_NULL;
  size_t need = 0;
  sop_wr_workspace(M, K, &need);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;

  WrArgs a;
  a.W = (const uint16_t*)W_dev; a.c = c_dev; a.M = M; a.K = K; a.ldw = ldw; a.nbk = K / SOP_G; a.NB = M * a.nbk;
  a.index_a = index_a; a.index_b = index_b; a.k_mode = k_mode; a.use_sign = use_sign;
  a.container_bits = container_bits; a.word_sign_bits = word_sign_bits; a.meta_bits = meta;
  a.codes = codes_dev; a.words = (const unsigned*)words_dev; a.n_keep = n_keep;
  unsigned char* wsb = (unsigned char*)workspace_dev;
  SparseWs* ws = (SparseWs*)workspace_dev;
  a.tile_sums = (unsigned*)(wsb + sparse_tiles_off());
  a.row_start = row_start_dev; a.records = records_dev; a.capacity = capacity;
  a.kept = (unsigned short*)(wsb + sparse_masks_off(a.NB));
  a.cand_cap = wr_cand_cap(a.NB);
  {
    const size_t one = ((size_t)a.cand_cap * 4 + 255) & ~(size_t)255;
    a.cand_pos = (unsigned*)(wsb + wr_cand_off(a.NB));
    a.cand_e = (unsigned*)(wsb + wr_cand_off(a.NB) + one);
    a.cand_m = (unsigned*)(wsb + wr_cand_off(a.NB) + 2 * one);
  }
  cudaStream_t st = (cudaStream_t)stream;
  const long long n_tiles = sparse_tiles(a.NB);
  const long long cap = (long long)num_sms() * 6;
  const int lgrid = num_sms() * 2;                       // the kernels over the candidate list
  SOP_CUDA_TRY(cudaMemsetAsync(a.kept, 0, ((size_t)a.NB * 2 + 3) & ~(size_t)3, st));
  SOP_CUDA_TRY(cudaMemsetAsync(a.tile_sums, 0, (size_t)n_tiles * 4, st));
  const int grid = (int)(n_tiles < cap ? n_tiles : cap);
  SOP_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(SparseWs), st));
  if ((rc = profile_mark(SOP_PROFILE_WR, 0, st))) return rc;
  // both codebooks tables of at most 16 entries: the decode with constant shifts (a pair taken from a search result is
  // always a pair of tables, and n_bits is then the alphabet's)
  bool lut4 = true;
  if (from_result) {
    for (int i = 0; i < n_atoms; ++i)
      if (atoms[i].kind == SOP_KIND_LUT && atoms[i].n_bits != 4) lut4 = false;
  } else {
    lut4 = atoms[index_a].kind == SOP_KIND_LUT && atoms[index_a].n_bits == 4 &&
           (index_b == SOP_NO_ATOM || (atoms[index_b].kind == SOP_KIND_LUT && atoms[index_b].n_bits == 4));
  }
#define SOP_WR_LAUNCHES(L4)                                                          \
  do {                                                                               \
    wr_hist_kernel<-1, L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);           \
    wr_pick_kernel<<<1, 1024, 0, st>>>(ws, -1, n_keep);                              \
    wr_collect_kernel<L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);            \
    wr_mode_kernel<<<1, 32, 0, st>>>(ws, a.cand_cap);                                \
    wr_cand_hist_kernel<0><<<lgrid, STB, 0, st>>>(a, ws);                            \
    wr_hist_kernel<0, L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);            \
    wr_pick_kernel<<<1, 1024, 0, st>>>(ws, 0, n_keep);                               \
    wr_cand_hist_kernel<1><<<lgrid, STB, 0, st>>>(a, ws);                            \
    wr_hist_kernel<1, L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);            \
    wr_pick_kernel<<<1, 1024, 0, st>>>(ws, 1, n_keep);                               \
    wr_cand_hist_kernel<2><<<lgrid, STB, 0, st>>>(a, ws);                            \
    wr_hist_kernel<2, L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);            \
    wr_pick_kernel<<<1, 1024, 0, st>>>(ws, 2, n_keep);                               \
    wr_mark_kernel<<<lgrid, STB, 0, st>>>(a, ws);                                    \
    wr_count_kernel<L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);              \
    tile_scan_kernel<<<1, 1024, 0, st>>>(a.tile_sums, n_tiles, row_start_dev, M, count_dev, ws, 1, scale_exp_dev, tau_dev); \
    wr_map_write_kernel<L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);          \
    wr_write_kernel<L4><<<grid, STB, 0, st>>>(a, A, F, search_dev, ws);              \
  } while (0)
  if (lut4) SOP_WR_LAUNCHES(true); else SOP_WR_LAUNCHES(false);
#undef SOP_WR_LAUNCHES
  SOP_CUDA_TRY(cudaGetLastError());
  if ((rc = profile_mark(SOP_PROFILE_WR, 1, st))) return rc;
  return SOP_OK;
}

}  // extern "C"
