// sop_pair_search: the per-layer candidate sweep.
//
//   prepass_kernel   reads W once: per-block absmax -> exponent histogram of sigma = absmax / tmax
//                    for every scale class that needs an F_layer search, and max|W|   (HBM-bound);
//                    the CTA that finishes last derives the F_layer shift k* per class from the
//                    histogram and the layer power-of-two scale for "^0" candidates.
//   kselect_kernel   that last step alone: the shifts of another scale format from the histogram a prepass of the
//                    same layer left in the workspace (SOP_SEARCH_REUSE_PREPASS).
//   sweep_kernel     persistent, one thread per 16-element block: evaluates every candidate of the call
//                    in registers (cell-table lookup of the reconstruction value, packed f32x2
//                    fused multiply-adds for the block metric, fixed quad-tree order) and writes
//                    the per-block cosine and squared error of each as one column.          (ALU-bound)
//   reduce_kernel    reads the columns of every candidate present in the call (those just written
//                    and those an earlier call wrote) tile by tile into shared memory and forms
//                    the table entries: a warp owns a few "tasks" (one anchor column against up to
//                    four partner columns, so five columns are fetched for up to five entries), a
//                    lane owns eight blocks of every tile, the sums of those eight are fp32 and go
//                    to FP64 accumulators after every tile (two tiles per step where the shared
//                    memory allows: the accumulators are then touched once per sixteen blocks).
//                    The CTA that finishes last adds the per-CTA partials in a fixed order
//                    (deterministic), writes the tables and picks the best pair / best single.
#include <math.h>
#include <string.h>

#include "sop_device.cuh"

namespace sop {

constexpr int TB = 512;             // threads per CTA of the sweep kernel
constexpr int MAX_SLOTS = 192;      // pair slots per call: 16 singles + 120 pairs + 36 signed < 192
constexpr int MAX_GRID = 1024;
constexpr float MAGIC = 12582912.0f;  // 1.5 * 2^23: adding it rounds to an integer in the low mantissa bits

struct CandDev { unsigned char cls, kind, neg, table; };
struct ClassDev {
  float tmax;
  float invh;        // cells per unit of u (a power of two)
  int scope, kind;   // kind of the quantiser: LUT, E2M3, E4M3
  int c_half;        // table rows = 2 * c_half + 1
  int auto_k;        // 1: k* from the histogram
  int n_cand;                            // candidates evaluated in this call
  unsigned char cand[SOP_MAX_ATOMS];
  int n_mem;                             // candidates present in this call (evaluated or loaded)
  unsigned char mem[SOP_MAX_ATOMS];
  int k_src;                             // candidate whose shift an earlier result holds (k from result), or -1
  GridDev grid;                          // kind SOP_KIND_FP_GRID: the grid's parameters
};
struct SlotDev { unsigned char type, i0, i1, pad; };  // type 0: pair (i0, i1) (i0 == i1: single); 1: signed (i0, i0+1, i1, i1+1)

// One unit of work of the reduction: an anchor candidate against up to four partners.  Entry q is the table slot
// slot[q] of the pair {anchor, part[q]}; rev = 0: the anchor is the first candidate of all its entries (it keeps a
// tie), rev = 1: it is the second one.  self_slot is the slot of the anchor alone (255: none).  sgn = 1: anchor and
// partners are base atoms and stand for the better of the atom and its negation (a signed four-way entry).
constexpr int TASK_PART = 4;
constexpr int MAX_TASKS = 96;
constexpr int MAX_TPW = 3;             // tasks per warp and launch
struct TaskDev {
  unsigned char anchor, n_part, self_slot, sgn, rev, pad[3];
  unsigned char part[TASK_PART], slot[TASK_PART];
};
// One launch of the reduction: per warp its tasks (255: empty seat) and the first accumulator seat of each; the
// candidates whose columns the launch fetches (col_slot: candidate -> column of the tile buffers, 255: not fetched)
// and the base atoms whose signed-best column it forms (sb_slot likewise).
struct SeatsDev {
  unsigned char task[8][MAX_TPW];
  unsigned short acc0[8][MAX_TPW];
  unsigned char col_slot[SOP_MAX_ATOMS], sb_slot[SOP_MAX_ATOMS];
  unsigned char cols[SOP_MAX_ATOMS], bases[SOP_MAX_ATOMS];      // the inverse lists
  int n_cols, n_bases, n_seats;
};

struct Plan {
  int n_atoms, n_classes, n_tables, n_slots, n_pair_slots;
  int k_mode, rows, a_pad;
  unsigned eval_mask, load_mask;   // candidates evaluated here / read from the per-block arrays of an earlier call
  int k_from_result;               // 1: shifts and max|W| come from the result block of an earlier call, no prepass
  int n_bases;                               // base atoms (each followed by its negation) of the signed table
  unsigned char base_atom[SOP_MAX_ATOMS];    // signed-best column n_atoms + b holds the better of base_atom[b] and its negation
  CandDev cand[SOP_MAX_ATOMS];
  ClassDev cls[SOP_MAX_CLASSES];
  unsigned char table_atom[SOP_MAX_TABLES];   // atom whose lut fills the table
  unsigned char table_cls[SOP_MAX_TABLES];
  unsigned char table_pos[SOP_MAX_TABLES];    // candidate that uses the table as it is (255: none)
  unsigned char table_neg[SOP_MAX_TABLES];    // candidate that uses the negated table (255: none)
  unsigned char cls_tables[SOP_MAX_CLASSES];  // bit t: table t belongs to the class
  SlotDev slots[MAX_SLOTS];
  int keep_loaded;                            // entries among loaded candidates stay as the tables hold them
  int n_tasks;
  TaskDev tasks[MAX_TASKS];
};

struct WsHeader {
  unsigned wmax_bits;
  int cls_k[SOP_MAX_CLASSES];
  float cls_pot[SOP_MAX_CLASSES];
  unsigned done_prepass, done_reduce;  // CTAs that have finished (the last one does the serial tail)
  int pad[5];
};
struct Partial { double gap, sse; long long n1, nneg; };

static size_t ws_hist_off() { return 256; }
// after the histograms: max|W| as the prepass found it (the header is cleared by every call, the histograms and this
// word stay until the next prepass)
static size_t ws_wmax_off() { return 256 + sizeof(unsigned) * SOP_MAX_CLASSES * SOP_HIST_BINS; }
static size_t ws_part_off() { return ws_wmax_off() + 256; }
static size_t ws_total() { return ((ws_part_off() + sizeof(Partial) * (size_t)MAX_GRID * MAX_SLOTS) + 255) & ~(size_t)255; }

struct LayerArgs {
  const uint16_t* W;
  const float* c;
  long long M, K, ldw;
  long long nbk;      // K / 16
  long long NB;       // M * nbk
};

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void load_block_bits(const uint16_t* p, uint32_t (&v)[8]) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
  const uint4 b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

__device__ __forceinline__ float absmax_bits(const uint32_t (&v)[8]) {
  // bf16 magnitudes order like their bit patterns: the maximum of the sixteen 15-bit patterns, two per word at a time
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) m = __vmaxu2(m, v[i] & 0x7FFF7FFFu);
  m = max(m & 0xFFFFu, m >> 16);
  return __uint_as_float(m << 16);
}

__device__ void kselect_body(const Plan& P, const FmtDev& F, const unsigned* hist, WsHeader* hdr);

__global__ void __launch_bounds__(256) prepass_kernel(LayerArgs L, Plan P, FmtDev F, unsigned* __restrict__ hist, WsHeader* __restrict__ hdr) {
  __shared__ unsigned sh[SOP_MAX_CLASSES * SOP_HIST_BINS];
  for (int i = threadIdx.x; i < P.n_classes * SOP_HIST_BINS; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  uint32_t wmax = 0;
  const unsigned nbk32 = (unsigned)L.nbk, NB32 = (unsigned)L.NB;         // the block count fits 31 bits
  for (unsigned b = blockIdx.x * blockDim.x + threadIdx.x; b < NB32; b += gridDim.x * blockDim.x) {
    const unsigned m = b / nbk32, j = b - m * nbk32;
    uint32_t v[8];
    load_block_bits(L.W + (long long)m * L.ldw + (long long)j * SOP_G, v);
    const float a = absmax_bits(v);
    wmax = max(wmax, __float_as_uint(a));
    if (a > 0.0f) {
      for (int cl = 0; cl < P.n_classes; ++cl) {
        if (!P.cls[cl].auto_k) continue;
        const float sigma = P.cls[cl].tmax == 1.0f ? a : __fdiv_rn(a, P.cls[cl].tmax);
        if (sigma > 0.0f) atomicAdd(&sh[cl * SOP_HIST_BINS + ilogb_pos(sigma) + SOP_HIST_OFF], 1u);
      }
    }
  }
  for (int o = 16; o; o >>= 1) wmax = max(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
  if ((threadIdx.x & 31) == 0) atomicMax(&hdr->wmax_bits, wmax);
  __syncthreads();
  for (int i = threadIdx.x; i < P.n_classes * SOP_HIST_BINS; i += blockDim.x)
    if (sh[i]) atomicAdd(&hist[i], sh[i]);
  // the CTA that arrives last turns the histogram into shifts; nobody waits for anybody
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&hdr->done_prepass, 1u) == gridDim.x - 1 ? 1 : 0;
  __syncthreads();
  if (s_last) {
    __threadfence();
    if (threadIdx.x == 0) hist[SOP_MAX_CLASSES * SOP_HIST_BINS] = __ldcg(&hdr->wmax_bits);    // kept for later calls on this layer
    kselect_body(P, F, hist, hdr);
  }
}

// The shifts of another scale format from the histograms that an earlier prepass of the same layer left in the workspace.
__global__ void __launch_bounds__(256) kselect_kernel(Plan P, FmtDev F, const unsigned* __restrict__ hist, WsHeader* __restrict__ hdr) {
  if (threadIdx.x == 0) hdr->wmax_bits = hist[SOP_MAX_CLASSES * SOP_HIST_BINS];
  __threadfence();
  __syncthreads();
  kselect_body(P, F, hist, hdr);
}

// One CTA of 256 threads.  Reads the global histogram and max|W| through the L2 (they were written by
// other CTAs' atomics).  Per class: prefix sums of the 320 bins, the count of every shift k in
// [-64, 64] as a difference of two prefix values, then the largest count with ties to the smallest |k|
// and then to k > 0 (preference order 0, +1, -1, +2, -2, ...).
__device__ void kselect_body(const Plan& P, const FmtDev& F, const unsigned* hist, WsHeader* hdr) {
  __shared__ unsigned long long pre[SOP_HIST_BINS + 1];
  __shared__ unsigned long long red_c[8];
  __shared__ int red_o[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float wmax = __uint_as_float(__ldcg(&hdr->wmax_bits));
  for (int cl = 0; cl < P.n_classes; ++cl) {
    int kstar = P.k_mode == SOP_K_AUTO ? 0 : P.k_mode;
    if (P.cls[cl].scope == 0) kstar = 0;
    if (P.cls[cl].auto_k) {
      // inclusive prefix of the bins: two bins per thread (320 <= 512), warp scan, warp totals
      unsigned long long v0 = 0, v1 = 0;
      if (2 * tid < SOP_HIST_BINS) v0 = __ldcg(&hist[cl * SOP_HIST_BINS + 2 * tid]);
      if (2 * tid + 1 < SOP_HIST_BINS) v1 = __ldcg(&hist[cl * SOP_HIST_BINS + 2 * tid + 1]);
      unsigned long long incl = v0 + v1;
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      __syncthreads();
      if (lane == 31) red_c[warp] = incl;
      __syncthreads();
      unsigned long long base = 0;
      for (int w = 0; w < warp; ++w) base += red_c[w];
      if (tid == 0) pre[0] = 0;
      if (2 * tid < SOP_HIST_BINS) pre[2 * tid + 1] = base + incl - v1;
      if (2 * tid + 1 < SOP_HIST_BINS) pre[2 * tid + 2] = base + incl;
      __syncthreads();
      // shift k = tid - 64 keeps the exponents e with emin <= e + k <= emax; bin of e is e + SOP_HIST_OFF
      unsigned long long c = 0;
      int order = 1 << 30;
      if (tid < 129) {
        const int k = tid - 64;
        const int lo = max(F.emin - k + SOP_HIST_OFF, 0), hi = min(F.emax - k + SOP_HIST_OFF, SOP_HIST_BINS - 1);
        c = hi >= lo ? pre[hi + 1] - pre[lo] : 0ull;
        order = k == 0 ? 0 : (k > 0 ? 2 * k - 1 : -2 * k);
      }
      for (int o = 16; o; o >>= 1) {
        const unsigned long long oc = __shfl_xor_sync(0xFFFFFFFFu, c, o);
        const int oo = __shfl_xor_sync(0xFFFFFFFFu, order, o);
        if (oc > c || (oc == c && oo < order)) { c = oc; order = oo; }
      }
      __syncthreads();
      if (lane == 0) { red_c[warp] = c; red_o[warp] = order; }
      __syncthreads();
      if (tid == 0) {
        for (int w = 1; w < 8; ++w)
          if (red_c[w] > c || (red_c[w] == c && red_o[w] < order)) { c = red_c[w]; order = red_o[w]; }
        kstar = order == 0 ? 0 : ((order & 1) ? (order + 1) / 2 : -(order / 2));
      }
      __syncthreads();
    }
    if (tid == 0) {
      hdr->cls_k[cl] = kstar;
      hdr->cls_pot[cl] = P.cls[cl].scope == 0 ? layer_pot_scale(wmax, P.cls[cl].tmax) : 0.0f;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Phase-1 evaluators.  Element layout inside a thread: index idx = 2 * i + p holds, as a float2,
// element i of quads 2p (x) and 2p + 1 (y): the two lanes of a packed f32x2 operation are two
// independent sequential chains, which is exactly the quad-tree summation order.
// ---------------------------------------------------------------------------------------------
struct BlockRegs {
  float2 w[8], c[8], u[8];
  unsigned off[16]; // byte offset of the element's cell row: row * (n_tables * 128) + (lane & 15) * 8; table t adds t * 128
};

__device__ __forceinline__ float fold(const float2 a, const float2 b) {
  return __fadd_rn(__fadd_rn(a.x, a.y), __fadd_rn(b.x, b.y));
}

struct Metric { float nq, dot, sse; };

// One cell entry is {threshold, hi bf16 : lo bf16}: the reconstruction value is hi when u lies
// strictly above the threshold, else lo.  A negated candidate runs the base table on -u (mirrored
// row) and flips the sign of the dot product and of the scale in the error term.
template <bool NEG>
__device__ __forceinline__ Metric eval_lut_cells(const unsigned char* __restrict__ tp, unsigned moff, const BlockRegs& B, float s_hat) {
  float2 nq[2], dot[2], sse[2];
  nq[0] = nq[1] = dot[0] = dot[1] = sse[0] = sse[1] = make_float2(0.0f, 0.0f);
  const float sg = NEG ? s_hat : -s_hat;
  const float2 ns = make_float2(sg, sg);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      const int idx = 2 * i + p;
      const uint2 ea = *reinterpret_cast<const uint2*>(tp + (NEG ? moff - B.off[2 * idx] : B.off[2 * idx]));
      const uint2 eb = *reinterpret_cast<const uint2*>(tp + (NEG ? moff - B.off[2 * idx + 1] : B.off[2 * idx + 1]));
      const bool pa = NEG ? (-B.u[idx].x > __uint_as_float(ea.x)) : (B.u[idx].x > __uint_as_float(ea.x));
      const bool pb = NEG ? (-B.u[idx].y > __uint_as_float(eb.x)) : (B.u[idx].y > __uint_as_float(eb.x));
      float2 q;
      q.x = __uint_as_float(__byte_perm(ea.y, 0u, pa ? 0x3244u : 0x1044u));
      q.y = __uint_as_float(__byte_perm(eb.y, 0u, pb ? 0x3244u : 0x1044u));
      const float2 cq = __fmul2_rn(B.c[idx], q);
      nq[p] = __ffma2_rn(cq, q, nq[p]);
      dot[p] = __ffma2_rn(cq, B.w[idx], dot[p]);
      const float2 e = __ffma2_rn(ns, q, B.w[idx]);
      sse[p] = __ffma2_rn(e, e, sse[p]);
    }
  }
  Metric m;
  m.nq = fold(nq[0], nq[1]);
  const float d = fold(dot[0], dot[1]);
  m.dot = NEG ? -d : d;
  m.sse = fold(sse[0], sse[1]);
  return m;
}

// mode 0: table through binary search over the thresholds (any table); mode 1 / 2: E2M3 / E4M3 grid;
// mode 3: grid given by parameters
template <int MODE, bool NEG>
__device__ __forceinline__ Metric eval_generic(const float* __restrict__ tau, const float* __restrict__ lutv, const BlockRegs& B, float s_hat,
                                               const GridDev grid = GridDev()) {
  float2 nq[2], dot[2], sse[2];
  nq[0] = nq[1] = dot[0] = dot[1] = sse[0] = sse[1] = make_float2(0.0f, 0.0f);
  const float sg = NEG ? s_hat : -s_hat;
  const float2 ns = make_float2(sg, sg);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      const int idx = 2 * i + p;
      const float ux = B.u[idx].x, uy = B.u[idx].y;
      float2 q;
      if constexpr (MODE == 0) {
        q.x = lutv[count_below(tau, NEG ? -ux : ux)];
        q.y = lutv[count_below(tau, NEG ? -uy : uy)];
      } else if constexpr (MODE == SOP_KIND_FP_GRID) {
        q.x = grid_quantize(ux, grid);
        q.y = grid_quantize(uy, grid);
      } else {
        q.x = fp_quantize<MODE>(ux);
        q.y = fp_quantize<MODE>(uy);
      }
      const float2 cq = __fmul2_rn(B.c[idx], q);
      nq[p] = __ffma2_rn(cq, q, nq[p]);
      dot[p] = __ffma2_rn(cq, B.w[idx], dot[p]);
      const float2 e = __ffma2_rn(ns, q, B.w[idx]);
      sse[p] = __ffma2_rn(e, e, sse[p]);
    }
  }
  Metric m;
  m.nq = fold(nq[0], nq[1]);
  const float d = fold(dot[0], dot[1]);
  m.dot = NEG ? -d : d;
  m.sse = fold(sse[0], sse[1]);
  return m;
}

// Build the shared-memory tables of one CTA: table values and thresholds, then the cell tables.
// A cell row r (k = r - c_half) covers the u values that round to k: u * invh in [k - 1/2, k + 1/2];
// row 0 and the last row extend to -inf / +inf.  A row is usable when at most one distinct threshold
// falls inside its closed interval and both neighbouring table values are bf16 numbers (they are
// stored as one 32-bit pair); otherwise the whole table is marked slow and its candidates take the
// binary-search path.  Every row is stored 16 times (128 bytes): lanes l and l + 16 read copy l & 15,
// so a 64-bit load of any 32 rows by a warp is free of bank conflicts.  The tables are interleaved
// row by row ([row][table][copy]): a thread keeps one offset per element and the table is an
// immediate displacement of the load.
__device__ void build_tables(const Plan& P, const AtomsDev& A, uint2* cell, float* tau, float* lutv, int* fast) {
  const int tid = threadIdx.x;
  for (int i = tid; i < P.n_tables * 32; i += blockDim.x) {
    const int t = i >> 5, j = i & 31;
    const int a = P.table_atom[t];
    const int ne = A.atoms[a].n_entries;
    const int jj = min(j, ne - 1);
    lutv[i] = ((A.dd_mask >> a) & 1u) ? A.dd_lut[jj] : A.atoms[a].lut[jj];
  }
  if (tid < SOP_MAX_TABLES) fast[tid] = 1;
  __syncthreads();
  // decision thresholds, one thread per entry (the rule of build_thresholds: the largest fp32 <= the midpoint,
  // a repeated entry takes the threshold above it, +inf from the last entry on)
  for (int i = tid; i < P.n_tables * 32; i += blockDim.x) {
    const int t = i >> 5, j = i & 31;
    const int ne = A.atoms[P.table_atom[t]].n_entries;
    const float* lv = lutv + t * 32;
    int jj = j;
    while (jj < ne - 1 && lv[jj] == lv[jj + 1]) ++jj;
    tau[i] = jj < ne - 1 ? __double2float_rd(0.5 * ((double)lv[jj] + (double)lv[jj + 1])) : __int_as_float(0x7F800000);
  }
  __syncthreads();
  const int rows = P.rows;
  for (int i = tid; i < P.n_tables * rows; i += blockDim.x) {
    const int t = i / rows, r = i - t * rows;
    const ClassDev& C = P.cls[P.table_cls[t]];
    const int ne = A.atoms[P.table_atom[t]].n_entries;
    const int nrow = 2 * C.c_half + 1;
    uint2 entry = make_uint2(0x7F800000u, 0u);
    if (r < nrow) {
      const float hh = __fdiv_rn(1.0f, C.invh);                     // cell width in u (a power of two)
      const float kf = (float)(r - C.c_half);
      const float lo_edge = r == 0 ? -INFINITY : __fmul_rn(kf - 0.5f, hh);
      const float hi_edge = r == nrow - 1 ? INFINITY : __fmul_rn(kf + 0.5f, hh);
      const float* tt = tau + t * 32;
      const float* lv = lutv + t * 32;
      int nbelow = 0, ninside = 0, ndistinct = 0;
      float prev = 0.0f;
      for (int j = 0; j < ne - 1; ++j) {
        const float x = tt[j];
        if (x < lo_edge) ++nbelow;
        else if (x <= hi_edge) {
          if (ninside == 0 || x != prev) ++ndistinct;
          prev = x;
          ++ninside;
        }
      }
      const float lo = lv[nbelow], hi = lv[min(nbelow + ninside, ne - 1)];
      const uint32_t lb = __float_as_uint(lo), hb = __float_as_uint(hi);
      const bool ok = ndistinct <= 1 && (lb & 0xFFFFu) == 0 && (hb & 0xFFFFu) == 0;
      if (!ok) atomicAnd(&fast[t], 0);
      entry.x = ninside ? __float_as_uint(prev) : 0x7F800000u;
      entry.y = (hb & 0xFFFF0000u) | (lb >> 16);
    }
    uint2* dst = cell + ((size_t)r * P.n_tables + t) * 16;
    for (int l = 0; l < 16; ++l) dst[l] = entry;
  }
  __syncthreads();
}

// One evaluated candidate of one block: the cosine, then both per-block values into their columns.
__device__ __forceinline__ void emit(float* __restrict__ block_cos, float* __restrict__ block_sse, size_t col_off, bool on, float nw,
                                     const Metric& mt) {
  const float cosv = block_cosine(nw, mt.nq, mt.dot);
  if (on) {
    block_cos[col_off] = cosv;
    block_sse[col_off] = mt.sse;
  }
}

// Evaluates the candidates of eval_mask on every block and writes their columns of block_cos / block_sse.
__global__ void __launch_bounds__(TB, 1) sweep_kernel(LayerArgs L, Plan P, AtomsDev A, FmtDev F, const WsHeader* __restrict__ hdr,
                                                      float* __restrict__ block_cos, float* __restrict__ block_sse,
                                                      const sop_search_result* __restrict__ prev) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint2* cell = reinterpret_cast<uint2*>(smem);
  float* tau = reinterpret_cast<float*>(cell + (size_t)P.n_tables * P.rows * 16);
  float* lutv = tau + SOP_MAX_TABLES * 32;
  int* fast = reinterpret_cast<int*>(lutv + SOP_MAX_TABLES * 32);
  int* cls_k = fast + SOP_MAX_TABLES;
  float* cls_pot = reinterpret_cast<float*>(cls_k + SOP_MAX_CLASSES);

  const int tid = threadIdx.x, lane = tid & 31;
  build_tables(P, A, cell, tau, lutv, fast);
  if (tid < SOP_MAX_CLASSES) {
    if (P.k_from_result) {
      const bool live = tid < P.n_classes;
      cls_k[tid] = live && P.cls[tid].k_src >= 0 ? prev->k[P.cls[tid].k_src] : 0;
      cls_pot[tid] = live && P.cls[tid].scope == 0 ? layer_pot_scale(prev->layer_absmax, P.cls[tid].tmax) : 0.0f;
    } else {
      cls_k[tid] = hdr->cls_k[tid];
      cls_pot[tid] = hdr->cls_pot[tid];
    }
  }
  __syncthreads();

  // thread -> fixed column block j, rows m = r0, r0 + R, ...
  const long long GT = (long long)gridDim.x * TB;
  const long long R = GT / L.nbk;                 // rows in flight (host guarantees R >= 1)
  const long long gt = (long long)blockIdx.x * TB + tid;
  const bool lane_on = gt < R * L.nbk;
  const long long j = lane_on ? gt % L.nbk : 0;
  const long long r0 = gt / L.nbk;
  const long long n_iter = (L.M + R - 1) / R;

  BlockRegs B;
  {
    const float4* cp = reinterpret_cast<const float4*>(L.c + j * SOP_G);
    float cc[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = __ldg(cp + q);
      cc[4 * q] = v.x; cc[4 * q + 1] = v.y; cc[4 * q + 2] = v.z; cc[4 * q + 3] = v.w;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int p = 0; p < 2; ++p) B.c[2 * i + p] = make_float2(cc[8 * p + i], cc[8 * p + 4 + i]);
  }
  const int copy_off = (lane & 15) * 8;
  const unsigned char* cell_bytes = reinterpret_cast<const unsigned char*>(cell);

  // Warp-uniform control flow: every thread evaluates a block in every iteration (a thread without
  // work re-evaluates a valid block and stores nothing), so the class / candidate loops below are
  // uniform branches.
  const unsigned fast_mask = __ballot_sync(0xFFFFFFFFu, fast[lane & (SOP_MAX_TABLES - 1)] != 0);
  const uint16_t* wcol = L.W + j * SOP_G;
  uint32_t wb[8];
  load_block_bits(wcol + min(r0, L.M - 1) * L.ldw, wb);
  const size_t NBs = (size_t)L.NB;

  for (long long it = 0; it < n_iter; ++it) {
    const long long m = r0 + it * R;
    const bool on = lane_on && m < L.M;
    // ---- unpack, block statistics ----
    float wf[16];
#pragma unroll
    for (int q = 0; q < 8; ++q) { wf[2 * q] = bf16lo(wb[q]); wf[2 * q + 1] = bf16hi(wb[q]); }
    const float amax = absmax_bits(wb);
    load_block_bits(wcol + min(m + R, L.M - 1) * L.ldw, wb);   // prefetch the next row's block
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int p = 0; p < 2; ++p) B.w[2 * i + p] = make_float2(wf[8 * p + i], wf[8 * p + 4 + i]);
    float2 nw2[2];
    nw2[0] = nw2[1] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int p = 0; p < 2; ++p) {
        const float2 cw = __fmul2_rn(B.c[2 * i + p], B.w[2 * i + p]);
        nw2[p] = __ffma2_rn(cw, B.w[2 * i + p], nw2[p]);
      }
    const float nw = fold(nw2[0], nw2[1]);
    const size_t blk = (size_t)(m * L.nbk + j);

    for (int cl = 0; cl < P.n_classes; ++cl) {
      const ClassDev& C = P.cls[cl];
      if (C.n_cand == 0) continue;
      float s_hat;
      if (C.scope == 0) {
        s_hat = amax > 0.0f ? cls_pot[cl] : 0.0f;
      } else {
        const float sigma = C.tmax == 1.0f ? amax : __fdiv_rn(amax, C.tmax);
        s_hat = scale_quantize(sigma, cls_k[cl], F).s_hat;
      }
      const float rcp = s_hat > 0.0f ? __frcp_rn(s_hat) : 0.0f;
      const float2 r2 = make_float2(rcp, rcp);
#pragma unroll
      for (int idx = 0; idx < 8; ++idx) B.u[idx] = __fmul2_rn(B.w[idx], r2);
      if (C.kind == SOP_KIND_LUT) {
        const float tlo = MAGIC, thi = MAGIC + (float)(2 * C.c_half), toff = MAGIC + (float)C.c_half;
        const float invh = C.invh;
        const unsigned pitch = (unsigned)P.n_tables * 128u;
        const unsigned cbias = (unsigned)copy_off - __float_as_uint(MAGIC) * pitch;   // modulo 2^32
#pragma unroll
        for (int idx = 0; idx < 8; ++idx) {
          const float tx = fminf(fmaxf(__fmaf_rn(B.u[idx].x, invh, toff), tlo), thi);
          const float ty = fminf(fmaxf(__fmaf_rn(B.u[idx].y, invh, toff), tlo), thi);
          B.off[2 * idx] = __float_as_uint(tx) * pitch + cbias;
          B.off[2 * idx + 1] = __float_as_uint(ty) * pitch + cbias;
        }
        const unsigned moff = 2u * (unsigned)C.c_half * pitch + 2u * (unsigned)copy_off;
        // tables of this class with a usable cell grid: the table slot is a compile-time displacement
        const unsigned cls_fast = P.cls_tables[cl] & fast_mask;
#pragma unroll
        for (int T = 0; T < SOP_MAX_TABLES; ++T) {
          if ((cls_fast >> T) & 1u) {
            const unsigned char* tp = cell_bytes + T * 128;
            const int ap = P.table_pos[T], an = P.table_neg[T];
            if (ap != 255) emit(block_cos, block_sse, (size_t)ap * NBs + blk, on, nw, eval_lut_cells<false>(tp, moff, B, s_hat));
            if (an != 255) emit(block_cos, block_sse, (size_t)an * NBs + blk, on, nw, eval_lut_cells<true>(tp, moff, B, s_hat));
          }
        }
        // tables without a usable cell grid: binary search over the thresholds
        if (P.cls_tables[cl] & ~fast_mask) {
          for (int ci = 0; ci < C.n_cand; ++ci) {
            const int a = C.cand[ci];
            const int t = P.cand[a].table;
            if ((fast_mask >> t) & 1u) continue;
            const Metric mt = P.cand[a].neg ? eval_generic<0, true>(tau + t * 32, lutv + t * 32, B, s_hat)
                                            : eval_generic<0, false>(tau + t * 32, lutv + t * 32, B, s_hat);
            emit(block_cos, block_sse, (size_t)a * NBs + blk, on, nw, mt);
          }
        }
      } else if (C.kind == SOP_KIND_FP_E2M3) {
        for (int ci = 0; ci < C.n_cand; ++ci)
          emit(block_cos, block_sse, (size_t)C.cand[ci] * NBs + blk, on, nw, eval_generic<SOP_KIND_FP_E2M3, false>(nullptr, nullptr, B, s_hat));
      } else if (C.kind == SOP_KIND_FP_GRID) {
        for (int ci = 0; ci < C.n_cand; ++ci)
          emit(block_cos, block_sse, (size_t)C.cand[ci] * NBs + blk, on, nw,
               eval_generic<SOP_KIND_FP_GRID, false>(nullptr, nullptr, B, s_hat, C.grid));
      } else {
        for (int ci = 0; ci < C.n_cand; ++ci)
          emit(block_cos, block_sse, (size_t)C.cand[ci] * NBs + blk, on, nw, eval_generic<SOP_KIND_FP_E4M3, false>(nullptr, nullptr, B, s_hat));
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The reduction of the per-block columns into table entries.
//   A CTA takes tiles of RTILE blocks.  The columns (cosines and errors of every candidate that a task of the
//   launch touches) of a tile are brought into a ring of shared-memory buffers by 16-byte asynchronous copies
//   (cp.async, every thread a few), up to three tiles ahead of the arithmetic; a thread waits for its own copy
//   groups and the one barrier per tile makes everybody's visible.  (One-dimensional bulk copies with an
//   mbarrier, one kilobyte per column, were measured first: the per-request cost of twenty small requests per
//   tile bound the kernel.)  16-byte copies need aligned addresses, which holds when the number of blocks is a
//   multiple of four and the arrays are 16-byte aligned; otherwise (odd small layers) the tile is fetched with
//   plain loads.  Nothing in this kernel spins on a flag.
//   A warp owns up to three tasks.  A lane owns eight blocks of the tile (two runs of four): per
//   entry it sums eight gaps 1 - cos (exact in fp32 for cos in [0.5, 1]) and eight errors in fp32, then adds
//   both to the lane's FP64 accumulators of that entry, which live in shared memory.  At the end the 32 lanes'
//   accumulators of an entry are added in lane order: the result depends on the grid size only.
//   A signed four-way entry {i, -i, j, -j} is the two-way entry of "the better of i and -i" and "the better of
//   j and -j" (ties to the atom; the sign of the error marks a negated winner), formed on the fly from the two
//   columns of each base atom.  A block beyond the end of the layer reads as (cos 1, error 0): it adds nothing.
// ---------------------------------------------------------------------------------------------
constexpr int RTB = 256;              // threads per CTA of the reduction: eight warps
constexpr int RTILE = 256;            // blocks per tile: eight per lane
constexpr int ENT = TASK_PART + 1;    // entries of a task: the anchor alone, then its partners
constexpr int MAX_STAGE = 4;           // tile buffers of the ring

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ void finalize_body(const LayerArgs& L, const Plan& P, int grid, const Partial* partials, sop_pair_stat* s_pair, sop_pair_stat* s_sig,
                              Partial* s_red, sop_pair_stat* pair_table, sop_pair_stat* signed_table, sop_search_result* res,
                              const int* cls_k, float wmax);

constexpr int ACC_BYTES = 32 * 20;     // accumulators of one entry: 32 lanes x (two FP64 sums, two 16-bit counts)

__device__ __forceinline__ void lds128(unsigned addr, float (&v)[4]) {
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "r"(addr));
}

// The accumulators of one entry and lane, in shared memory: FP64 sums (gap, error) at sums + seat * 512 + lane * 16 and
// counts (second candidate chosen, negated winner; 16 bits each: a lane sees at most 8 blocks per tile and a CTA a few
// thousand tiles) at counts + seat * 128 + lane * 4.
// NT = 1: the sums of one tile; NT = 2: of two tiles, added one after the other (the same additions in the same order
// as two calls, with one load and one store of the accumulators).
template <int NT>
__device__ __forceinline__ void acc_add(unsigned sums, unsigned counts, const float (&cg)[NT], const float (&ce)[NT], const int (&n1)[NT],
                                        const int (&nn)[NT]) {
  double g, e;
  asm volatile("ld.shared.v2.f64 {%0, %1}, [%2];" : "=d"(g), "=d"(e) : "r"(sums));
#pragma unroll
  for (int t = 0; t < NT; ++t) { g += (double)cg[t]; e += (double)ce[t]; }
  asm volatile("st.shared.v2.f64 [%0], {%1, %2};" ::"r"(sums), "d"(g), "d"(e) : "memory");
  unsigned c;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(c) : "r"(counts));
#pragma unroll
  for (int t = 0; t < NT; ++t) c += (unsigned)n1[t] + ((unsigned)nn[t] << 16);       // neither half can carry: both stay below 2^16
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(counts), "r"(c) : "memory");
}

// One task on the lane's eight blocks of one tile (blocks 4 lane .. 4 lane + 3 and the same 128 further on: two 128-bit
// loads per column and array).  The code is the same for every warp and task -- tasks differ in data only -- and small:
// a loop over the task's partners whose body handles the eight blocks.  Per entry the eight gaps and errors are summed
// in fp32 and added to the lane's FP64 accumulators.
//   cos_base / sse_base: shared-memory addresses of the tile's columns (for a signed task the signed-best columns);
//   tk: the task (in shared memory); sums / counts: shared-memory addresses of this lane's accumulators of the task's
//   first seat: the anchor alone if the task has that entry, then the partners.
//   NT = 2: the same task on two tiles at once -- the tile in work and the one `pair_off` bytes further on in shared
//   memory -- so that the accumulators are loaded and stored once for both.
template <bool SEL_ERR, bool SGN, bool REV, int NT>
__device__ __forceinline__ void run_task(const TaskDev* __restrict__ tk, unsigned cos_base, unsigned sse_base, unsigned pair_off, int lane,
                                         unsigned sums, unsigned counts) {
  constexpr unsigned COL = RTILE * 4u;          // bytes of one column
  const unsigned lane_off = (unsigned)lane * 16u;
  float ac0[NT][4], ac1[NT][4], ae0[NT][4], ae1[NT][4], ga0[NT][4], ga1[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    const unsigned a = (unsigned)tk->anchor * COL + lane_off + (unsigned)t * pair_off;
    lds128(cos_base + a, ac0[t]); lds128(cos_base + a + 512u, ac1[t]);
    lds128(sse_base + a, ae0[t]); lds128(sse_base + a + 512u, ae1[t]);
#pragma unroll
    for (int r = 0; r < 4; ++r) { ga0[t][r] = __fsub_rn(1.0f, ac0[t][r]); ga1[t][r] = __fsub_rn(1.0f, ac1[t][r]); }
  }
  if (tk->self_slot != 255) {
    float cg[NT], ce[NT];
    int n1[NT], nn[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      cg[t] = 0.0f; ce[t] = 0.0f; n1[t] = 0; nn[t] = 0;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        cg[t] = __fadd_rn(cg[t], ga0[t][r]); ce[t] = __fadd_rn(ce[t], fabsf(ae0[t][r]));
        cg[t] = __fadd_rn(cg[t], ga1[t][r]); ce[t] = __fadd_rn(ce[t], fabsf(ae1[t][r]));
        if (SGN) nn[t] += (int)(__float_as_uint(ae0[t][r]) >> 31) + (int)(__float_as_uint(ae1[t][r]) >> 31);
      }
    }
    acc_add<NT>(sums, counts, cg, ce, n1, nn);
    sums += 512u; counts += 128u;            // the partners' seats follow
  }
  const int np = tk->n_part;
#pragma unroll 1
  for (int q = 0; q < np; ++q) {
    float cg[NT], ce[NT];
    int n1[NT], nn[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      const unsigned b = (unsigned)tk->part[q] * COL + lane_off + (unsigned)t * pair_off;
      float bc0[4], bc1[4], be0[4], be1[4];
      lds128(cos_base + b, bc0); lds128(cos_base + b + 512u, bc1);
      lds128(sse_base + b, be0); lds128(sse_base + b + 512u, be1);
      cg[t] = 0.0f; ce[t] = 0.0f; n1[t] = 0; nn[t] = 0;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        // mu: the entry's second candidate is strictly better and takes the block.  REV = false: the anchor is the
        // first candidate and the partner the second; REV = true: the other way round.
        bool mu0, mu1;
        float g0, g1, e0, e1;
        if (!REV) {
          mu0 = SEL_ERR ? fabsf(be0[r]) < fabsf(ae0[t][r]) : bc0[r] > ac0[t][r];
          mu1 = SEL_ERR ? fabsf(be1[r]) < fabsf(ae1[t][r]) : bc1[r] > ac1[t][r];
          g0 = mu0 ? __fsub_rn(1.0f, bc0[r]) : ga0[t][r]; e0 = mu0 ? be0[r] : ae0[t][r];
          g1 = mu1 ? __fsub_rn(1.0f, bc1[r]) : ga1[t][r]; e1 = mu1 ? be1[r] : ae1[t][r];
        } else {
          mu0 = SEL_ERR ? fabsf(ae0[t][r]) < fabsf(be0[r]) : ac0[t][r] > bc0[r];
          mu1 = SEL_ERR ? fabsf(ae1[t][r]) < fabsf(be1[r]) : ac1[t][r] > bc1[r];
          g0 = mu0 ? ga0[t][r] : __fsub_rn(1.0f, bc0[r]); e0 = mu0 ? ae0[t][r] : be0[r];
          g1 = mu1 ? ga1[t][r] : __fsub_rn(1.0f, bc1[r]); e1 = mu1 ? ae1[t][r] : be1[r];
        }
        cg[t] = __fadd_rn(cg[t], g0); ce[t] = __fadd_rn(ce[t], fabsf(e0));
        cg[t] = __fadd_rn(cg[t], g1); ce[t] = __fadd_rn(ce[t], fabsf(e1));
        n1[t] += (mu0 ? 1 : 0) + (mu1 ? 1 : 0);
        if (SGN) nn[t] += (int)(__float_as_uint(e0) >> 31) + (int)(__float_as_uint(e1) >> 31);
      }
    }
    acc_add<NT>(sums + (unsigned)q * 512u, counts + (unsigned)q * 128u, cg, ce, n1, nn);
  }
}

// PAIR (with VEC and a ring of four buffers): the CTA works on two tiles at a time -- buffers (0, 1), then (2, 3) while
// (0, 1) are refilled -- so that a lane owns sixteen blocks per step and touches its accumulators half as often.  The
// additions and their order are those of the one-tile path: the results are the same bit for bit.
template <bool SEL_ERR, int TPW, bool VEC, bool PAIR>
__global__ void __launch_bounds__(RTB, 2) reduce_kernel(LayerArgs L, Plan P, SeatsDev seats, int n_stage, int do_final, WsHeader* __restrict__ hdr,
                                                     Partial* __restrict__ partials, const float* __restrict__ block_cos,
                                                     const float* __restrict__ block_sse, sop_pair_stat* pair_table,
                                                     sop_pair_stat* signed_table, sop_search_result* __restrict__ res,
                                                     const sop_search_result* __restrict__ prev) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int A = seats.n_cols;                                            // columns of a tile buffer
  const int NBUF = VEC ? n_stage : 1;                                    // tile buffers: a ring, filled n_stage - 1 tiles ahead
  float* cos0 = reinterpret_cast<float*>(smem);                          // [NBUF][A][RTILE]
  float* sse0 = cos0 + (size_t)NBUF * A * RTILE;                         // [NBUF][A][RTILE]
  // signed-best columns of the tile in work
  constexpr int NSB = PAIR ? 2 : 1;                                      // tiles in work at a time
  float* scos = sse0 + (size_t)NBUF * A * RTILE;                         // [NSB][n_bases][RTILE]
  float* ssse = scos + (size_t)NSB * seats.n_bases * RTILE;              // [NSB][n_bases][RTILE]
  double2* acc_sums = reinterpret_cast<double2*>(ssse + (size_t)NSB * seats.n_bases * RTILE);   // [n_seats][32]: seat-major, then lane
  unsigned* acc_counts = reinterpret_cast<unsigned*>(acc_sums + (size_t)seats.n_seats * 32);   // [n_seats][32]: two 16-bit counts
  __shared__ unsigned long long s_coloff[SOP_MAX_ATOMS];   // first element of every fetched column in the arrays
  __shared__ TaskDev s_task[RTB / 32][TPW];        // anchors and partners translated to columns of the buffers
  __shared__ int s_acc0[RTB / 32][TPW];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (lane < TPW) {
    const int ti = seats.task[warp][lane];
    TaskDev t;
    if (ti != 255) {
      t = P.tasks[ti];
      const unsigned char* map = t.sgn ? seats.sb_slot : seats.col_slot;
      t.anchor = map[t.anchor];
      for (int q = 0; q < t.n_part; ++q) t.part[q] = map[t.part[q]];
    } else { t.anchor = 0; t.n_part = 0; t.self_slot = 255; t.sgn = 2; }   // sgn 2: an empty seat
    s_task[warp][lane] = t;
    s_acc0[warp][lane] = seats.acc0[warp][lane];
  }
  for (int i = tid; i < seats.n_seats * 32; i += RTB) { acc_sums[i] = make_double2(0.0, 0.0); acc_counts[i] = 0u; }
  if (tid < seats.n_cols) s_coloff[tid] = (unsigned long long)seats.cols[tid] * (unsigned long long)L.NB;
  __syncthreads();
  const int ncols = seats.n_cols, nbases = seats.n_bases;
  const long long n_tiles = (L.NB + RTILE - 1) / RTILE;

  // Every thread's share of the 16-byte copies of one tile into buffer b.  Chunk c = (column, array, run of four blocks);
  // thread t takes the chunks t, t + 256, ...: always the same array and run, every second column.  Runs beyond the
  // end of the layer are filled with (cos 1, error 0) instead.  One commit group per tile.
  const int f_arr = (tid >> 6) & 1, f_ch = tid & 63;
  const float* f_src = (f_arr ? block_sse : block_cos) + 4 * f_ch;
  const unsigned f_dst = smem_u32(f_arr ? sse0 : cos0) + (unsigned)(((tid >> 7) * RTILE + 4 * f_ch) * 4);
  auto fetch = [&](long long tile, int b) {
    if (tile < n_tiles) {
      const long long blk0 = tile * RTILE;
      const bool live = blk0 + 4 * f_ch < L.NB;
      unsigned dst = f_dst + (unsigned)(b * A * RTILE * 4);
      for (int i = tid >> 7; i < ncols; i += 2, dst += 2u * RTILE * 4u) {
        if (live) {
          const float* src = f_src + s_coloff[i] + blk0;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
        } else {
          const float v = f_arr ? 0.0f : 1.0f;
          asm volatile("st.shared.v4.f32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "f"(v) : "memory");
        }
      }
    } else if (PAIR) {
      // the second tile of the last pair does not exist: it reads as (cos 1, error 0) and adds nothing
      unsigned dst = f_dst + (unsigned)(b * A * RTILE * 4);
      const float v = f_arr ? 0.0f : 1.0f;
      for (int i = tid >> 7; i < ncols; i += 2, dst += 2u * RTILE * 4u)
        asm volatile("st.shared.v4.f32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "f"(v) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  if constexpr (PAIR) {
    const long long step = gridDim.x;
    long long tile = blockIdx.x;
    fetch(tile, 0);
    fetch(tile + step, 1);
    int ps = 0;                  // the pair of buffers in work: (0, 1) or (2, 3)
    for (; tile < n_tiles; tile += 2 * step) {
      float* cosb = cos0 + (size_t)(2 * ps) * A * RTILE;
      float* sseb = sse0 + (size_t)(2 * ps) * A * RTILE;
      asm volatile("cp.async.wait_group 0;" ::: "memory");       // this thread's copies of both tiles have landed
      if (nbases) {
        __syncthreads();                                          // ... and everybody's; the previous pair's readers are done
        for (int t = 0; t < 2; ++t)
          for (int i = 0; i < nbases; ++i) {
            const int a = seats.bases[i], cp = seats.col_slot[a], cn = seats.col_slot[a + 1];
            const float* cb = cosb + (size_t)t * A * RTILE;
            const float* sb = sseb + (size_t)t * A * RTILE;
            const float pc = cb[cp * RTILE + tid], pe = sb[cp * RTILE + tid];
            const float nc = cb[cn * RTILE + tid], ne = sb[cn * RTILE + tid];
            const bool neg = SEL_ERR ? ne < pe : nc > pc;
            scos[((size_t)t * nbases + i) * RTILE + tid] = neg ? nc : pc;
            ssse[((size_t)t * nbases + i) * RTILE + tid] = neg ? -ne : pe;
          }
      }
      __syncthreads();
      // the other pair of buffers is free (everybody has passed the barrier, so nobody reads the previous pair any more)
      fetch(tile + 2 * step, 2 * (ps ^ 1));
      fetch(tile + 3 * step, 2 * (ps ^ 1) + 1);
#pragma unroll 1
      for (int k = 0; k < TPW; ++k) {
        const TaskDev* tk = &s_task[warp][k];
        const unsigned sums = smem_u32(acc_sums) + (unsigned)(s_acc0[warp][k] * 32 + lane) * 16u;
        const unsigned counts = smem_u32(acc_counts) + (unsigned)(s_acc0[warp][k] * 32 + lane) * 4u;
        const int sgn = tk->sgn;
        const int rev = tk->rev;
        const unsigned poff = (unsigned)(A * RTILE * 4), soff = (unsigned)(nbases * RTILE * 4);
        if (sgn == 0) {
          if (rev) run_task<SEL_ERR, false, true, 2>(tk, smem_u32(cosb), smem_u32(sseb), poff, lane, sums, counts);
          else run_task<SEL_ERR, false, false, 2>(tk, smem_u32(cosb), smem_u32(sseb), poff, lane, sums, counts);
        } else if (sgn == 1) {
          if (rev) run_task<SEL_ERR, true, true, 2>(tk, smem_u32(scos), smem_u32(ssse), soff, lane, sums, counts);
          else run_task<SEL_ERR, true, false, 2>(tk, smem_u32(scos), smem_u32(ssse), soff, lane, sums, counts);
        }
      }
      ps ^= 1;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");         // nothing of this CTA's is in flight when it leaves
  } else {
    long long tile = blockIdx.x;
    if (VEC)
      for (int b = 0; b < n_stage - 1; ++b) fetch(tile + (long long)b * gridDim.x, b);
    int cur = 0;                 // buffer of the tile in work
    for (; tile < n_tiles; tile += gridDim.x) {
      float* cosb = cos0 + (size_t)cur * A * RTILE;
      float* sseb = sse0 + (size_t)cur * A * RTILE;
      if (VEC) {
        // this thread's copies of the tile in work are complete when at most n_stage - 2 newer groups are still pending
        if (n_stage == 4) asm volatile("cp.async.wait_group 2;" ::: "memory");
        else if (n_stage == 3) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
      } else {
        const long long blk0 = tile * RTILE;
        const int nv = (int)min((long long)RTILE, L.NB - blk0);
        __syncthreads();                                      // everybody has finished the previous tile
        for (int i = 0; i < ncols; ++i) {
          const size_t a = seats.cols[i];
          cosb[i * RTILE + tid] = tid < nv ? __ldg(block_cos + a * L.NB + blk0 + tid) : 1.0f;
          sseb[i * RTILE + tid] = tid < nv ? __ldg(block_sse + a * L.NB + blk0 + tid) : 0.0f;
        }
      }
      if (nbases) {
        // Signed-best columns: this thread's block.  The values come from other threads' copies, and the previous tile's
        // readers of these columns must be done first: hence the barrier.
        __syncthreads();
        for (int i = 0; i < nbases; ++i) {
          const int a = seats.bases[i], cp = seats.col_slot[a], cn = seats.col_slot[a + 1];     // the atom and its negation
          const float pc = cosb[cp * RTILE + tid], pe = sseb[cp * RTILE + tid];
          const float nc = cosb[cn * RTILE + tid], ne = sseb[cn * RTILE + tid];
          const bool neg = SEL_ERR ? ne < pe : nc > pc;           // ties to the atom; a negative error marks a negated winner
          scos[i * RTILE + tid] = neg ? nc : pc;
          ssse[i * RTILE + tid] = neg ? -ne : pe;
        }
      }
      // One barrier per tile: the tile is complete for everybody, and everybody has finished the previous tile, whose
      // buffer (the one before this in the ring) the next copies refill.
      __syncthreads();
      if (VEC) fetch(tile + (long long)(n_stage - 1) * gridDim.x, cur == 0 ? n_stage - 1 : cur - 1);
  #pragma unroll 1
      for (int k = 0; k < TPW; ++k) {
        const TaskDev* tk = &s_task[warp][k];
        const unsigned sums = smem_u32(acc_sums) + (unsigned)(s_acc0[warp][k] * 32 + lane) * 16u;
        const unsigned counts = smem_u32(acc_counts) + (unsigned)(s_acc0[warp][k] * 32 + lane) * 4u;
        const int sgn = tk->sgn;
        const int rev = tk->rev;
        if (sgn == 0) {
          if (rev) run_task<SEL_ERR, false, true, 1>(tk, smem_u32(cosb), smem_u32(sseb), 0u, lane, sums, counts);
          else run_task<SEL_ERR, false, false, 1>(tk, smem_u32(cosb), smem_u32(sseb), 0u, lane, sums, counts);
        } else if (sgn == 1) {
          if (rev) run_task<SEL_ERR, true, true, 1>(tk, smem_u32(scos), smem_u32(ssse), 0u, lane, sums, counts);
          else run_task<SEL_ERR, true, false, 1>(tk, smem_u32(scos), smem_u32(ssse), 0u, lane, sums, counts);
        }
      }
      if (VEC && ++cur == n_stage) cur = 0;
    }
  }

  // ---- per-CTA partials: lane (k, q) of a warp adds the 32 lanes' sums of entry q of the warp's task k, in lane order ----
  __syncwarp();
  if (lane < TPW * ENT) {
    const int k = lane / ENT, q = lane - k * ENT;
    const TaskDev t = s_task[warp][k];
    const int slot = t.sgn == 2 ? 255 : (q == 0 ? t.self_slot : (q - 1 < t.n_part ? t.slot[q - 1] : 255));
    if (slot != 255) {
      Partial p; p.gap = 0.0; p.sse = 0.0; p.n1 = 0; p.nneg = 0;
      const int seat = s_acc0[warp][k] + (q == 0 ? 0 : q - 1 + (t.self_slot != 255 ? 1 : 0));
      for (int l = 0; l < 32; ++l) {
        const double2 a = acc_sums[(size_t)seat * 32 + l];
        const unsigned c = acc_counts[(size_t)seat * 32 + l];
        p.gap += a.x; p.sse += a.y; p.n1 += (long long)(c & 0xFFFFu); p.nneg += (long long)(c >> 16);
      }
      partials[(size_t)blockIdx.x * MAX_SLOTS + slot] = p;
    }
  }
  if (!do_final) return;
  // the CTA that arrives last adds everybody's partials and writes the tables; nobody waits for anybody
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&hdr->done_reduce, 1u) == gridDim.x - 1 ? 1 : 0;
  __syncthreads();
  if (s_last) {
    __threadfence();
    __shared__ int cls_k[SOP_MAX_CLASSES];
    if (tid < SOP_MAX_CLASSES) {
      const bool live = tid < P.n_classes;
      cls_k[tid] = P.k_from_result ? (live && P.cls[tid].k_src >= 0 ? prev->k[P.cls[tid].k_src] : 0) : __ldcg(&hdr->cls_k[tid]);
    }
    const float wmax = P.k_from_result ? prev->layer_absmax : __uint_as_float(__ldcg(&hdr->wmax_bits));
    __syncthreads();
    sop_pair_stat* s_pair = reinterpret_cast<sop_pair_stat*>(smem);
    sop_pair_stat* s_sig = s_pair + SOP_MAX_ATOMS * SOP_MAX_ATOMS;
    finalize_body(L, P, (int)gridDim.x, partials, s_pair, s_sig, reinterpret_cast<Partial*>(s_sig + SOP_MAX_ATOMS * SOP_MAX_ATOMS), pair_table,
                  signed_table, res, cls_k, wmax);
  }
}

// One warp.  The defined entry of `tab` ([A x A]) with the largest acos, ties to the smallest index: among the
// entries above the diagonal (diag = 0) or among the diagonal entries of the candidates in lut_mask (diag = 1).  -1: none.
__device__ __noinline__ int warp_best(const sop_pair_stat* tab, int A, int diag, unsigned lut_mask) {
  const int lane = threadIdx.x & 31;
  int best = -1;
  double bv = 0.0;
#pragma unroll 1
  for (int i = lane; i < A * A; i += 32) {
    const int a = i / A, b = i - a * A;
    const bool in = diag ? (b == a && ((lut_mask >> a) & 1u)) : b > a;
    if (in && tab[i].n_sel1 >= 0 && (best < 0 || tab[i].acos > bv)) { best = i; bv = tab[i].acos; }
  }
#pragma unroll 1
  for (int o = 16; o; o >>= 1) {
    const double ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    if (oi >= 0 && (best < 0 || ov > bv || (ov == bv && oi < best))) { bv = ov; best = oi; }
  }
  return best;
}

// Run by one whole CTA of TB threads.  Thread (slot, chunk) adds the partials of CTAs chunk, chunk + C,
// ... in that order (C = min(TB / n_slots, ceil(grid / 4)) chunks, loads coalesced over the slots and issued four at a
// time), the chunks are then added in chunk order: the result depends only on the grid size, not on
// scheduling.  s_pair / s_sig (n_atoms^2 entries each) and s_red (TB entries) are shared-memory staging.
__device__ void finalize_body(const LayerArgs& L, const Plan& P, int grid, const Partial* partials, sop_pair_stat* s_pair, sop_pair_stat* s_sig,
                              Partial* s_red, sop_pair_stat* pair_table, sop_pair_stat* signed_table, sop_search_result* res,
                              const int* cls_k, float wmax) {
  const int A = P.n_atoms, tid = threadIdx.x, n_slots = P.n_slots;
  for (int i = tid; i < A * A; i += blockDim.x) {
    sop_pair_stat u; u.acos = 0.0; u.mse = 0.0; u.n_sel1 = -1; u.n_neg = -1;
    // entries among candidates that an earlier call evaluated stay as that call left them in the tables
    const int a = i / A, b = i - a * A;
    const bool keep = P.keep_loaded && ((P.load_mask >> a) & 1u) && ((P.load_mask >> b) & 1u);
    s_pair[i] = keep ? pair_table[i] : u;
    s_sig[i] = keep && signed_table ? signed_table[i] : u;
  }
  __syncthreads();
  const int n_chunks = max(1, min((int)blockDim.x / max(n_slots, 1), (grid + 3) / 4));   // at best one round of four loads per thread
  const int slot = tid % max(n_slots, 1), chunk = tid / max(n_slots, 1);
  if (chunk < n_chunks && n_slots > 0) {
    Partial t; t.gap = 0.0; t.sse = 0.0; t.n1 = 0; t.nneg = 0;
#pragma unroll 1
    for (int g0 = chunk; g0 < grid; g0 += 4 * n_chunks) {
      double2 a[4];
      longlong2 b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int g = g0 + u * n_chunks;
        a[u] = make_double2(0.0, 0.0);
        b[u] = make_longlong2(0, 0);
        if (g < grid) {
          const double2* q = reinterpret_cast<const double2*>(partials + (size_t)g * MAX_SLOTS + slot);
          a[u] = __ldcg(q);
          b[u] = __ldcg(reinterpret_cast<const longlong2*>(q + 1));
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (g0 + u * n_chunks < grid) { t.gap += a[u].x; t.sse += a[u].y; t.n1 += b[u].x; t.nneg += b[u].y; }
    }
    s_red[tid] = t;
  }
  __syncthreads();
  if (tid < n_slots) {
    Partial t = s_red[tid];
#pragma unroll 1
    for (int c = 1; c < n_chunks; ++c) {
      const Partial q = s_red[c * n_slots + tid];
      t.gap += q.gap; t.sse += q.sse; t.n1 += q.n1; t.nneg += q.nneg;
    }
    sop_pair_stat st;
    st.acos = ((double)L.NB - t.gap) / (double)L.NB;
    st.mse = t.sse / ((double)L.M * (double)L.K);
    st.n_sel1 = t.n1;
    const SlotDev sd = P.slots[tid];
    if (sd.type == 0) { st.n_neg = 0; s_pair[sd.i0 * A + sd.i1] = st; }
    else { st.n_neg = t.nneg; s_sig[sd.i0 * A + sd.i1] = st; }
  }
  __syncthreads();
  for (int i = tid; i < A * A; i += blockDim.x) {
    pair_table[i] = s_pair[i];
    if (signed_table) signed_table[i] = s_sig[i];
  }
  if (tid < SOP_MAX_ATOMS) {
    const bool present = tid < A && (((P.eval_mask | P.load_mask) >> tid) & 1u);
    res->k[tid] = present ? cls_k[P.cand[tid].cls] : 0;
  }
  // best two-codebook pair, best single LUT candidate, best signed pair: largest ACos, ties to the smallest
  // (a, b).  One warp, one small routine called three times: this code runs once per launch, so its size
  // (instruction fetches that miss) costs more than its arithmetic.
  if (tid < 32) {
    unsigned lut_mask = 0;
    for (int a = 0; a < A; ++a) lut_mask |= P.cand[a].kind == SOP_KIND_LUT ? 1u << a : 0u;
    const int ip = warp_best(s_pair, A, 0, lut_mask);
    const int is = warp_best(s_pair, A, 1, lut_mask);
    const int isg = signed_table ? warp_best(s_sig, A, 0, lut_mask) : -1;
    if (tid == 0) {
      res->layer_absmax = wmax;
      res->reserved[0] = res->reserved[1] = 0;
      res->best_a = ip >= 0 ? ip / A : -1; res->best_b = ip >= 0 ? ip % A : -1;
      res->best_single = is >= 0 ? is / A : -1;
      res->best_sa = isg >= 0 ? isg / A : -1; res->best_sb = isg >= 0 ? isg % A : -1;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// host: plan construction
// ---------------------------------------------------------------------------------------------
static bool same_table(const sop_atom& a, const sop_atom& b) {
  return a.n_entries == b.n_entries && memcmp(a.lut, b.lut, sizeof(float) * a.n_entries) == 0;
}

// smallest gap between distinct decision thresholds of a host-known table (in u)
static double min_threshold_gap(const sop_atom& a) {
  double prev = 0, best = 1e30;
  bool have = false;
  for (int j = 0; j + 1 < a.n_entries; ++j) {
    if (a.lut[j] == a.lut[j + 1]) continue;
    const double t = 0.5 * ((double)a.lut[j] + (double)a.lut[j + 1]);
    if (have && t > prev) best = fmin(best, t - prev);
    prev = t;
    have = true;
  }
  return best;
}

int build_plan(const AtomsDev& A, const FmtDev& F, int k_mode, unsigned eval_mask, unsigned load_mask, int singles_only, int keep_loaded, Plan* P) {
  memset(P, 0, sizeof(*P));
  const int n = A.n_atoms;
  P->n_atoms = n;
  P->k_mode = k_mode;
  P->eval_mask = eval_mask;
  P->load_mask = load_mask;
  const unsigned present = eval_mask | load_mask;
  // classes
  for (int i = 0; i < n; ++i) {
    const sop_atom& a = A.atoms[i];
    P->cand[i].kind = (unsigned char)a.kind;
    P->cand[i].neg = (unsigned char)a.negated;
    if (!((present >> i) & 1u)) continue;
    int cl = -1;
    for (int c = 0; c < P->n_classes; ++c)
      if (P->cls[c].scope == a.scope && P->cls[c].tmax == a.tmax && P->cls[c].kind == a.kind &&
          (a.kind != SOP_KIND_FP_GRID || (P->cls[c].grid.min_eb == 128 - a.grid_bias && P->cls[c].grid.sh == 23 - a.grid_man_bits &&
                                          P->cls[c].grid.vneg == a.grid_neg_max))) cl = c;
    if (cl < 0) {
      if (P->n_classes == SOP_MAX_CLASSES) return SOP_ERR_ALPHABET;
      cl = P->n_classes++;
      P->cls[cl].scope = a.scope; P->cls[cl].tmax = a.tmax; P->cls[cl].kind = a.kind;
      P->cls[cl].auto_k = (k_mode == SOP_K_AUTO && a.scope != 0) ? 1 : 0;
      P->cls[cl].invh = 1.0f; P->cls[cl].c_half = 0;
      P->cls[cl].grid.min_eb = 128 - a.grid_bias; P->cls[cl].grid.sh = 23 - a.grid_man_bits;
      P->cls[cl].grid.vpos = a.tmax; P->cls[cl].grid.vneg = a.grid_neg_max;
    }
    ClassDev& C = P->cls[cl];
    C.mem[C.n_mem++] = (unsigned char)i;
    P->cand[i].cls = (unsigned char)cl;
    P->cand[i].table = 0;
    if (!((eval_mask >> i) & 1u)) continue;
    C.cand[C.n_cand++] = (unsigned char)i;
    if (a.kind != SOP_KIND_LUT) continue;
    const bool dd = (A.dd_mask >> i) & 1u;
    int t = -1;
    for (int q = 0; q < P->n_tables; ++q) {
      const int o = P->table_atom[q];
      const bool odd = (A.dd_mask >> o) & 1u;
      if (P->table_cls[q] != cl || odd != dd) continue;
      if ((a.negated ? P->table_neg[q] : P->table_pos[q]) != 255) continue;   // one candidate per table and sign
      if (dd ? (A.atoms[o].n_entries == a.n_entries) : same_table(A.atoms[o], a)) t = q;
    }
    if (t < 0) {
      if (P->n_tables == SOP_MAX_TABLES) return SOP_ERR_ALPHABET;
      t = P->n_tables++;
      P->table_atom[t] = (unsigned char)i;
      P->table_cls[t] = (unsigned char)cl;
      P->table_pos[t] = P->table_neg[t] = 255;
    }
    (a.negated ? P->table_neg[t] : P->table_pos[t]) = (unsigned char)i;
    P->cls_tables[cl] |= (unsigned char)(1u << t);
    P->cand[i].table = (unsigned char)t;
  }
  // cell geometry per LUT class: cell width (in u) below the smallest threshold gap, a power of two
  int rows = 1;
  for (int c = 0; c < P->n_classes; ++c) {
    ClassDev& C = P->cls[c];
    if (C.kind != SOP_KIND_LUT) continue;
    double gap = 1e30;
    bool any_dd = false;
    for (int q = 0; q < P->n_tables; ++q) {
      if (P->table_cls[q] != c) continue;
      const int o = P->table_atom[q];
      if ((A.dd_mask >> o) & 1u) { any_dd = true; continue; }
      gap = fmin(gap, min_threshold_gap(A.atoms[o]));
    }
    if (gap > C.tmax) gap = C.tmax / 8.0;
    if (any_dd) gap = fmin(gap, C.tmax / 48.0);           // a data-derived table: assume a finer grid
    int e = (int)floor(log2(gap * 0.999));
    double h = ldexp(1.0, e);
    const double reach = 1.25 * C.tmax;                    // scale rounding can push |u| a little above tmax
    while (2 * (int)ceil(reach / h) + 1 > 257) h *= 2.0;   // bound the table size
    C.c_half = (int)ceil(reach / h);
    C.invh = (float)(1.0 / h);
    rows = rows > 2 * C.c_half + 1 ? rows : 2 * C.c_half + 1;
  }
  P->rows = rows;
  P->a_pad = n | 1;
  // slots: pair-type first (singles as (a, a)), then signed.  With keep_loaded an entry whose candidates were all
  // evaluated by an earlier call is not formed again: the tables hold it.
  P->keep_loaded = keep_loaded;
  int ns = 0;
  auto has = [present](int i) { return ((present >> i) & 1u) != 0; };
  auto old = [keep_loaded, load_mask](int i) { return keep_loaded && ((load_mask >> i) & 1u) != 0; };
  for (int a = 0; a < n; ++a) {
    if (!has(a) || old(a)) continue;
    P->slots[ns].type = 0; P->slots[ns].i0 = P->slots[ns].i1 = (unsigned char)a; ++ns;
  }
  for (int a = 0; a < n && !singles_only; ++a)
    for (int b = a + 1; b < n; ++b) {
      if (!has(a) || !has(b) || (old(a) && old(b))) continue;
      if (A.atoms[a].kind != SOP_KIND_LUT || A.atoms[b].kind != SOP_KIND_LUT || A.atoms[a].n_bits != A.atoms[b].n_bits) continue;
      P->slots[ns].type = 0; P->slots[ns].i0 = (unsigned char)a; P->slots[ns].i1 = (unsigned char)b; ++ns;
    }
  P->n_pair_slots = ns;
  if (F.sign_bits && !singles_only) {
    bool base[SOP_MAX_ATOMS];
    for (int i = 0; i < n; ++i) {
      base[i] = false;
      if (i + 1 >= n || !has(i) || !has(i + 1)) continue;
      const sop_atom &a = A.atoms[i], &b = A.atoms[i + 1];
      if (a.kind != SOP_KIND_LUT || b.kind != SOP_KIND_LUT || a.negated || !b.negated || a.tmax != b.tmax) continue;
      const bool da = (A.dd_mask >> i) & 1u, db = (A.dd_mask >> (i + 1)) & 1u;
      base[i] = (da && db && a.n_entries == b.n_entries) || (!da && !db && same_table(a, b));
    }
    for (int i = 0; i < n; ++i)
      if (base[i]) P->base_atom[P->n_bases++] = (unsigned char)i;
    for (int i = 0; i < n; ++i)
      for (int j = i; j < n; ++j) {
        if (!base[i] || !base[j] || A.atoms[i].n_bits != A.atoms[j].n_bits) continue;
        if (old(i) && old(i + 1) && old(j) && old(j + 1)) continue;
        P->slots[ns].type = 1; P->slots[ns].i0 = (unsigned char)i; P->slots[ns].i1 = (unsigned char)j; ++ns;   // base atoms
      }
  }
  if (ns > MAX_SLOTS) return SOP_ERR_ALPHABET;
  P->n_slots = ns;
  // tasks of the reduction: repeatedly the candidate with the most entries still to form on one side of it (as their
  // first candidate, the one that keeps a tie, or as their second) becomes an anchor and takes up to four of them as
  // partners; its own (single) entry rides with its first task.  Signed entries (type 1) make tasks of their own.
  {
    bool done[MAX_SLOTS];
    int self_of[2][SOP_MAX_ATOMS];
    bool self_used[2][SOP_MAX_ATOMS];
    for (int ty = 0; ty < 2; ++ty)
      for (int c = 0; c < SOP_MAX_ATOMS; ++c) { self_of[ty][c] = -1; self_used[ty][c] = false; }
    for (int i = 0; i < ns; ++i) {
      done[i] = P->slots[i].i0 == P->slots[i].i1;
      if (done[i]) self_of[P->slots[i].type][P->slots[i].i0] = i;
    }
    int nt = 0;
    for (;;) {
      int cnt[2][2][SOP_MAX_ATOMS] = {};          // [type][side][candidate]; side 0: the candidate is the entry's first
      for (int i = 0; i < ns; ++i)
        if (!done[i]) { ++cnt[P->slots[i].type][0][P->slots[i].i0]; ++cnt[P->slots[i].type][1][P->slots[i].i1]; }
      int pt = -1, pside = 0, pc = 0;
      for (int ty = 0; ty < 2; ++ty)
        for (int side = 0; side < 2; ++side)
          for (int c = 0; c < SOP_MAX_ATOMS; ++c) {
            // at most four partners ride with one anchor, so more than four entries count like four
            const int v = cnt[ty][side][c] < TASK_PART ? cnt[ty][side][c] : TASK_PART;
            const int best = pt < 0 ? 0 : (cnt[pt][pside][pc] < TASK_PART ? cnt[pt][pside][pc] : TASK_PART);
            if (v > best) { pt = ty; pside = side; pc = c; }
          }
      if (pt < 0) break;
      if (nt == MAX_TASKS) return SOP_ERR_ALPHABET;
      TaskDev& t = P->tasks[nt++];
      memset(&t, 0, sizeof(t));
      t.anchor = (unsigned char)pc;
      t.sgn = (unsigned char)pt;
      t.rev = (unsigned char)pside;
      t.self_slot = 255;
      if (self_of[pt][pc] >= 0 && !self_used[pt][pc]) { t.self_slot = (unsigned char)self_of[pt][pc]; self_used[pt][pc] = true; }
      for (int i = 0; i < ns && t.n_part < TASK_PART; ++i) {
        if (done[i] || P->slots[i].type != pt || (pside ? P->slots[i].i1 : P->slots[i].i0) != pc) continue;
        const int q = t.n_part++;
        t.part[q] = pside ? P->slots[i].i0 : P->slots[i].i1;
        t.slot[q] = (unsigned char)i;
        done[i] = true;
      }
    }
    for (int ty = 0; ty < 2; ++ty)
      for (int c = 0; c < SOP_MAX_ATOMS; ++c) {
        if (self_of[ty][c] < 0 || self_used[ty][c]) continue;
        if (nt == MAX_TASKS) return SOP_ERR_ALPHABET;
        TaskDev& t = P->tasks[nt++];
        memset(&t, 0, sizeof(t));
        t.anchor = (unsigned char)c; t.sgn = (unsigned char)ty; t.self_slot = (unsigned char)self_of[ty][c];
      }
    // heaviest first (a signed task costs about twice as much per entry: two columns per candidate)
    auto weight = [](const TaskDev& t) { return (2 + 3 * (int)t.n_part) * (t.sgn ? 2 : 1); };
    for (int i = 1; i < nt; ++i)
      for (int j = i; j > 0 && weight(P->tasks[j]) > weight(P->tasks[j - 1]); --j) { const TaskDev x = P->tasks[j]; P->tasks[j] = P->tasks[j - 1]; P->tasks[j - 1] = x; }
    P->n_tasks = nt;
  }
  return SOP_OK;
}

// Seats of one launch of the reduction: tasks [task0, task0 + n) dealt to the eight warps, always to the warp with the
// least work so far that still has a free seat; the columns to fetch and their places in the tile buffers; one
// accumulator seat per entry.  Returns the largest number of tasks on one warp.
static int deal_tasks(const Plan& P, int task0, int n, SeatsDev* seats) {
  int load[8] = {0}, used[8] = {0};
  memset(seats, 0, sizeof(*seats));
  memset(seats->task, 255, sizeof(seats->task));
  memset(seats->col_slot, 255, sizeof(seats->col_slot));
  memset(seats->sb_slot, 255, sizeof(seats->sb_slot));
  int tpw = 0;
  unsigned cand = 0, bases = 0;
  for (int i = 0; i < n; ++i) {
    const TaskDev& t = P.tasks[task0 + i];
    int w = -1;
    for (int x = 0; x < 8; ++x)
      if (used[x] < MAX_TPW && (w < 0 || load[x] < load[w])) w = x;
    seats->task[w][used[w]++] = (unsigned char)(task0 + i);
    load[w] += 2 + 3 * (int)t.n_part;
    tpw = tpw > used[w] ? tpw : used[w];
    unsigned m = 1u << t.anchor;
    for (int q = 0; q < t.n_part; ++q) m |= 1u << t.part[q];
    if (t.sgn) { bases |= m; cand |= m | (m << 1); }     // a base atom stands for itself and its negation
    else cand |= m;
  }
  for (int a = 0; a < P.n_atoms; ++a) {
    if ((cand >> a) & 1u) { seats->col_slot[a] = (unsigned char)seats->n_cols; seats->cols[seats->n_cols++] = (unsigned char)a; }
    if ((bases >> a) & 1u) { seats->sb_slot[a] = (unsigned char)seats->n_bases; seats->bases[seats->n_bases++] = (unsigned char)a; }
  }
  for (int w = 0; w < 8; ++w)
    for (int k = 0; k < MAX_TPW; ++k) {
      if (seats->task[w][k] == 255) continue;
      seats->acc0[w][k] = (unsigned short)seats->n_seats;
      const TaskDev& t = P.tasks[seats->task[w][k]];
      seats->n_seats += (t.self_slot != 255 ? 1 : 0) + t.n_part;
    }
  return tpw > 0 ? tpw : 1;
}

size_t sweep_smem_bytes(const Plan& P) {
  size_t b = (size_t)P.n_tables * P.rows * 16 * 8;
  b += SOP_MAX_TABLES * 32 * 4 * 2 + SOP_MAX_TABLES * 4 + SOP_MAX_CLASSES * 8;
  return (b + 15) & ~(size_t)15;
}

// the ring of tile buffers, the signed-best columns, the lanes' accumulators; at least the room the closing
// reduction of the last CTA needs
static size_t reduce_smem_bytes(const SeatsDev& S, int n_stage, bool pair = false) {
  const size_t tiles = ((size_t)n_stage * S.n_cols + (pair ? 2 : 1) * (size_t)S.n_bases) * 2 * RTILE * sizeof(float);
  const size_t acc = (size_t)S.n_seats * ACC_BYTES;
  const size_t fin = sizeof(Partial) * (size_t)RTB + 2 * sizeof(sop_pair_stat) * SOP_MAX_ATOMS * SOP_MAX_ATOMS;
  const size_t b = tiles + acc;
  return ((b > fin ? b : fin) + 127) & ~(size_t)127;
}

// Doubles the cell width of the LUT class with the most rows (its tables then hold several thresholds per cell
// where they are dense, and such tables take the exact binary search).  False when no class can shrink further.
// Two tiles per step in the reduction (see reduce_kernel) wherever the shared memory allows; sop_pair_search_tuning
// turns it off (tests compare both paths: the results are the same bit for bit).
static bool g_reduce_pairs = true;

static bool coarsen_cells(Plan* P) {
  int pick = -1;
  for (int c = 0; c < P->n_classes; ++c)
    if (P->cls[c].kind == SOP_KIND_LUT && P->cls[c].c_half > 1 && (pick < 0 || P->cls[c].c_half > P->cls[pick].c_half)) pick = c;
  if (pick < 0) return false;
  ClassDev& C = P->cls[pick];
  C.invh *= 0.5f;
  C.c_half = (int)ceil(1.25 * (double)C.tmax * (double)C.invh);
  if (C.c_half < 1) C.c_half = 1;
  int rows = 1;
  for (int c = 0; c < P->n_classes; ++c)
    if (P->cls[c].kind == SOP_KIND_LUT) rows = rows > 2 * P->cls[c].c_half + 1 ? rows : 2 * P->cls[c].c_half + 1;
  P->rows = rows;
  return true;
}

}  // namespace sop

extern "C" {

int sop_pair_search_tuning(int reduce_tile_pairs) {
  if (reduce_tile_pairs != 0 && reduce_tile_pairs != 1) return SOP_ERR_RANGE;
  sop::g_reduce_pairs = reduce_tile_pairs != 0;
  return SOP_OK;
}

int sop_pair_search_workspace(long long M, long long K, int n_atoms, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (M < 1 || K < 1 || (K % SOP_G) != 0) return SOP_ERR_SHAPE;
  if (n_atoms < 1 || n_atoms > SOP_MAX_ATOMS) return SOP_ERR_ALPHABET;
  *bytes = sop::ws_total();
  return SOP_OK;
}

int sop_pair_search(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                    const sop_scale_fmt* fmt, int k_mode, const sop_atom* atoms, int n_atoms,
                    const float* dd_lut_dev, unsigned dd_mask, unsigned eval_mask, unsigned load_mask, int flags,
                    const sop_search_result* prev_result_dev,
                    sop_pair_stat* pair_table_dev, sop_pair_stat* signed_table_dev,
                    sop_search_result* result_dev, float* block_cos_dev, float* block_sse_dev,
                    void* workspace_dev, size_t workspace_bytes, void* stream) {
  using namespace sop;
  int rc = validate_layer(W_dev, M, K, ldw, c_dev, g);
  if (rc) return rc;
  if (!pair_table_dev || !result_dev) return SOP_ERR_NULL;
  FmtDev F;
  if ((rc = validate_fmt(fmt, &F))) return rc;
  AtomsDev A;
  if ((rc = validate_atoms(atoms, n_atoms, dd_mask, dd_lut_dev, &A))) return rc;
  const bool k_from_result = k_mode == SOP_K_FROM_RESULT;
  if (k_mode != SOP_K_AUTO && !k_from_result && (k_mode < -64 || k_mode > 64)) return SOP_ERR_RANGE;
  if (k_from_result && (!prev_result_dev || prev_result_dev == result_dev)) return SOP_ERR_NULL;
  const long long NB = M * (K / SOP_G);
  // without the caller's per-block arrays the columns live behind the fixed part of the workspace
  const bool own_columns = !block_cos_dev || !block_sse_dev;
  const size_t col_bytes = (((size_t)n_atoms * (size_t)NB * sizeof(float)) + 255) & ~(size_t)255;
  const size_t need = ws_total() + (own_columns ? 2 * col_bytes : 0);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;
  const unsigned all = n_atoms >= 32 ? 0xFFFFFFFFu : ((1u << n_atoms) - 1u);
  eval_mask &= all;
  if ((load_mask & ~all) || (load_mask & eval_mask) || !(eval_mask | load_mask)) return SOP_ERR_ALPHABET;
  if (load_mask && own_columns) return SOP_ERR_NULL;
  if (flags & ~(SOP_SEARCH_SINGLES_ONLY | SOP_SEARCH_SELECT_MSE | SOP_SEARCH_KEEP_LOADED_ENTRIES | SOP_SEARCH_REUSE_PREPASS)) return SOP_ERR_RANGE;
  const bool reuse_prepass = (flags & SOP_SEARCH_REUSE_PREPASS) && !k_from_result;
  const int keep_loaded = (flags & SOP_SEARCH_KEEP_LOADED_ENTRIES) && load_mask ? 1 : 0;
  Plan P;
  if ((rc = build_plan(A, F, k_from_result ? 0 : k_mode, eval_mask, load_mask, flags & SOP_SEARCH_SINGLES_ONLY, keep_loaded, &P))) return rc;
  P.k_from_result = k_from_result ? 1 : 0;
  for (int c = 0; c < P.n_classes; ++c) {
    // the shift of a class is read from a candidate of that class that the earlier call had
    P.cls[c].k_src = -1;
    for (int i = 0; i < P.cls[c].n_mem; ++i)
      if ((load_mask >> P.cls[c].mem[i]) & 1u) { P.cls[c].k_src = P.cls[c].mem[i]; break; }
    if (k_from_result && P.cls[c].scope != 0 && P.cls[c].k_src < 0) return SOP_ERR_RANGE;
  }

  LayerArgs L;
  L.W = (const uint16_t*)W_dev; L.c = c_dev; L.M = M; L.K = K; L.ldw = ldw; L.nbk = K / SOP_G; L.NB = NB;
  cudaStream_t st = (cudaStream_t)stream;
  unsigned char* ws = (unsigned char*)workspace_dev;
  WsHeader* hdr = (WsHeader*)ws;
  unsigned* hist = (unsigned*)(ws + ws_hist_off());
  Partial* partials = (Partial*)(ws + ws_part_off());
  float* cos_cols = own_columns ? (float*)(ws + ws_total()) : block_cos_dev;
  float* sse_cols = own_columns ? (float*)(ws + ws_total() + col_bytes) : block_sse_dev;

  // everything that can refuse the call is decided before the first enqueue
  constexpr size_t SMEM_MAX = 226 * 1024;   // 227 KB per CTA minus the kernels' few static bytes
  size_t smem = sweep_smem_bytes(P);
  while (smem > SMEM_MAX && coarsen_cells(&P)) smem = sweep_smem_bytes(P);   // cell tables too large: coarser cells, exact search where needed
  if (smem > SMEM_MAX) return SOP_ERR_ALPHABET;
  const int sms = num_sms();
  // persistent grid: one CTA per SM, fewer when the layer is small; at least enough threads for one row
  long long grid = (L.NB + TB - 1) / TB;
  if (grid > sms) grid = sms;
  const long long min_grid = (L.nbk + TB - 1) / TB;
  if (grid < min_grid) grid = min_grid;
  if (grid > MAX_GRID) return SOP_ERR_SHAPE;
  // the reduction: up to MAX_TPW tasks per warp and launch, more launches for more tasks; persistent grid over tiles.
  // 16-byte copies need 16-byte aligned column starts and runs: a block count that is a multiple of four.
  constexpr int PER_LAUNCH = (RTB / 32) * MAX_TPW;
  const int n_launch = P.n_tasks ? (P.n_tasks + PER_LAUNCH - 1) / PER_LAUNCH : 1;
  const bool vec = (L.NB % 4) == 0 && (((uintptr_t)cos_cols | (uintptr_t)sse_cols) & 15u) == 0;
  const long long n_tiles = (L.NB + RTILE - 1) / RTILE;
  long long rgrid = n_tiles < (long long)sms * 2 ? n_tiles : (long long)sms * 2;
  if (rgrid < 1) rgrid = 1;
  // a lane counts at most 8 blocks per tile in 16 bits: a CTA takes fewer than 8000 tiles (never near it on a GPU with
  // a hundred SMs: 2^19 tiles at most)
  if (n_tiles / rgrid >= 8000) rgrid = (n_tiles + 7999) / 8000;

  // the header always starts from zero; the histograms (and max|W| behind them) only when this call fills them
  SOP_CUDA_TRY(cudaMemsetAsync(ws, 0, (k_from_result || reuse_prepass) ? ws_hist_off() : ws_part_off(), st));
  if ((rc = profile_mark(SOP_PROFILE_PREPASS, 0, st))) return rc;
  if (reuse_prepass) {
    kselect_kernel<<<1, 256, 0, st>>>(P, F, hist, hdr);
    SOP_CUDA_TRY(cudaGetLastError());
  } else if (!k_from_result) {
    // one read of W: block scales' exponent histogram, max|W|, then the shifts (last CTA)
    long long want = (L.NB + 255) / 256;
    const int pgrid = (int)(want < (long long)sms * 8 ? want : (long long)sms * 8);
    prepass_kernel<<<pgrid, 256, 0, st>>>(L, P, F, hist, hdr);
    SOP_CUDA_TRY(cudaGetLastError());
  }
  if ((rc = profile_mark(SOP_PROFILE_PREPASS, 1, st))) return rc;
  DeviceFacts* facts = device_facts();
  if (!facts->search_attr_set) {
    SOP_CUDA_TRY(cudaFuncSetAttribute(sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_MAX));
#define SOP_REDUCE_ATTR(SE, T, BK, PR) \
  SOP_CUDA_TRY(cudaFuncSetAttribute(reduce_kernel<SE, T, BK, PR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_MAX))
    SOP_REDUCE_ATTR(false, 1, false, false); SOP_REDUCE_ATTR(false, 2, false, false); SOP_REDUCE_ATTR(false, 3, false, false);
    SOP_REDUCE_ATTR(false, 1, true, false); SOP_REDUCE_ATTR(false, 2, true, false); SOP_REDUCE_ATTR(false, 3, true, false);
    SOP_REDUCE_ATTR(true, 1, false, false); SOP_REDUCE_ATTR(true, 2, false, false); SOP_REDUCE_ATTR(true, 3, false, false);
    SOP_REDUCE_ATTR(true, 1, true, false); SOP_REDUCE_ATTR(true, 2, true, false); SOP_REDUCE_ATTR(true, 3, true, false);
    SOP_REDUCE_ATTR(false, 1, true, true); SOP_REDUCE_ATTR(false, 2, true, true); SOP_REDUCE_ATTR(false, 3, true, true);
    SOP_REDUCE_ATTR(true, 1, true, true); SOP_REDUCE_ATTR(true, 2, true, true); SOP_REDUCE_ATTR(true, 3, true, true);
#undef SOP_REDUCE_ATTR
    facts->search_attr_set = true;
  }
  if ((rc = profile_mark(SOP_PROFILE_SWEEP, 0, st))) return rc;
  if (eval_mask) {
    sweep_kernel<<<(int)grid, TB, smem, st>>>(L, P, A, F, hdr, cos_cols, sse_cols, prev_result_dev);
    SOP_CUDA_TRY(cudaGetLastError());
  }
  if ((rc = profile_mark(SOP_PROFILE_SWEEP, 1, st))) return rc;
  if ((rc = profile_mark(SOP_PROFILE_REDUCE, 0, st))) return rc;
  const bool sel_err = (flags & SOP_SEARCH_SELECT_MSE) != 0;
  for (int l = 0; l < n_launch; ++l) {
    const int task0 = l * PER_LAUNCH;
    const int nt = P.n_tasks - task0 < PER_LAUNCH ? P.n_tasks - task0 : PER_LAUNCH;
    SeatsDev seats;
    const int tpw = deal_tasks(P, task0, nt, &seats);
    // as many tile buffers as still let two CTAs share an SM (at most 16 columns, 8 signed-best ones and 120 seats: two
    // buffers always fit one CTA)
    int n_stage = vec ? MAX_STAGE : 1;
    while (n_stage > 2 && reduce_smem_bytes(seats, n_stage) > SMEM_MAX / 2) --n_stage;
    // two tiles at a time when the ring has its four buffers and the second set of signed-best columns still fits
    const bool pair = vec && n_stage == MAX_STAGE && reduce_smem_bytes(seats, n_stage, true) <= SMEM_MAX / 2 && g_reduce_pairs;
    const size_t rs = reduce_smem_bytes(seats, n_stage, pair);
    const int fin = l == n_launch - 1 ? 1 : 0;
#define SOP_LAUNCH_REDUCE(SE, T, BK, PR)                                                                                      \
  reduce_kernel<SE, T, BK, PR><<<(int)rgrid, RTB, rs, st>>>(L, P, seats, n_stage, fin, hdr, partials, cos_cols, sse_cols, pair_table_dev, \
                                                            signed_table_dev, result_dev, prev_result_dev)
#define SOP_LAUNCH_REDUCE_T(SE, BK, PR) \
  do { if (tpw == 1) SOP_LAUNCH_REDUCE(SE, 1, BK, PR); else if (tpw == 2) SOP_LAUNCH_REDUCE(SE, 2, BK, PR); else SOP_LAUNCH_REDUCE(SE, 3, BK, PR); } while (0)
    if (sel_err) { if (pair) SOP_LAUNCH_REDUCE_T(true, true, true); else if (vec) SOP_LAUNCH_REDUCE_T(true, true, false); else SOP_LAUNCH_REDUCE_T(true, false, false); }
    else { if (pair) SOP_LAUNCH_REDUCE_T(false, true, true); else if (vec) SOP_LAUNCH_REDUCE_T(false, true, false); else SOP_LAUNCH_REDUCE_T(false, false, false); }
#undef SOP_LAUNCH_REDUCE_T
#undef SOP_LAUNCH_REDUCE
    SOP_CUDA_TRY(cudaGetLastError());
  }
  if ((rc = profile_mark(SOP_PROFILE_REDUCE, 1, st))) return rc;
  return SOP_OK;
}

}  // extern "C"
