// sop_dd4_lloyd: per-layer data-derived codebook (DD-n) by Lloyd iteration on the pool of blocks
// that the primary codebook reconstructs worst.
//
//   select_kernel<PASS>   three-pass radix select (11 + 11 + 10 bits) of the pool_rank-th worst block by
//                         its ranking key (cosine ascending, or error descending); each pass re-derives
//                         the prefix from the previous histograms with a CTA-wide scan.  Not run when the
//                         caller fixes the pool threshold.
//   lloyd_setup_kernel    threshold key from the last histogram (or from the given threshold), max(c),
//                         the shift k, the initial table (FMTa, reversed and negated if FMTa is a negated
//                         atom), the per-channel weight table omega = c / max(c) (or 1), and the first
//                         iteration descriptor.
//   pool_list_kernel      compacts the indices of the pool blocks into a dense list.
//   pool_cache_kernel     the pool elements never change between iterations, only the table does:
//                         (u, omega) of every pool element is computed once (u = w / scale) and kept
//                         in tiles of 4096 elements, each counting-sorted by the cell of u on a
//                         uniform grid (641 cells of width 2^-8); the start of every cell inside
//                         every tile is kept too, and per cell, over the whole pool, the int64
//                         fixed-point sums of omega and omega u and the moments
//                         sum omega, sum omega u, sum omega u^2.
//   lloyd_iteration       one iteration (device function).  A cell that holds no decision threshold of
//                         the current table lies inside one entry's interval: its elements are
//                         accounted for by the cell's sums and moments, without touching them.  Only
//                         the cells that hold a threshold are walked element by element, exactly: one
//                         warp per tile, the lanes taking contiguous shares of those cells' elements.
//                         Per-entry sums are int64 fixed point (exactly associative: the table is the
//                         same bit for bit as a sequential sum over all elements gives), distortion
//                         FP64.  The CTA that finishes last turns the sums into centroids, snaps them to
//                         bf16, sorts, publishes the next iteration's descriptor and clears the
//                         accumulators.
//   lloyd_persistent_kernel  all iterations in one cooperative launch; between iterations the CTAs wait,
//                         bounded, for the flag of the CTA that finished last.
//   lloyd_split_kernel    one iteration per launch: used where the grid cannot be resident at once.
#include <math.h>
#include <stddef.h>
#include <string.h>

#include "sop_device.cuh"

namespace sop {

constexpr int LTB = 256;
constexpr int SETUP_TB = 1024;
constexpr int SOP_MAX_LLOYD_ITERS = 64;
constexpr int SORT_CHALF = 320;                 // lookup grid on u: cell width 2^-8, rows cover |u| <= 1.25,
constexpr int SORT_ROWS = 2 * SORT_CHALF + 1;   // the first and last row take everything beyond
constexpr float SORT_INVH = 256.0f;
constexpr float SORT_MAGIC = 12582912.0f;       // 1.5 * 2^23

struct CellEntry { float thr; unsigned codes; };   // codes: lo | hi << 8; 0xFFFF: more than one threshold in the cell

// Everything an iteration reads about the current table, contiguous so that a CTA fetches it with one
// load per thread: the table (padded with its last entry), the exact decision thresholds (+inf padded)
// and the lookup cell of every threshold (ascending, like the thresholds).
struct IterDesc {
  int n_entries;
  int pad[3];
  float lut[SOP_MAX_ENTRIES];
  float tau[SOP_MAX_ENTRIES];
  int thr_cell[SOP_MAX_ENTRIES];
};

struct LloydWs {
  // radix select state
  unsigned hist[3][2048];
  // iteration state
  unsigned long long accN[SOP_MAX_ENTRIES];
  long long accS[SOP_MAX_ENTRIES];
  double accD;
  unsigned tau_key;  // pool threshold as a ranking key: the pool is every block whose key is not above it
  float cmax;
  int k;
  int fmta;
  unsigned done;         // CTAs of the running iteration that have added their sums (one launch per iteration)
  // one launch for all iterations: CTAs that have added their sums in iteration i, and the flag that the
  // table of iteration i + 1 is published; never reset (the header is cleared before every call)
  unsigned arrive[SOP_MAX_LLOYD_ITERS + 1];
  unsigned ready[SOP_MAX_LLOYD_ITERS + 1];
  unsigned error;        // a CTA gave up waiting for a flag
  unsigned list_count;   // blocks appended to the pool list
  int pad;
  // the current codebook, rewritten by whoever changes it (set-up, then each update)
  IterDesc desc;
  // per cell, over the whole pool (filled once by pool_cache_kernel)
  unsigned long long cellN[SORT_ROWS];     // sum fix(omega)
  long long cellS[SORT_ROWS];              // sum fix(omega u)
  double cellA[3][SORT_ROWS];              // sum omega, sum omega u, sum omega u^2
  long long cellQ[SORT_ROWS];              // sum fix((omega u) u): the exact second moment the grid-constrained construction needs
  // not cleared per call: scratch of the dynamic programme, and where the last run starts per (number of runs, last cell)
  short dp_cut[SOP_MAX_ENTRIES][SORT_ROWS];
  long long dp_scratch[4 * (SORT_ROWS + 1) + 2 * SORT_ROWS];
};

struct LloydArgs {
  const uint16_t* W;
  const float* c;
  const float* cosrow_base;   // [n_atoms x NB]
  long long M, K, ldw, nbk, NB;
  long long pool_rank;
  int k_mode, fmta_index, n_atoms;
  int flags;                  // SOP_LLOYD_*
  float pool_threshold;       // with SOP_LLOYD_POOL_THRESHOLD
  float* omega;               // workspace: K floats, c / max(c)
  unsigned* pool_idx;         // workspace: NB words, indices of the pool blocks
  uint2* cache;               // workspace: pairs (u, omega) as bit patterns, tiles of TILE_ELEMS sorted by cell
  unsigned short* tile_start; // workspace: [tiles][SORT_ROWS + 1] first sorted position of every cell in every tile
};

static size_t lloyd_off_omega() { return (sizeof(LloydWs) + 255) & ~(size_t)255; }
static size_t lloyd_off_idx(long long K) { return lloyd_off_omega() + (((size_t)K * 4 + 255) & ~(size_t)255); }
static size_t lloyd_off_cache(long long M, long long K) { return lloyd_off_idx(K) + ((((size_t)M * (size_t)(K / SOP_G)) * 4 + 255) & ~(size_t)255); }
constexpr int TILE_ELEMS = LTB * SOP_G;   // pool elements per cache tile: one block per thread of a CTA
static size_t lloyd_off_tiles(long long M, long long K) {
  const size_t nb = (size_t)M * (size_t)(K / SOP_G);
  return lloyd_off_cache(M, K) + ((nb + LTB - 1) / LTB) * TILE_ELEMS * sizeof(uint2);   // whole tiles
}
static size_t lloyd_ws_bytes(long long M, long long K) {
  const size_t nb = (size_t)M * (size_t)(K / SOP_G);
  return lloyd_off_tiles(M, K) + ((((nb + LTB - 1) / LTB) * (SORT_ROWS + 1) * sizeof(unsigned short) + 255) & ~(size_t)255);
}

__device__ __forceinline__ unsigned cos_key(float x) {
  const unsigned b = __float_as_uint(__fadd_rn(x, 0.0f));   // -0 -> +0
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
// Ranking key of a block: ascending key = worst block first.  By cosine the worst is the smallest value,
// by error (SOP_LLOYD_POOL_BY_ERROR) the largest.
__device__ __forceinline__ unsigned pool_key(float x, int flags) {
  const unsigned k = cos_key(x);
  return (flags & SOP_LLOYD_POOL_BY_ERROR) ? ~k : k;
}

__device__ __forceinline__ int resolve_fmta(const LloydArgs& a, const sop_search_result* res) {
  int f = a.fmta_index == SOP_FMTA_FROM_RESULT ? res->best_single : a.fmta_index;
  return max(0, min(a.n_atoms - 1, f));
}

// CTA-wide (a multiple of 32 threads, at most 1024): the bin of `hist` (nb <= 2048 bins) holding the
// element of 1-based rank `rank`; *before = elements in lower bins, *count = elements in that bin.
__device__ void find_bin(const unsigned* __restrict__ hist, int nb, long long rank, int* bin, long long* before, unsigned* count) {
  __shared__ long long s_warp[32];
  __shared__ int s_bin;
  __shared__ long long s_before;
  __shared__ unsigned s_cnt;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int per = (nb + nt - 1) / nt;
  const int b0 = tid * per;
  long long local = 0;
  for (int i = 0; i < per; ++i)
    if (b0 + i < nb) local += hist[b0 + i];
  long long incl = local;
  for (int o = 1; o < 32; o <<= 1) {
    const long long v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  long long base = 0;
  for (int w = 0; w < warp; ++w) base += s_warp[w];
  const long long excl = base + incl - local;
  if (local > 0 && excl < rank && rank <= excl + local) {
    long long run = excl;
    for (int i = 0; i < per; ++i) {
      const unsigned h = hist[b0 + i];
      if (run + h >= rank) { s_bin = b0 + i; s_before = run; s_cnt = h; break; }
      run += h;
    }
  }
  __syncthreads();
  *bin = s_bin; *before = s_before; *count = s_cnt;
  __syncthreads();
}

// After pass p the selected element lies in one bin of hist[p]; the key prefix, the rank inside
// that bin and the number of elements below it follow from the histograms of the passes so far.
__device__ void derive_prefix(const LloydWs* ws, long long pool_rank, int passes, unsigned* prefix, long long* rank_out,
                              long long* below_out, unsigned* last_count) {
  long long rank = pool_rank, below = 0;
  unsigned pre = 0, cnt = 0;
  for (int p = 0; p < passes; ++p) {
    int bin;
    long long before;
    find_bin(ws->hist[p], p < 2 ? 2048 : 1024, rank, &bin, &before, &cnt);
    rank -= before;
    below += before;
    pre = (pre << (p < 2 ? 11 : 10)) | (unsigned)bin;
  }
  *prefix = pre; *rank_out = rank; *below_out = below; *last_count = cnt;
}

template <int PASS>
__global__ void __launch_bounds__(LTB) select_kernel(LloydArgs a, const sop_search_result* __restrict__ res, LloydWs* __restrict__ ws) {
  __shared__ unsigned sh[2048];
  for (int i = threadIdx.x; i < 2048; i += LTB) sh[i] = 0;
  unsigned prefix = 0, cnt;
  long long rank, below;
  if (PASS > 0) derive_prefix(ws, a.pool_rank, PASS, &prefix, &rank, &below, &cnt);
  __syncthreads();
  const float* row = a.cosrow_base + (size_t)resolve_fmta(a, res) * a.NB;
  auto count = [&](float x) {
    const unsigned key = pool_key(x, a.flags);
    if (PASS == 0) atomicAdd(&sh[key >> 21], 1u);
    else if (PASS == 1) { if ((key >> 21) == prefix) atomicAdd(&sh[(key >> 10) & 2047u], 1u); }
    else { if ((key >> 10) == prefix) atomicAdd(&sh[key & 1023u], 1u); }
  };
  // sixteen keys per thread and round, their loads in flight together (the pass is bound by memory latency otherwise):
  // four 128-bit loads where the row is 16-byte aligned, else four rounds of four single loads
  const long long stride = (long long)gridDim.x * LTB;
  const long long nv = (reinterpret_cast<uintptr_t>(row) & 15u) == 0 ? a.NB / 4 : 0;      // whole float4 groups
  for (long long i = (long long)blockIdx.x * LTB + threadIdx.x; i < nv; i += 4 * stride) {
    float4 v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) v[q] = i + q * stride < nv ? __ldg(reinterpret_cast<const float4*>(row) + i + q * stride) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (i + q * stride >= nv) break;
      count(v[q].x); count(v[q].y); count(v[q].z); count(v[q].w);
    }
  }
  for (long long i = 4 * nv + (long long)blockIdx.x * LTB + threadIdx.x; i < a.NB; i += 4 * stride) {
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) v[q] = i + q * stride < a.NB ? __ldg(row + i + q * stride) : 0.0f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (i + q * stride >= a.NB) break;
      count(v[q]);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 2048; i += LTB)
    if (sh[i]) atomicAdd(&ws->hist[PASS][i], sh[i]);
}

__device__ __forceinline__ int sort_cell(float u) {
  const float t = fminf(fmaxf(__fmaf_rn(u, SORT_INVH, SORT_MAGIC + (float)SORT_CHALF), SORT_MAGIC), SORT_MAGIC + (float)(2 * SORT_CHALF));
  return (int)(__float_as_uint(t) - __float_as_uint(SORT_MAGIC));
}

// Threads 0..31 of a CTA; s_lut holds the sorted table padded to 32 entries with its last value.
// Thread j writes entry j, its decision threshold (the same rule as build_thresholds: the largest
// fp32 <= the midpoint, a repeated entry takes the threshold above it, +inf from n_entries - 1 on)
// and the lookup cell of that threshold.  sort_cell is monotone, so an element in a lower cell than a
// threshold's is below the threshold and one in a higher cell is above it: only the elements of the
// cells listed here need the comparison itself.
__device__ void lloyd_publish_desc(LloydWs* ws, const float* s_lut, int ne) {
  const int j = threadIdx.x;
  if (j >= SOP_MAX_ENTRIES) return;
  int jj = j;
  while (jj < ne - 1 && s_lut[jj] == s_lut[jj + 1]) ++jj;
  const float t = jj < ne - 1 ? __double2float_rd(0.5 * ((double)s_lut[jj] + (double)s_lut[jj + 1])) : __int_as_float(0x7F800000);
  ws->desc.lut[j] = s_lut[j];
  ws->desc.tau[j] = t;
  ws->desc.thr_cell[j] = j < ne - 1 ? sort_cell(t) : SORT_ROWS;
  if (j == 0) ws->desc.n_entries = ne;
}

__global__ void __launch_bounds__(SETUP_TB) lloyd_setup_kernel(LloydArgs a, AtomsDev A, const sop_search_result* __restrict__ res,
                                                               LloydWs* __restrict__ ws, double* __restrict__ distortion, int iters) {
  unsigned prefix = 0, cnt = 0;
  long long rank = 0, below = 0;
  if (a.flags & SOP_LLOYD_POOL_THRESHOLD) prefix = pool_key(a.pool_threshold, a.flags);   // the caller fixes the threshold
  else derive_prefix(ws, a.pool_rank, 3, &prefix, &rank, &below, &cnt);
  __shared__ float red[SETUP_TB / 32];
  __shared__ float s_cmax;
  __shared__ float s_lut[SOP_MAX_ENTRIES];
  __shared__ int s_ne;
  float mx = 0.0f;
  for (long long i = threadIdx.x; i < a.K; i += SETUP_TB) mx = fmaxf(mx, __ldg(a.c + i));
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = red[0];
    for (int w = 1; w < SETUP_TB / 32; ++w) t = fmaxf(t, red[w]);
    s_cmax = t;
  }
  __syncthreads();
  const float cmax = s_cmax;
  for (long long i = threadIdx.x; i < a.K; i += SETUP_TB) {
    const float om = (a.flags & SOP_LLOYD_UNIFORM_WEIGHTS) ? 1.0f : (cmax > 0.0f ? __fdiv_rn(__ldg(a.c + i), cmax) : 0.0f);
    a.omega[i] = om;
  }
  if (threadIdx.x == 0) {
    ws->tau_key = prefix;          // full 32-bit key after three passes (or the key of the given threshold)
    ws->cmax = cmax;
    const int f = resolve_fmta(a, res);
    ws->fmta = f;
    ws->k = a.k_mode == SOP_K_FROM_RESULT ? res->k[f] : a.k_mode;
    const sop_atom& at = A.atoms[f];
    const int ne = at.n_entries;
    s_ne = ne;
    const bool dd = (A.dd_mask >> f) & 1u;
    for (int j = 0; j < SOP_MAX_ENTRIES; ++j) {
      const int src = at.negated ? ne - 1 - min(j, ne - 1) : min(j, ne - 1);   // padded with the last entry
      float v = dd ? A.dd_lut[src] : at.lut[src];
      if (at.negated) v = -v;
      s_lut[j] = v;
    }
    for (int j = 0; j < SOP_MAX_ENTRIES; ++j) { ws->accN[j] = 0; ws->accS[j] = 0; }
    ws->accD = 0.0;
    ws->done = 0;
    ws->list_count = 0;
    // "not finished": the closing iteration overwrites it with the final distortion (never negative)
    distortion[iters] = -1.0;
  }
  for (int r = threadIdx.x; r < SORT_ROWS; r += SETUP_TB) {
    ws->cellN[r] = 0; ws->cellS[r] = 0; ws->cellQ[r] = 0; ws->cellA[0][r] = 0.0; ws->cellA[1][r] = 0.0; ws->cellA[2][r] = 0.0;
  }
  __syncthreads();
  lloyd_publish_desc(ws, s_lut, s_ne);
}

// Dense list of the pool blocks.  A thread takes sixteen consecutive blocks per round (four 128-bit loads in flight
// where the row is 16-byte aligned); the CTA's count goes to the list's counter once per round (a warp scan of the
// threads' counts, then a scan of the eight warp totals).  The order of the list depends on the scheduling of the
// CTAs; nothing downstream depends on it (integer sums, and an FP64 sum compared with a tolerance).
constexpr int LIST_PER_THREAD = 16;
__global__ void __launch_bounds__(LTB) pool_list_kernel(LloydArgs a, LloydWs* __restrict__ ws) {
  __shared__ unsigned s_cnt[LTB / 32];
  __shared__ unsigned s_base;
  const unsigned tau_key = ws->tau_key;
  const float* row = a.cosrow_base + (size_t)ws->fmta * a.NB;
  const bool vec = (reinterpret_cast<uintptr_t>(row) & 15u) == 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long stride = (long long)gridDim.x * LTB * LIST_PER_THREAD;
  const long long n_round = (a.NB + stride - 1) / stride;
  long long i = ((long long)blockIdx.x * LTB + threadIdx.x) * LIST_PER_THREAD;
  for (long long r = 0; r < n_round; ++r, i += stride) {
    unsigned in = 0;
    if (vec && i + LIST_PER_THREAD <= a.NB) {
      float4 v[LIST_PER_THREAD / 4];
#pragma unroll
      for (int q = 0; q < LIST_PER_THREAD / 4; ++q) v[q] = __ldg(reinterpret_cast<const float4*>(row + i) + q);
#pragma unroll
      for (int q = 0; q < LIST_PER_THREAD / 4; ++q) {
        in |= (pool_key(v[q].x, a.flags) <= tau_key ? 1u : 0u) << (4 * q);
        in |= (pool_key(v[q].y, a.flags) <= tau_key ? 1u : 0u) << (4 * q + 1);
        in |= (pool_key(v[q].z, a.flags) <= tau_key ? 1u : 0u) << (4 * q + 2);
        in |= (pool_key(v[q].w, a.flags) <= tau_key ? 1u : 0u) << (4 * q + 3);
      }
    } else {
#pragma unroll 4
      for (int q = 0; q < LIST_PER_THREAD; ++q)
        if (i + q < a.NB && pool_key(__ldg(row + i + q), a.flags) <= tau_key) in |= 1u << q;
    }
    const unsigned mine = (unsigned)__popc(in);
    unsigned incl = mine;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_cnt[warp] = incl;
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned tot = 0;
      for (int w = 0; w < LTB / 32; ++w) { const unsigned c = s_cnt[w]; s_cnt[w] = tot; tot += c; }
      s_base = tot ? atomicAdd(&ws->list_count, tot) : 0u;
    }
    __syncthreads();
    unsigned at = s_base + s_cnt[warp] + incl - mine;
    for (unsigned rest = in; rest; rest &= rest - 1u) a.pool_idx[at++] = (unsigned)(i + (__ffs((int)rest) - 1));
    __syncthreads();             // s_cnt and s_base are rewritten in the next round
  }
}


// u of the 16 elements of pool block `blk`
__device__ __forceinline__ void pool_block_u(const LloydArgs& a, const FmtDev& F, int k, unsigned blk, float (&u)[16], unsigned& j_out) {
  const unsigned nbk = (unsigned)a.nbk;
  const unsigned m = blk / nbk, j = blk - m * nbk;
  j_out = j;
  const uint4* p = reinterpret_cast<const uint4*>(a.W + (long long)m * a.ldw + (long long)j * SOP_G);
  const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
  const uint32_t wb[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
  uint32_t mb = 0;       // the maximum of the sixteen 15-bit magnitude patterns, two per word at a time
#pragma unroll
  for (int q = 0; q < 8; ++q) mb = __vmaxu2(mb, wb[q] & 0x7FFF7FFFu);
  mb = max(mb & 0xFFFFu, mb >> 16);
  const float amax = __uint_as_float(mb << 16);
  const float s_hat = scale_quantize(amax, k, F).s_hat;    // a DD table declares tmax = 1
  const float rcp = s_hat > 0.0f ? __frcp_rn(s_hat) : 0.0f;
#pragma unroll
  for (int e = 0; e < 16; ++e) u[e] = __fmul_rn((e & 1) ? bf16hi(wb[e >> 1]) : bf16lo(wb[e >> 1]), rcp);
}

// One tile = the 256 pool blocks (4096 elements) of one CTA pass.  The tile is counting-sorted by
// cell in shared memory.  Sorted position p is stored at slot (p & ~15) | ((p ^ (p >> 4)) & 15): the elements of a
// cell stay next to each other in memory (an iteration reads the split cells' runs, a few 32-byte sectors each,
// instead of one sector per element), and the thread that sums positions 16 t .. 16 t + 15 of the tile in shared
// memory meets no bank conflict (the slots of one step differ in their low four bits over a half-warp).  The
// exclusive-or keeps a group of four consecutive positions inside one 32-byte sector.
// A tile that the pool does not fill is padded with (u, omega) = (0, 0): such elements add nothing.
__device__ __forceinline__ unsigned tile_slot(unsigned p) { return (p & ~15u) | ((p ^ (p >> 4)) & 15u); }
__device__ __forceinline__ long long fix24(float v) {   // llrint(v * 2^24): exact scaling, one rounding to an integer
  const float s = __fmul_rn(v, 16777216.0f);
  return fabsf(s) < 2147483648.0f ? (long long)__float2int_rn(s) : __float2ll_rn(s);
}

constexpr int CELL_LIMBS = 14;            // Lloyd: counts (2), sum omega u (3), three moments (3 each)
constexpr int CELL_LIMBS_DP = 8;          // dynamic programme: counts (2), sum omega u (3), sum omega u u (3)
constexpr int CELL_SPILL_TILES_MAX = 128;     // a low limb takes at most 258 * (2^16 - 1) per tile: 128 tiles stay below 2^32
constexpr int TILES_PER_WARP_MAX = 4;         // tiles a warp of an iteration CTA walks between two folds of its limb sums (see flush_limbs)

// Launch-shape parameters of the pool cache and of the iteration grid.  The defaults are the largest values the
// limb arithmetic allows; sop_dd4_lloyd_tuning lowers them (tests reach the mid-loop spill and a multi-tile warp
// share on small layers that way).  Results do not depend on them.
struct LloydTune { int spill_tiles, cache_ctas, tiles_per_warp, iter_ctas; };
static LloydTune g_tune = {CELL_SPILL_TILES_MAX, 0, TILES_PER_WARP_MAX, 0};
constexpr double MOMENT_UNIT = 1099511627776.0;   // 2^40

__device__ __forceinline__ void add_limbs3(unsigned (*cL)[SORT_ROWS], int first, int cell, long long v) {
  atomicAdd(&cL[first][cell], (unsigned)(v & 0xFFFFll));
  atomicAdd(&cL[first + 1][cell], (unsigned)((v >> 16) & 0xFFFFll));
  atomicAdd(&cL[first + 2][cell], (unsigned)(int)(v >> 32));
}

// One run of elements of one cell (at most 16): fix(omega) sums below 2^28, fix(omega u) and fix(omega u u) sums below
// 2^37 in magnitude, moments below 2^6 in magnitude (so below 2^46 in units of 2^-40).
// DP: the sums that the grid-constrained construction reads (fix(omega), fix(omega u), fix(omega u u)); otherwise those of
// the Lloyd iterations (fix(omega), fix(omega u) and the three moments).
template <bool DP>
__device__ __forceinline__ void flush_cell(unsigned (*cL)[SORT_ROWS], int cell, unsigned long long n, unsigned long long sv,
                                           unsigned long long sq, double a0, double a1, double a2) {
  atomicAdd(&cL[0][cell], (unsigned)(n & 0xFFFFull));
  atomicAdd(&cL[1][cell], (unsigned)(n >> 16));
  add_limbs3(cL, 2, cell, (long long)sv);
  if (DP) {
    add_limbs3(cL, 5, cell, (long long)sq);
  } else {
    add_limbs3(cL, 5, cell, __double2ll_rn(a0 * MOMENT_UNIT));
    add_limbs3(cL, 8, cell, __double2ll_rn(a1 * MOMENT_UNIT));
    add_limbs3(cL, 11, cell, __double2ll_rn(a2 * MOMENT_UNIT));
  }
}

__device__ __forceinline__ long long join_limbs3(unsigned (*cL)[SORT_ROWS], int first, int cell) {
  return (long long)cL[first][cell] + ((long long)cL[first + 1][cell] << 16) + ((long long)(int)cL[first + 2][cell] << 32);
}

// Whole CTA, after a barrier: the CTA's limbs are added to the per-cell sums of the pool and cleared.
template <bool DP>
__device__ void spill_cells(unsigned (*cL)[SORT_ROWS], LloydWs* ws) {
  for (int r = threadIdx.x; r < SORT_ROWS; r += blockDim.x) {
    const unsigned long long n = (unsigned long long)cL[0][r] + ((unsigned long long)cL[1][r] << 16);
    const long long sv = join_limbs3(cL, 2, r);
    if (n) atomicAdd(&ws->cellN[r], n);
    if (sv) atomicAdd(reinterpret_cast<unsigned long long*>(&ws->cellS[r]), (unsigned long long)sv);
    if (DP) {
      const long long sq = join_limbs3(cL, 5, r);
      if (sq) atomicAdd(reinterpret_cast<unsigned long long*>(&ws->cellQ[r]), (unsigned long long)sq);
    } else {
      const long long m0 = join_limbs3(cL, 5, r), m1 = join_limbs3(cL, 8, r), m2 = join_limbs3(cL, 11, r);
      if (m0) atomicAdd(&ws->cellA[0][r], (double)m0 * (1.0 / MOMENT_UNIT));
      if (m1) atomicAdd(&ws->cellA[1][r], (double)m1 * (1.0 / MOMENT_UNIT));
      if (m2) atomicAdd(&ws->cellA[2][r], (double)m2 * (1.0 / MOMENT_UNIT));
    }
#pragma unroll
    for (int l = 0; l < (DP ? CELL_LIMBS_DP : CELL_LIMBS); ++l) cL[l][r] = 0;
  }
}

template <bool DP>
__global__ void __launch_bounds__(LTB) pool_cache_kernel(LloydArgs a, FmtDev F, LloydWs* __restrict__ ws, long long* __restrict__ pool_count_out,
                                                         unsigned spill_tiles) {
  __shared__ unsigned hist[SORT_ROWS + 3];
  __shared__ unsigned warp_tot[LTB / 32];
  extern __shared__ __align__(16) uint2 stage[];                  // TILE_ELEMS pairs (dynamic: the kernel needs 60 KB in all)
  // this CTA's share of the per-cell sums, as 32-bit limbs that native shared-memory atomics add:
  // [0..1] sum fix(omega), [2..4] sum fix(omega u), then either [5..7], [8..10], [11..13] the three moments in units
  // of 2^-40 or (DP) [5..7] sum fix(omega u u).  Low limbs hold 16 bits, the top limb the signed rest.
  constexpr int NL = DP ? CELL_LIMBS_DP : CELL_LIMBS;
  __shared__ unsigned cL[NL][SORT_ROWS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < NL * SORT_ROWS; i += LTB) (&cL[0][0])[i] = 0;
  unsigned tiles_since_spill = 0;
  const unsigned count = ws->list_count;
  const unsigned n_tiles = (count + LTB - 1) / LTB;
  const int k = ws->k;
  if (blockIdx.x == 0 && tid == 0) *pool_count_out = (long long)count;   // the list is complete: its length is the pool size
  for (unsigned tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    for (int i = tid; i < SORT_ROWS + 3; i += LTB) hist[i] = 0;
    __syncthreads();
    const unsigned i = tile * LTB + tid;
    float u[16], om[16];
    if (i < count) {
      unsigned j;
      pool_block_u(a, F, k, a.pool_idx[i], u, j);
      const float4* op = reinterpret_cast<const float4*>(a.omega + (size_t)j * SOP_G);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 o = __ldg(op + q);
        om[4 * q] = o.x; om[4 * q + 1] = o.y; om[4 * q + 2] = o.z; om[4 * q + 3] = o.w;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e) { u[e] = 0.0f; om[e] = 0.0f; }
    }
    unsigned where[16];   // cell << 16 | arrival number inside the cell
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const unsigned c = (unsigned)sort_cell(u[e]);
      where[e] = (c << 16) | atomicAdd(&hist[c], 1u);
    }
    __syncthreads();
    // exclusive scan of the 641 counts: three bins per thread
    {
      const int b0 = 3 * tid;
      unsigned c0 = 0, c1 = 0, c2 = 0;
      if (b0 < SORT_ROWS) { c0 = hist[b0]; c1 = hist[b0 + 1]; c2 = hist[b0 + 2]; }
      const unsigned local = c0 + c1 + c2;
      unsigned incl = local;
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      if (lane == 31) warp_tot[warp] = incl;
      __syncthreads();
      unsigned base = 0;
      for (int w = 0; w < warp; ++w) base += warp_tot[w];
      const unsigned excl = base + incl - local;
      if (b0 < SORT_ROWS) { hist[b0] = excl; hist[b0 + 1] = excl + c0; hist[b0 + 2] = excl + c0 + c1; }
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const unsigned p = hist[where[e] >> 16] + (where[e] & 0xFFFFu);
      stage[tile_slot(p)] = make_uint2(__float_as_uint(u[e]), __float_as_uint(om[e]));
    }
    __syncthreads();
    if (!DP) {      // the dynamic programme reads the per-cell sums only: no iteration walks the elements again
      uint4* dst = reinterpret_cast<uint4*>(a.cache + (size_t)tile * TILE_ELEMS);
      const uint4* src = reinterpret_cast<const uint4*>(stage);
#pragma unroll
      for (int q = 0; q < TILE_ELEMS / 2 / LTB; ++q) dst[q * LTB + tid] = src[q * LTB + tid];
      unsigned short* ts = a.tile_start + (size_t)tile * (SORT_ROWS + 1);
      for (int r = tid; r <= SORT_ROWS; r += LTB) ts[r] = (unsigned short)hist[r];      // hist[SORT_ROWS] = 4096: the end of the last cell
    }
    // per-cell sums: thread t owns the sorted positions 16 t .. 16 t + 15 (ascending cells), keeps the
    // current cell's sums in registers and adds them to the CTA's limbs when the cell changes
    {
      int cur = -1;
      unsigned long long n = 0, sv = 0, sq = 0;
      double a0 = 0.0, a1 = 0.0, a2 = 0.0;
#pragma unroll 4
      for (int i2 = 0; i2 < 16; ++i2) {
        const uint2 v = stage[tile_slot(16u * (unsigned)tid + (unsigned)i2)];
        const float u = __uint_as_float(v.x), om = __uint_as_float(v.y);
        const int c = sort_cell(u);
        if (c != cur) {
          if (cur >= 0) flush_cell<DP>(cL, cur, n, sv, sq, a0, a1, a2);
          cur = c; n = 0; sv = 0; sq = 0; a0 = a1 = a2 = 0.0;
        }
        const float ou = fminf(fmaxf(__fmul_rn(om, u), -256.0f), 256.0f);
        n += (unsigned long long)__float2uint_rn(__fmul_rn(om, 16777216.0f));   // omega in [0, 1]
        sv += (unsigned long long)fix24(ou);
        if (DP) {
          sq += (unsigned long long)fix24(__fmul_rn(ou, u));
        } else {
          const double dou = (double)om * (double)u;
          a0 += (double)om; a1 += dou; a2 += dou * (double)u;
        }
      }
      flush_cell<DP>(cL, cur, n, sv, sq, a0, a1, a2);
    }
    __syncthreads();
    // a cell takes at most 258 flushes per tile and a low limb 2^16 - 1 per flush: the limbs go to the
    // global sums before they can wrap
    if (++tiles_since_spill == spill_tiles) {
      spill_cells<DP>(cL, ws);
      tiles_since_spill = 0;
      __syncthreads();
    }
  }
  if (tiles_since_spill) spill_cells<DP>(cL, ws);
}

// One warp per tile.  The elements of the tile that lie in cells holding a threshold (sorted positions
// [start[c], start[c + 1]) for every such cell c) are dealt to the 32 lanes in contiguous shares, four
// loads in flight per lane: entry lo or hi by the exact threshold.  Sums go to the CTA's per-entry
// accumulators with shared-memory atomics (a few hundred elements per tile).
constexpr int MAX_SPLIT = 32;   // a table has at most 31 thresholds, so at most 31 cells hold one

// Between two folds a CTA walks at most 2^17 elements (8 warps, at most four tiles each), every element adds at most
// 2^24 to n and 2^32 in magnitude to sv, and there is at most one flush per element.  With 12-bit low
// limbs every limb sum stays below 2^31: n = 12 bits + the rest, sv = 12 + 12 bits + the signed rest.
__device__ __forceinline__ void flush_limbs(unsigned* n0, unsigned* n1, unsigned* s0, unsigned* s1, int* s2, int code,
                                            unsigned long long n, unsigned long long sv) {
  atomicAdd(&n0[code], (unsigned)(n & 0xFFFull));
  atomicAdd(&n1[code], (unsigned)(n >> 12));
  atomicAdd(&s0[code], (unsigned)(sv & 0xFFFull));
  atomicAdd(&s1[code], (unsigned)((sv >> 12) & 0xFFFull));
  atomicAdd(&s2[code], (int)((long long)sv >> 24));
}

// One iteration, by a whole CTA.  `counter` counts the CTAs that have added their sums; the CTA that arrives
// last updates the table and returns true.  FRESH: the descriptor was written during this launch by another
// CTA, so it is read past the L1.
template <bool FRESH>
__device__ __forceinline__ bool lloyd_iteration(const LloydArgs& a, LloydWs* __restrict__ ws, double* __restrict__ distortion,
                                                int it, int last, float* __restrict__ out_lut, unsigned* counter, bool reset_counter,
                                                unsigned fold_period) {
  __shared__ __align__(16) IterDesc d;
  __shared__ unsigned long long sN[SOP_MAX_ENTRIES], sS[SOP_MAX_ENTRIES];
  // flushes of the element walk: native 32-bit atomics on limbs, combined into sN / sS afterwards
  __shared__ unsigned lN[2][SOP_MAX_ENTRIES], lS0[SOP_MAX_ENTRIES], lS1[SOP_MAX_ENTRIES];
  __shared__ int lS2[SOP_MAX_ENTRIES];
  __shared__ double sD;
  __shared__ int s_is_last;
  __shared__ unsigned s_list_count;
  __shared__ CellEntry s_entry[MAX_SPLIT];
  __shared__ unsigned short s_cell[MAX_SPLIT];
  __shared__ unsigned short s_off[LTB / 32][MAX_SPLIT + 1];   // per warp: first item of every split cell in the tile
  __shared__ unsigned short s_p0[LTB / 32][MAX_SPLIT];
  __shared__ float s_new[SOP_MAX_ENTRIES];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  {
    constexpr int DW = (int)(sizeof(IterDesc) / sizeof(unsigned));
    static_assert(DW <= LTB, "one descriptor word per thread");
    if (tid < DW) {
      const unsigned* src = reinterpret_cast<const unsigned*>(&ws->desc) + tid;
      reinterpret_cast<unsigned*>(&d)[tid] = FRESH ? __ldcg(src) : *src;
    }
    if (tid == LTB - 1) s_list_count = ws->list_count;
    if (tid < 32) { sN[tid] = 0; sS[tid] = 0; lN[0][tid] = lN[1][tid] = lS0[tid] = lS1[tid] = 0; lS2[tid] = 0; }
    if (tid == 0) sD = 0.0;
  }
  __syncthreads();
  const int ne = d.n_entries;
  const unsigned n_tiles = (s_list_count + LTB - 1) / LTB;
  const float* lutv = d.lut;
  const float* tau = d.tau;
  // the cells that hold thresholds: thresholds ascend, so those of one cell are neighbours.  Every warp
  // derives the same list and writes the same values.
  int n_split;
  {
    const bool on = lane < ne - 1;
    const int c = d.thr_cell[lane];
    const int cp = __shfl_up_sync(0xFFFFFFFFu, c, 1), cn = __shfl_down_sync(0xFFFFFFFFu, c, 1);
    const bool first = on && (lane == 0 || cp != c);
    const bool single = lane == ne - 2 || cn != c;
    const unsigned fm = __ballot_sync(0xFFFFFFFFu, first);
    n_split = __popc(fm);
    if (first) {
      const int idx = __popc(fm & ((1u << lane) - 1u));
      CellEntry e;
      e.thr = tau[lane];
      e.codes = single ? ((unsigned)lane | ((unsigned)(lane + 1) << 8)) : 0xFFFFu;
      s_cell[idx] = (unsigned short)c;
      s_entry[idx] = e;
    }
    __syncwarp();
  }
  double D = 0.0;
  {
    // every cell without a threshold through its sums and moments, spread over the grid (a thread takes
    // one cell): its entry is the number of thresholds in lower cells, and
    // sum omega (u - q)^2 = A2 - 2 q A1 + q^2 A0 for the entry's value q
    for (int r = (int)blockIdx.x + (int)gridDim.x * (LTB - 1 - tid); r < SORT_ROWS; r += (int)gridDim.x * LTB) {
      const unsigned long long cn = ws->cellN[r];
      const long long cs = ws->cellS[r];
      const double a0 = ws->cellA[0][r], a1 = ws->cellA[1][r], a2 = ws->cellA[2][r];
      int j = 0;
      bool split = false;
      for (int k = 0; k < ne - 1; ++k) { const int c = d.thr_cell[k]; j += c < r ? 1 : 0; split |= c == r; }
      if (!split && (cn || a0 != 0.0)) {
        if (!last) { atomicAdd(&sN[j], cn); atomicAdd(&sS[j], (unsigned long long)cs); }
        const double q = (double)lutv[j];
        D += a2 - 2.0 * q * a1 + q * q * a0;
      }
    }
  }
  // Round k of the CTA covers tiles (k gridDim + blockIdx) 8 .. + 7, one per warp.  The limb accumulators hold what a
  // warp adds in at most four rounds (flush_limbs), so every fold_period <= 4 rounds the CTA folds them into its
  // 64-bit sums: a CTA may then walk any number of tiles, and a grid that is resident at once serves any pool.
  for (unsigned k = 0;; ++k) {
    const unsigned tile0 = (k * gridDim.x + blockIdx.x) * (LTB / 32);
    if (tile0 >= n_tiles) break;                       // the same for every warp of the CTA
    if (k != 0 && k % fold_period == 0) {
      __syncthreads();
      if (tid < 32 && !last) {
        sN[tid] += (unsigned long long)lN[0][tid] + ((unsigned long long)lN[1][tid] << 12);
        sS[tid] += (unsigned long long)lS0[tid] + ((unsigned long long)lS1[tid] << 12) + ((unsigned long long)(long long)lS2[tid] << 24);
        lN[0][tid] = lN[1][tid] = lS0[tid] = lS1[tid] = 0; lS2[tid] = 0;
      }
      __syncthreads();
    }
    const unsigned tile = tile0 + warp;
    if (tile >= n_tiles) continue;
    const unsigned short* ts = a.tile_start + (size_t)tile * (SORT_ROWS + 1);
    const uint2* src = a.cache + (size_t)tile * TILE_ELEMS;
    // segment lengths -> exclusive offsets (one cell per lane)
    unsigned len0 = 0, q0 = 0;
    if (lane < n_split) { const int c = s_cell[lane]; q0 = ts[c]; len0 = ts[c + 1] - q0; }
    unsigned inc0 = len0;
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v0 = __shfl_up_sync(0xFFFFFFFFu, inc0, o);
      if (lane >= o) inc0 += v0;
    }
    const unsigned total = __shfl_sync(0xFFFFFFFFu, inc0, 31);
    __syncwarp();
    s_off[warp][lane] = (unsigned short)(inc0 - len0); s_p0[warp][lane] = (unsigned short)q0;
    if (lane == 0) s_off[warp][MAX_SPLIT] = (unsigned short)total;
    __syncwarp();
    // every lane takes a contiguous share of the items: its entry changes a few times at most, so the
    // sums of the current entry stay in registers and reach the CTA's accumulators on a change
    const unsigned share = (total + 31u) / 32u;
    const unsigned i_lo = min(total, lane * share), i_hi = min(total, i_lo + share);
    int cur = -1;
    unsigned long long n = 0, sv = 0;
    for (unsigned base = i_lo; base < i_hi; base += 4) {
      uint2 v[4];
      int cell_l[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const unsigned item = base + k;
        cell_l[k] = -1;
        v[k] = make_uint2(0u, 0u);
        if (item < i_hi) {
          int l = 0;                       // the split cell whose item range holds `item`: binary search over <= 32 offsets
#pragma unroll
          for (int step = 16; step >= 1; step >>= 1) {     // branch-free: s_off has MAX_SPLIT + 1 entries
            const int t = l + step;
            const bool ok = (t < n_split) & (s_off[warp][min(t, MAX_SPLIT)] <= item);
            l = ok ? t : l;
          }
          cell_l[k] = l;
          const unsigned pp = s_p0[warp][l] + (item - s_off[warp][l]);
          v[k] = __ldg(src + tile_slot(pp));
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (cell_l[k] < 0) continue;
        const CellEntry e = s_entry[cell_l[k]];
        const float u = __uint_as_float(v[k].x), om = __uint_as_float(v[k].y);
        int code;
        if (e.codes == 0xFFFFu) code = count_below(tau, u);   // several thresholds in one cell: the general search
        else code = (int)((u > e.thr ? e.codes >> 8 : e.codes) & 0xFFu);
        const float dd = __fsub_rn(u, lutv[code]);
        D += (double)__fmul_rn(__fmul_rn(om, dd), dd);
        if (!last) {
          if (code != cur) {
            if (cur >= 0) flush_limbs(lN[0], lN[1], lS0, lS1, lS2, cur, n, sv);
            cur = code; n = 0; sv = 0;
          }
          const float ou = fminf(fmaxf(__fmul_rn(om, u), -256.0f), 256.0f);
          n += (unsigned long long)__float2uint_rn(__fmul_rn(om, 16777216.0f));   // omega in [0, 1]
          sv += (unsigned long long)fix24(ou);
        }
      }
    }
    if (cur >= 0) flush_limbs(lN[0], lN[1], lS0, lS1, lS2, cur, n, sv);
  }
  for (int o = 16; o; o >>= 1) D += __shfl_xor_sync(0xFFFFFFFFu, D, o);
  if (lane == 0 && D != 0.0) atomicAdd(&sD, D);
  __syncthreads();
  if (tid < ne && !last) {
    sN[tid] += (unsigned long long)lN[0][tid] + ((unsigned long long)lN[1][tid] << 12);
    sS[tid] += (unsigned long long)lS0[tid] + ((unsigned long long)lS1[tid] << 12) + ((unsigned long long)(long long)lS2[tid] << 24);
    if (sN[tid]) atomicAdd(&ws->accN[tid], sN[tid]);
    if (sS[tid]) atomicAdd(reinterpret_cast<unsigned long long*>(&ws->accS[tid]), sS[tid]);
  }
  if (tid == 0 && sD != 0.0) atomicAdd(&ws->accD, sD);
  // the CTA that arrives last owns the update; no CTA waits for another
  __threadfence();
  __syncthreads();
  if (tid == 0) s_is_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1 : 0;
  __syncthreads();
  const bool is_last = s_is_last != 0;
  if (is_last && tid < 32) {
    // one warp: every CTA has added its share (cells with a threshold element by element, the others by
    // their sums).  Centroids one lane per entry, a rank sort, and the next iteration's descriptor.
    __threadfence();
    const unsigned long long n = __ldcg(&ws->accN[tid]);
    const long long sv = __ldcg(&ws->accS[tid]);
    if (tid == 0) distortion[it] = __ldcg(&ws->accD);
    ws->accN[tid] = 0; ws->accS[tid] = 0;
    if (tid == 0) { ws->accD = 0.0; if (reset_counter) *counter = 0; }
    if (last) {
      out_lut[tid] = tid < ne ? lutv[tid] : 0.0f;
    } else {
      float t = lutv[tid];                       // lanes from n_entries on hold the last entry's value
      if (tid < ne && n) {
        const float cen = __double2float_rn(__ddiv_rn(__ll2double_rn(sv), __ull2double_rn(n)));
        uint32_t b = __float_as_uint(cen);
        b += 0x7FFFu + ((b >> 16) & 1u);
        b &= 0xFFFF0000u;                        // nearest bf16, ties to even
        t = __uint_as_float(b);
      }
      // ascending order: the rank of an entry is the number of entries before it (ties by index)
      int rank = 0;
      for (int k = 0; k < 32; ++k) {
        const float o = __shfl_sync(0xFFFFFFFFu, t, k);
        rank += (k < ne && (o < t || (o == t && k < tid))) ? 1 : 0;
      }
      if (tid < ne) s_new[rank] = t;
      __syncwarp();
      if (tid >= ne) s_new[tid] = 0.0f;
      __syncwarp();
      const float top = s_new[ne - 1];
      __syncwarp();
      if (tid >= ne) s_new[tid] = top;           // padded with the last entry
      __syncwarp();
      lloyd_publish_desc(ws, s_new, ne);
    }
  }
  return is_last;
}

// One launch per iteration (the stream orders the iterations).
__global__ void __launch_bounds__(LTB) lloyd_split_kernel(LloydArgs a, LloydWs* __restrict__ ws, double* __restrict__ distortion,
                                                          int it, int last, float* __restrict__ out_lut, unsigned fold_period) {
  lloyd_iteration<false>(a, ws, distortion, it, last, out_lut, &ws->done, true, fold_period);
}

// All iterations in one launch (launched cooperatively: every CTA is resident).  Between two iterations the
// CTAs wait for the flag that the CTA which arrived last sets after it has published the next table.  The
// wait is bounded: a CTA that gives up raises ws->error, every CTA then leaves, and the last distortion entry
// is set to -1 (a distortion is never negative) so that the caller can tell.
constexpr unsigned WAIT_POLLS = 1u << 22;     // times ~100 ns: about half a second

__global__ void __launch_bounds__(LTB) lloyd_persistent_kernel(LloydArgs a, LloydWs* __restrict__ ws, double* __restrict__ distortion,
                                                               int iters, float* __restrict__ out_lut, unsigned fold_period) {
  __shared__ int s_stop;
  for (int it = 0; it <= iters; ++it) {
    const int last = it == iters;
    const bool updater = lloyd_iteration<true>(a, ws, distortion, it, last, out_lut, &ws->arrive[it], false, fold_period);
    if (last) break;
    __syncthreads();                       // the updater's first warp has written the descriptor
    if (threadIdx.x == 0) {
      int stop = 0;
      if (updater) {
        __threadfence();
        atomicExch(&ws->ready[it], 1u);
      } else {
        unsigned polls = 0;
        while (*(volatile unsigned*)&ws->ready[it] == 0u) {
          if (*(volatile unsigned*)&ws->error != 0u || ++polls > WAIT_POLLS) { atomicExch(&ws->error, 1u); stop = 1; break; }
          __nanosleep(100);
        }
        __threadfence();
      }
      s_stop = stop;
    }
    __syncthreads();
    if (s_stop) break;
  }
  // Whoever leaves with the error flag up marks the result as invalid, whichever CTA gave up and whenever: a CTA
  // that arrived late can still run the remaining iterations alone (nobody else arrives, so it never closes
  // the last one), and it must not leave a valid-looking trace behind.
  if (threadIdx.x == 0 && *(volatile unsigned*)&ws->error != 0u) distortion[iters] = -1.0;
}

// ---------------------------------------------------------------------------------------------
// Grid-constrained DD-n (pair-search steps 1 and 3: cluster selection by dynamic programming on the grid points of the
// LUT value format).  The histogram is the per-cell sums that pool_cache_kernel has formed -- H = sum fix(omega),
// S = sum fix(omega u), Q = sum fix((omega u) u), integers, so independent of any order.  The cells with H > 0, in
// ascending order, are cut into min(n_entries, cells) runs; a run's code point is the bf16 value nearest to S / H
// (clamped to +-1.25) and it costs Q - 2 q S + q^2 H; the least total cost wins, a tie between cuts goes to the earliest.
// One launch per row of the programme (number of runs), one warp per last cell; the FP64 operations are written one by
// one (no contraction), so every comparison sees the same numbers as a sequential evaluation.
// ---------------------------------------------------------------------------------------------
constexpr int DP_TB = 256;

__device__ __forceinline__ double dp_run_cost(const long long* pH, const long long* pS, const long long* pQ, int i, int j, float* q_out) {
  const double h = __ll2double_rn(pH[j + 1] - pH[i]), sm = __ll2double_rn(pS[j + 1] - pS[i]), qq = __ll2double_rn(pQ[j + 1] - pQ[i]);
  const float mean = __double2float_rn(__ddiv_rn(sm, h));
  uint32_t b = __float_as_uint(mean);
  b += 0x7FFFu + ((b >> 16) & 1u);
  b &= 0xFFFF0000u;                                   // nearest bf16, ties to even
  float q = __uint_as_float(b);
  q = fminf(1.25f, fmaxf(-1.25f, q));
  if (q_out) *q_out = q;
  const double qd = (double)q;
  const double a = __dmul_rn(__dmul_rn(2.0, qd), sm);
  const double c = __dmul_rn(__dmul_rn(qd, qd), h);
  return __dadd_rn(__dsub_rn(qq, a), c);
}

// Scratch of the dynamic programme in the workspace: prefix sums of the non-empty cells, two rows of least costs.
struct DpScratch {
  int B;
  int pad;
  long long pH[SORT_ROWS + 1], pS[SORT_ROWS + 1], pQ[SORT_ROWS + 1];
  double best[2][SORT_ROWS];
};

// One CTA: the non-empty cells, their prefix sums, and row 0 (cells 0..j as one run).
__global__ void __launch_bounds__(DP_TB) grid_dp_first_kernel(const LloydWs* __restrict__ ws, DpScratch* __restrict__ dp) {
  __shared__ int s_B;
  if (threadIdx.x == 0) {
    int B = 0;
    dp->pH[0] = dp->pS[0] = dp->pQ[0] = 0;
    for (int t = 0; t < SORT_ROWS; ++t) {
      const long long h = (long long)ws->cellN[t];
      if (h > 0) { dp->pH[B + 1] = dp->pH[B] + h; dp->pS[B + 1] = dp->pS[B] + ws->cellS[t]; dp->pQ[B + 1] = dp->pQ[B] + ws->cellQ[t]; ++B; }
    }
    dp->B = B;
    s_B = B;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < s_B; j += DP_TB) dp->best[0][j] = dp_run_cost(dp->pH, dp->pS, dp->pQ, 0, j, nullptr);
}

// Row r of the programme: one warp per last cell j, the lanes share the starts i of the last run; the least value wins,
// a tie goes to the smallest i (what a sequential scan from the first start on keeps).
__global__ void __launch_bounds__(DP_TB) grid_dp_row_kernel(DpScratch* __restrict__ dp, int r, short* __restrict__ cut) {
  const int B = dp->B;
  const int lane = threadIdx.x & 31;
  const int j = blockIdx.x * (DP_TB / 32) + (threadIdx.x >> 5);
  if (j >= B || j < r) return;
  const double* prev = dp->best[(r - 1) & 1];
  double bv = 0.0;
  int bi = -1;
  for (int i = r + lane; i <= j; i += 32) {
    const double v = __dadd_rn(prev[i - 1], dp_run_cost(dp->pH, dp->pS, dp->pQ, i, j, nullptr));
    if (bi < 0 || v < bv) { bv = v; bi = i; }
  }
  for (int o = 16; o; o >>= 1) {
    const double ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
    const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, o);
    if (oi >= 0 && (bi < 0 || ov < bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
  }
  if (lane == 0) {
    dp->best[r & 1][j] = bv;
    cut[(size_t)r * SORT_ROWS + j] = (short)bi;
  }
}

// One thread: the backtrack, the code points in ascending order, the least total cost.  rows = rows the host launched
// (n_entries - 1 at most); with fewer cells than entries the programme stops at the last row that has a cell.
__global__ void grid_dp_last_kernel(const DpScratch* __restrict__ dp, int n_entries, const short* __restrict__ cut, float* __restrict__ out_lut,
                                    double* __restrict__ cost_out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int B = dp->B;
  if (B == 0) {
    for (int e = 0; e < SOP_MAX_ENTRIES; ++e) out_lut[e] = 0.0f;
    cost_out[0] = 0.0;
    return;
  }
  const int R = min(n_entries, B);
  float lut[SOP_MAX_ENTRIES];
  int j = B - 1, n = 0;
  for (int r = R - 1; r >= 0; --r) {
    const int i = r == 0 ? 0 : (int)cut[(size_t)r * SORT_ROWS + j];
    float q;
    dp_run_cost(dp->pH, dp->pS, dp->pQ, i, j, &q);
    lut[n++] = q;
    j = i - 1;
  }
  for (int a = 1; a < n; ++a) {                   // ascending: insertion sort of at most 32 values
    const float v = lut[a];
    int b = a - 1;
    while (b >= 0 && lut[b] > v) { lut[b + 1] = lut[b]; --b; }
    lut[b + 1] = v;
  }
  for (int e = 0; e < SOP_MAX_ENTRIES; ++e) out_lut[e] = e < n ? lut[e] : (e < n_entries ? lut[n - 1] : 0.0f);
  cost_out[0] = __ddiv_rn(dp->best[(R - 1) & 1][B - 1], 16777216.0);
}

int num_sms();

// Grid of the iteration kernels and whether all iterations run in one cooperative launch: they do wherever the device
// launches cooperatively (the CTAs wait for one another between iterations, so the whole grid has to be resident:
// the grid is cut to what is, and a CTA walks as many tiles as that takes); otherwise there is one launch per iteration.
static bool lloyd_iteration_plan(long long NB, long long pool_blocks, int iters, int flags, long long* grid_out) {
  const int sms = num_sms();
  const long long likely = (pool_blocks + LTB - 1) / LTB;           // cache tiles of the pool without ties at its threshold
  long long grid = (likely + LTB / 32 - 1) / (LTB / 32);            // one warp per cache tile
  if (grid > (long long)sms * 8) grid = (long long)sms * 8;
  if (g_tune.iter_ctas > 0 && grid > g_tune.iter_ctas) grid = g_tune.iter_ctas;
  if (grid < 1) grid = 1;
  (void)NB;
  DeviceFacts* facts = device_facts();
  if (facts->coop_blocks_per_sm < 0) {
    int dev = 0, coop = 0, nb = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, lloyd_persistent_kernel, LTB, 0) == cudaSuccess)
      facts->coop_blocks_per_sm = nb;
    else
      facts->coop_blocks_per_sm = 0;
    cudaGetLastError();
  }
  const long long resident = (long long)facts->coop_blocks_per_sm * sms;
  bool persistent = false;
  if (iters >= 1 && resident >= 1 && !(flags & SOP_LLOYD_LAUNCH_PER_ITERATION)) {
    persistent = true;
    if (grid > resident) grid = resident;
  }
  *grid_out = grid;
  return persistent;
}

}  // namespace sop

extern "C" {

int sop_dd4_lloyd_launches(long long M, long long K, int iters, int flags, int* launches) {
  if (!launches) return SOP_ERR_NULL;
  const int dp_entries = iters > 1 ? iters : 2;      // with SOP_LLOYD_GRID_DP the caller passes the number of table entries here
  if (M < 1 || K < 1 || (K % SOP_G) != 0 || iters < 0 || iters > sop::SOP_MAX_LLOYD_ITERS) return SOP_ERR_RANGE;
  long long grid = 1;
  const bool persistent = sop::lloyd_iteration_plan(M * (K / SOP_G), M * (K / SOP_G), iters, flags, &grid);
  // radix select (three passes, unless the pool is cut by a threshold), set-up, pool list, pool cache, iterations
  // the dynamic programme: first row, one launch per further row (callers with a 16-entry table: 15), the backtrack
  *launches = ((flags & SOP_LLOYD_POOL_THRESHOLD) ? 0 : 3) + 3 + ((flags & SOP_LLOYD_GRID_DP) ? 2 + (dp_entries - 1) : (persistent ? 1 : iters + 1));
  return SOP_OK;
}

int sop_dd4_lloyd_tuning(int cell_spill_tiles, int cache_ctas, int tiles_per_warp, int iter_ctas) {
  using namespace sop;
  if (cell_spill_tiles < 1 || cell_spill_tiles > CELL_SPILL_TILES_MAX || cache_ctas < 0 || tiles_per_warp < 1 ||
      tiles_per_warp > TILES_PER_WARP_MAX || iter_ctas < 0) return SOP_ERR_RANGE;
  g_tune.spill_tiles = cell_spill_tiles;
  g_tune.cache_ctas = cache_ctas;
  g_tune.tiles_per_warp = tiles_per_warp;
  g_tune.iter_ctas = iter_ctas;
  return SOP_OK;
}

int sop_dd4_lloyd_workspace(long long M, long long K, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (M < 1 || K < 1 || (K % SOP_G) != 0) return SOP_ERR_SHAPE;
  if (M > (1ll << 31) / (K / SOP_G)) return SOP_ERR_SHAPE;
  *bytes = sop::lloyd_ws_bytes(M, K);
  return SOP_OK;
}

int sop_dd4_lloyd(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                  const sop_scale_fmt* fmt, int k_mode, const sop_search_result* search_dev,
                  const float* block_metric_dev, long long pool_rank, float pool_threshold, int flags,
                  const sop_atom* atoms, int n_atoms,
                  int fmta_index, int iters, float* out_lut_dev, double* distortion_dev,
                  long long* pool_count_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
  using namespace sop;
  int rc = validate_layer(W_dev, M, K, ldw, c_dev, g);
  if (rc) return rc;
  if (!block_metric_dev || !out_lut_dev || !distortion_dev || !pool_count_dev) return SOP_ERR_NULL;
  if (flags & ~(SOP_LLOYD_POOL_BY_ERROR | SOP_LLOYD_UNIFORM_WEIGHTS | SOP_LLOYD_POOL_THRESHOLD | SOP_LLOYD_LAUNCH_PER_ITERATION | SOP_LLOYD_GRID_DP)) return SOP_ERR_RANGE;
  const bool grid_dp = (flags & SOP_LLOYD_GRID_DP) != 0;
  if (grid_dp && iters != 0) return SOP_ERR_RANGE;        // the dynamic programme replaces the iterations
  const bool by_threshold = (flags & SOP_LLOYD_POOL_THRESHOLD) != 0;
  if (by_threshold && !(pool_threshold == pool_threshold)) return SOP_ERR_RANGE;   // NaN orders nothing
  FmtDev F;
  if ((rc = validate_fmt(fmt, &F))) return rc;
  AtomsDev A;
  if ((rc = validate_atoms(atoms, n_atoms, 0u, nullptr, &A))) return rc;
  const long long NB = M * (K / SOP_G);
  if ((!by_threshold && (pool_rank < 1 || pool_rank > NB)) || iters < 0 || iters > 64) return SOP_ERR_RANGE;
  if (k_mode != SOP_K_FROM_RESULT && (k_mode < -64 || k_mode > 64)) return SOP_ERR_RANGE;
  if ((k_mode == SOP_K_FROM_RESULT || fmta_index == SOP_FMTA_FROM_RESULT) && !search_dev) return SOP_ERR_NULL;
  if (fmta_index != SOP_FMTA_FROM_RESULT && (fmta_index < 0 || fmta_index >= n_atoms)) return SOP_ERR_RANGE;
  if (fmta_index >= 0 && atoms[fmta_index].kind != SOP_KIND_LUT) return SOP_ERR_ALPHABET;
  if (NB * 16 > (1ll << 31)) return SOP_ERR_SHAPE;   // int64 fixed-point sums: at most 2^31 elements
  size_t need = 0;
  sop_dd4_lloyd_workspace(M, K, &need);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;

  // entries of the table the dynamic programme builds: FMTa's; when FMTa is chosen on the device every table atom must
  // agree on the number (decided here, before the first enqueue)
  int ne = 0;
  if (grid_dp) {
    ne = fmta_index >= 0 ? atoms[fmta_index].n_entries : 0;
    for (int i = 0; i < n_atoms && fmta_index < 0; ++i) {
      if (atoms[i].kind != SOP_KIND_LUT) continue;
      if (ne == 0) ne = atoms[i].n_entries;
      else if (atoms[i].n_entries != ne) return SOP_ERR_ALPHABET;
    }
    if (ne < 2) return SOP_ERR_ALPHABET;
  }

  unsigned char* wsb = (unsigned char*)workspace_dev;
  LloydArgs a;
  a.W = (const uint16_t*)W_dev; a.c = c_dev; a.cosrow_base = block_metric_dev;
  a.M = M; a.K = K; a.ldw = ldw; a.nbk = K / SOP_G; a.NB = NB; a.pool_rank = pool_rank;
  a.k_mode = k_mode; a.fmta_index = fmta_index; a.n_atoms = n_atoms;
  a.flags = flags; a.pool_threshold = pool_threshold;
  a.omega = (float*)(wsb + lloyd_off_omega());
  a.pool_idx = (unsigned*)(wsb + lloyd_off_idx(K));
  a.cache = (uint2*)(wsb + lloyd_off_cache(M, K));
  a.tile_start = (unsigned short*)(wsb + lloyd_off_tiles(M, K));
  LloydWs* ws = (LloydWs*)workspace_dev;
  cudaStream_t st = (cudaStream_t)stream;
  SOP_CUDA_TRY(cudaMemsetAsync(ws, 0, offsetof(LloydWs, dp_cut), st));
  if ((rc = profile_mark(SOP_PROFILE_POOL, 0, st))) return rc;
  const int sms = num_sms();
  long long sg = (NB + LTB * 8 - 1) / (LTB * 8);
  if (sg > sms * 4) sg = sms * 4;
  if (sg < 1) sg = 1;
  if (!by_threshold) {     // radix select of the pool_rank-th worst block (three passes over the ranking keys)
    select_kernel<0><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
    select_kernel<1><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
    select_kernel<2><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
    SOP_CUDA_TRY(cudaGetLastError());
  }
  lloyd_setup_kernel<<<1, SETUP_TB, 0, st>>>(a, A, search_dev, ws, distortion_dev, iters);
  SOP_CUDA_TRY(cudaGetLastError());
  pool_list_kernel<<<(int)sg, LTB, 0, st>>>(a, ws);
  SOP_CUDA_TRY(cudaGetLastError());

  // (u, omega) of every pool element, once: sorted tiles, cell starts, per-cell sums and moments
  {
    long long cg = (NB + LTB - 1) / LTB;      // one tile per CTA pass
    const long long cg_max = g_tune.cache_ctas > 0 ? g_tune.cache_ctas : (long long)sms * 3;
    if (cg > cg_max) cg = cg_max;
    const size_t stage_bytes = (size_t)TILE_ELEMS * sizeof(uint2);
    DeviceFacts* facts = device_facts();
    if (!facts->lloyd_attr_set) {
      SOP_CUDA_TRY(cudaFuncSetAttribute(pool_cache_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes));
      SOP_CUDA_TRY(cudaFuncSetAttribute(pool_cache_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stage_bytes));
      facts->lloyd_attr_set = true;
    }
    if (grid_dp) pool_cache_kernel<true><<<(int)cg, LTB, stage_bytes, st>>>(a, F, ws, pool_count_dev, (unsigned)g_tune.spill_tiles);
    else pool_cache_kernel<false><<<(int)cg, LTB, stage_bytes, st>>>(a, F, ws, pool_count_dev, (unsigned)g_tune.spill_tiles);
    SOP_CUDA_TRY(cudaGetLastError());
  }
  if ((rc = profile_mark(SOP_PROFILE_POOL, 1, st))) return rc;
  if (grid_dp) {
    if ((rc = profile_mark(SOP_PROFILE_LLOYD, 0, st))) return rc;
    static_assert(sizeof(DpScratch) <= sizeof(((LloydWs*)nullptr)->dp_scratch), "scratch of the dynamic programme");
    DpScratch* dp = reinterpret_cast<DpScratch*>(ws->dp_scratch);
    grid_dp_first_kernel<<<1, DP_TB, 0, st>>>(ws, dp);
    for (int r = 1; r < ne; ++r)      // a row without a cell (fewer cells than entries) returns at once
      grid_dp_row_kernel<<<(SORT_ROWS + DP_TB / 32 - 1) / (DP_TB / 32), DP_TB, 0, st>>>(dp, r, &ws->dp_cut[0][0]);
    grid_dp_last_kernel<<<1, 32, 0, st>>>(dp, ne, &ws->dp_cut[0][0], out_lut_dev, distortion_dev);
    SOP_CUDA_TRY(cudaGetLastError());
    if ((rc = profile_mark(SOP_PROFILE_LLOYD, 1, st))) return rc;
    return SOP_OK;
  }
  long long grid = 1;
  const bool persistent = lloyd_iteration_plan(NB, by_threshold ? NB : pool_rank, iters, flags, &grid);
  unsigned fold_period = (unsigned)g_tune.tiles_per_warp;
  if ((rc = profile_mark(SOP_PROFILE_LLOYD, 0, st))) return rc;
  if (persistent) {
    void* kargs[] = {(void*)&a, (void*)&ws, (void*)&distortion_dev, (void*)&iters, (void*)&out_lut_dev, (void*)&fold_period};
    SOP_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)lloyd_persistent_kernel, dim3((unsigned)grid), dim3(LTB), kargs, 0, st));
  } else {
    for (int it = 0; it <= iters; ++it) {
      const int last = it == iters;
      lloyd_split_kernel<<<(int)grid, LTB, 0, st>>>(a, ws, distortion_dev, it, last, out_lut_dev, fold_period);
    }
  }
  if ((rc = profile_mark(SOP_PROFILE_LLOYD, 1, st))) return rc;
  SOP_CUDA_TRY(cudaGetLastError());
  return SOP_OK;
}

}  // extern "C"
