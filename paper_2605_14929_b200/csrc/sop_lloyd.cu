// sop_dd4_lloyd: per-layer data-derived codebook (DD-n) by Lloyd iteration on the pool of blocks
// that the primary codebook reconstructs worst.
//
//   select_kernel<PASS>   three-pass radix select (11 + 11 + 10 bits) of the pool_rank-th smallest
//                         block cosine; each pass re-derives the prefix from the previous histogram.
//   lloyd_setup_kernel    threshold tau and pool count from the last histogram, max(c), the shift k,
//                         the initial table (FMTa, reversed and negated if FMTa is a negated atom).
//   lloyd_iter_kernel     one thread per pool block: u = w / scale, nearest entry by binary search
//                         over exact thresholds, per-entry int64 fixed-point sums (exactly
//                         associative, so atomics reproduce a sequential sum bit for bit), FP64 distortion.
//   lloyd_update_kernel   centroids -> bf16 -> sort; clears the accumulators.
#include <math.h>
#include <string.h>

#include "sop_device.cuh"

namespace sop {

constexpr int LTB = 256;

struct LloydWs {
  // radix select state
  unsigned hist[3][2048];
  // iteration state
  unsigned long long accN[SOP_MAX_ENTRIES];
  long long accS[SOP_MAX_ENTRIES];
  double accD;
  float lut[SOP_MAX_ENTRIES];
  float tau;         // pool threshold on the block cosine
  float cmax;
  int k;
  int fmta;
  int n_entries;
  int pad;
  long long pool_count;
};

struct LloydArgs {
  const uint16_t* W;
  const float* c;
  const float* cosrow_base;   // [n_atoms x NB] or [NB]
  long long M, K, ldw, nbk, NB;
  long long pool_rank;
  int k_mode, fmta_index, n_atoms;
};

__device__ __forceinline__ unsigned cos_key(float x) {
  const unsigned b = __float_as_uint(__fadd_rn(x, 0.0f));   // -0 -> +0
  return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}

__device__ __forceinline__ int resolve_fmta(const LloydArgs& a, const sop_search_result* res) {
  int f = a.fmta_index == SOP_FMTA_FROM_RESULT ? res->best_single : a.fmta_index;
  return max(0, min(a.n_atoms - 1, f));
}

// After pass p the selected element lies in bin sel[p] of hist[p]; rank is the rank inside that bin.
// Recomputed by every CTA from the histograms (a 2048-entry scan): cheaper than one more launch.
__device__ void derive_prefix(const LloydWs* ws, long long pool_rank, int passes, unsigned* prefix, long long* rank_out,
                              long long* below_out, unsigned* last_count) {
  __shared__ long long s_rank, s_below;
  __shared__ unsigned s_prefix, s_cnt;
  if (threadIdx.x == 0) {
    long long rank = pool_rank, below = 0;
    unsigned pre = 0, cnt = 0;
    for (int p = 0; p < passes; ++p) {
      const int nb = p < 2 ? 2048 : 1024;
      long long run = 0;
      int b = 0;
      for (; b < nb; ++b) {
        const unsigned h = ws->hist[p][b];
        if (run + h >= rank) { cnt = h; break; }
        run += h;
      }
      rank -= run;
      below += run;
      pre = (pre << (p < 2 ? 11 : 10)) | (unsigned)b;
    }
    s_rank = rank; s_below = below; s_prefix = pre; s_cnt = cnt;
  }
  __syncthreads();
  *prefix = s_prefix; *rank_out = s_rank; *below_out = s_below; *last_count = s_cnt;
}

template <int PASS>
__global__ void __launch_bounds__(LTB) select_kernel(LloydArgs a, const sop_search_result* __restrict__ res, LloydWs* __restrict__ ws) {
  __shared__ unsigned sh[2048];
  for (int i = threadIdx.x; i < 2048; i += LTB) sh[i] = 0;
  unsigned prefix = 0, cnt;
  long long rank, below;
  if (PASS > 0) derive_prefix(ws, a.pool_rank, PASS, &prefix, &rank, &below, &cnt);
  __syncthreads();
  const float* row = a.cosrow_base + (a.n_atoms > 0 ? (size_t)resolve_fmta(a, res) * a.NB : 0);
  for (long long i = (long long)blockIdx.x * LTB + threadIdx.x; i < a.NB; i += (long long)gridDim.x * LTB) {
    const unsigned key = cos_key(__ldg(row + i));
    if (PASS == 0) atomicAdd(&sh[key >> 21], 1u);
    else if (PASS == 1) { if ((key >> 21) == prefix) atomicAdd(&sh[(key >> 10) & 2047u], 1u); }
    else { if ((key >> 10) == prefix) atomicAdd(&sh[key & 1023u], 1u); }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 2048; i += LTB)
    if (sh[i]) atomicAdd(&ws->hist[PASS][i], sh[i]);
}

__global__ void __launch_bounds__(LTB) lloyd_setup_kernel(LloydArgs a, AtomsDev A, const sop_search_result* __restrict__ res,
                                                          LloydWs* __restrict__ ws, long long* __restrict__ pool_count_out) {
  unsigned prefix, cnt;
  long long rank, below;
  derive_prefix(ws, a.pool_rank, 3, &prefix, &rank, &below, &cnt);
  __shared__ float red[LTB];
  float mx = 0.0f;
  for (long long i = threadIdx.x; i < a.K; i += LTB) mx = fmaxf(mx, __ldg(a.c + i));
  red[threadIdx.x] = mx;
  __syncthreads();
  for (int s = LTB / 2; s; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + s]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const unsigned key = prefix;   // full 32-bit key after three passes
    const unsigned b = key ^ ((key >> 31) ? 0x80000000u : 0xFFFFFFFFu);
    ws->tau = __uint_as_float(b);
    ws->pool_count = below + cnt;
    *pool_count_out = below + cnt;
    ws->cmax = red[0];
    const int f = resolve_fmta(a, res);
    ws->fmta = f;
    ws->k = a.k_mode == SOP_K_FROM_RESULT ? res->k[f] : a.k_mode;
    const sop_atom& at = A.atoms[f];
    const int ne = at.n_entries;
    ws->n_entries = ne;
    const bool dd = (A.dd_mask >> f) & 1u;
    for (int j = 0; j < SOP_MAX_ENTRIES; ++j) {
      float v = 0.0f;
      if (j < ne) {
        const int src = at.negated ? ne - 1 - j : j;
        v = dd ? A.dd_lut[src] : at.lut[src];
        if (at.negated) v = -v;
      }
      ws->lut[j] = v;
    }
    for (int j = 0; j < SOP_MAX_ENTRIES; ++j) { ws->accN[j] = 0; ws->accS[j] = 0; }
    ws->accD = 0.0;
  }
}

__global__ void __launch_bounds__(LTB) lloyd_iter_kernel(LloydArgs a, FmtDev F, const sop_search_result* __restrict__ res,
                                                         LloydWs* __restrict__ ws, int accumulate_sums) {
  __shared__ float lutv[32], tau[32];
  __shared__ unsigned long long sN[LTB / 32][SOP_MAX_ENTRIES];
  __shared__ unsigned long long sS[LTB / 32][SOP_MAX_ENTRIES];
  __shared__ double sD[LTB / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ne = ws->n_entries;
  if (tid < 32) lutv[tid] = ws->lut[min(tid, ne - 1)];
  for (int i = tid; i < (LTB / 32) * SOP_MAX_ENTRIES; i += LTB) { (&sN[0][0])[i] = 0; (&sS[0][0])[i] = 0; }
  __syncthreads();
  if (tid == 0) build_thresholds(lutv, ne, tau);
  __syncthreads();
  const float cos_tau = ws->tau, cmax = ws->cmax;
  const int k = ws->k;
  const float* row = a.cosrow_base + (a.n_atoms > 0 ? (size_t)ws->fmta * a.NB : 0);

  const long long GT = (long long)gridDim.x * LTB;
  const long long R = GT / a.nbk;
  const long long gt = (long long)blockIdx.x * LTB + tid;
  const bool lane_on = gt < R * a.nbk;
  const long long j = lane_on ? gt % a.nbk : 0;
  const long long r0 = gt / a.nbk;
  float om[16];
  long long fixw[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float cv = __ldg(a.c + j * SOP_G + i);
    om[i] = cmax > 0.0f ? __fdiv_rn(cv, cmax) : 0.0f;
    fixw[i] = __float2ll_rn(__fmul_rn(om[i], 16777216.0f));
  }
  double D = 0.0;
  if (lane_on) {
    for (long long m = r0; m < a.M; m += R) {
      const long long blk = m * a.nbk + j;
      if (!(__ldg(row + blk) <= cos_tau)) continue;
      const uint4* p = reinterpret_cast<const uint4*>(a.W + m * a.ldw + j * SOP_G);
      const uint4 v0 = __ldg(p), v1 = __ldg(p + 1);
      const uint32_t wb[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      uint32_t mb = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) { mb = max(mb, wb[q] & 0x7FFFu); mb = max(mb, (wb[q] >> 16) & 0x7FFFu); }
      const float amax = __uint_as_float(mb << 16);
      const float s_hat = scale_quantize(amax, k, F).s_hat;    // a DD table declares tmax = 1
      const float rcp = s_hat > 0.0f ? __frcp_rn(s_hat) : 0.0f;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const float w = (i & 1) ? bf16hi(wb[i >> 1]) : bf16lo(wb[i >> 1]);
        const float u = __fmul_rn(w, rcp);
        const int code = count_below(tau, u);
        const double d = (double)u - (double)lutv[code];
        D += ((double)om[i] * d) * d;
        if (accumulate_sums) {
          const float ou = fminf(fmaxf(__fmul_rn(om[i], u), -256.0f), 256.0f);
          atomicAdd(&sN[warp][code], (unsigned long long)fixw[i]);
          atomicAdd(&sS[warp][code], (unsigned long long)__float2ll_rn(__fmul_rn(ou, 16777216.0f)));
        }
      }
    }
  }
  for (int o = 16; o; o >>= 1) D += __shfl_xor_sync(0xFFFFFFFFu, D, o);
  if (lane == 0) sD[warp] = D;
  __syncthreads();
  if (tid < ne && accumulate_sums) {
    unsigned long long n = 0, s = 0;
    for (int w = 0; w < LTB / 32; ++w) { n += sN[w][tid]; s += sS[w][tid]; }
    if (n) atomicAdd(&ws->accN[tid], n);
    if (s) atomicAdd(reinterpret_cast<unsigned long long*>(&ws->accS[tid]), s);
  }
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < LTB / 32; ++w) t += sD[w];
    if (t != 0.0) atomicAdd(&ws->accD, t);
  }
}

__global__ void lloyd_update_kernel(LloydWs* __restrict__ ws, double* __restrict__ distortion, int it, int last,
                                    float* __restrict__ out_lut) {
  if (threadIdx.x != 0) return;
  distortion[it] = ws->accD;
  const int ne = ws->n_entries;
  if (!last) {
    float v[SOP_MAX_ENTRIES];
    for (int j = 0; j < ne; ++j) {
      v[j] = ws->lut[j];
      const unsigned long long n = ws->accN[j];
      if (n) {
        const float cen = __double2float_rn(__ddiv_rn(__ll2double_rn(ws->accS[j]), __ull2double_rn(n)));
        uint32_t b = __float_as_uint(cen);
        b += 0x7FFFu + ((b >> 16) & 1u);
        b &= 0xFFFF0000u;                      // nearest bf16, ties to even
        v[j] = __uint_as_float(b);
      }
    }
    for (int i = 1; i < ne; ++i) {             // insertion sort, ascending
      const float x = v[i];
      int p = i - 1;
      while (p >= 0 && v[p] > x) { v[p + 1] = v[p]; --p; }
      v[p + 1] = x;
    }
    for (int j = 0; j < ne; ++j) ws->lut[j] = v[j];
  } else {
    for (int j = 0; j < SOP_MAX_ENTRIES; ++j) out_lut[j] = j < ne ? ws->lut[j] : 0.0f;
  }
  for (int j = 0; j < SOP_MAX_ENTRIES; ++j) { ws->accN[j] = 0; ws->accS[j] = 0; }
  ws->accD = 0.0;
}

int num_sms();

}  // namespace sop

extern "C" {

int sop_dd4_lloyd_workspace(long long M, long long K, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (M < 1 || K < 1 || (K % SOP_G) != 0) return SOP_ERR_SHAPE;
  *bytes = (sizeof(sop::LloydWs) + 255) & ~(size_t)255;
  return SOP_OK;
}

int sop_dd4_lloyd(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                  const sop_scale_fmt* fmt, int k_mode, const sop_search_result* search_dev,
                  const float* block_cos_dev, long long pool_rank, const sop_atom* atoms, int n_atoms,
                  int fmta_index, int iters, float* out_lut_dev, double* distortion_dev,
                  long long* pool_count_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
  using namespace sop;
  int rc = validate_layer(W_dev, M, K, ldw, c_dev, g);
  if (rc) return rc;
  if (!block_cos_dev || !out_lut_dev || !distortion_dev || !pool_count_dev) return SOP_ERR_NULL;
  FmtDev F;
  if ((rc = validate_fmt(fmt, &F))) return rc;
  AtomsDev A;
  if ((rc = validate_atoms(atoms, n_atoms, 0u, nullptr, &A))) return rc;
  const long long NB = M * (K / SOP_G);
  if (pool_rank < 1 || pool_rank > NB || iters < 0 || iters > 64) return SOP_ERR_RANGE;
  if (k_mode != SOP_K_FROM_RESULT && (k_mode < -64 || k_mode > 64)) return SOP_ERR_RANGE;
  if ((k_mode == SOP_K_FROM_RESULT || fmta_index == SOP_FMTA_FROM_RESULT) && !search_dev) return SOP_ERR_NULL;
  if (fmta_index != SOP_FMTA_FROM_RESULT && (fmta_index < 0 || fmta_index >= n_atoms)) return SOP_ERR_RANGE;
  if (fmta_index >= 0 && atoms[fmta_index].kind != SOP_KIND_LUT) return SOP_ERR_ALPHABET;
  if (NB * 16 > (1ll << 31)) return SOP_ERR_SHAPE;   // int64 fixed-point sums: at most 2^31 elements
  size_t need = 0;
  sop_dd4_lloyd_workspace(M, K, &need);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;

  LloydArgs a;
  a.W = (const uint16_t*)W_dev; a.c = c_dev; a.cosrow_base = block_cos_dev;
  a.M = M; a.K = K; a.ldw = ldw; a.nbk = K / SOP_G; a.NB = NB; a.pool_rank = pool_rank;
  a.k_mode = k_mode; a.fmta_index = fmta_index; a.n_atoms = n_atoms;
  LloydWs* ws = (LloydWs*)workspace_dev;
  cudaStream_t st = (cudaStream_t)stream;
  SOP_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(LloydWs), st));
  const int sms = num_sms();
  long long sg = (NB + LTB * 8 - 1) / (LTB * 8);
  if (sg > sms * 4) sg = sms * 4;
  if (sg < 1) sg = 1;
  select_kernel<0><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
  select_kernel<1><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
  select_kernel<2><<<(int)sg, LTB, 0, st>>>(a, search_dev, ws);
  SOP_CUDA_TRY(cudaGetLastError());
  lloyd_setup_kernel<<<1, LTB, 0, st>>>(a, A, search_dev, ws, pool_count_dev);
  SOP_CUDA_TRY(cudaGetLastError());
  long long grid = (NB + LTB - 1) / LTB;
  if (grid > (long long)sms * 4) grid = (long long)sms * 4;
  const long long min_grid = (a.nbk + LTB - 1) / LTB;
  if (grid < min_grid) grid = min_grid;
  for (int it = 0; it <= iters; ++it) {
    const int last = it == iters;
    lloyd_iter_kernel<<<(int)grid, LTB, 0, st>>>(a, F, search_dev, ws, last ? 0 : 1);
    lloyd_update_kernel<<<1, 32, 0, st>>>(ws, distortion_dev, it, last, out_lut_dev);
  }
  SOP_CUDA_TRY(cudaGetLastError());
  return SOP_OK;
}

}  // extern "C"
