// Host-side argument validation, error text and the channel-norm kernels of libsop.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "sop_device.cuh"

namespace sop {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e), where);
}

constexpr int PROFILE_RING = 8;            // the last eight calls of every kind stay readable
static bool g_profile = false;
static cudaEvent_t g_ev[SOP_PROFILE_KINDS][PROFILE_RING][2];
static bool g_ev_made = false;
static long long g_ev_count[SOP_PROFILE_KINDS];

constexpr int FACTS_DEVICES = 64;
static DeviceFacts g_facts[FACTS_DEVICES + 1];
static bool g_facts_init = false;

DeviceFacts* device_facts() {
  if (!g_facts_init) {
    for (int i = 0; i <= FACTS_DEVICES; ++i) { g_facts[i].sms = 0; g_facts[i].coop_blocks_per_sm = -1; g_facts[i].search_attr_set = g_facts[i].lloyd_attr_set = false; }
    g_facts_init = true;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= FACTS_DEVICES) {
    cudaGetLastError();
    DeviceFacts* f = &g_facts[FACTS_DEVICES];      // beyond the table: nothing is remembered
    f->sms = 0; f->coop_blocks_per_sm = -1; f->search_attr_set = f->lloyd_attr_set = false;
    return f;
  }
  return &g_facts[dev];
}

int num_sms() {
  DeviceFacts* f = device_facts();
  if (!f->sms) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    f->sms = n;
  }
  return f->sms;
}

int profile_mark(int which, int edge, cudaStream_t st) {
  if (!g_profile) return SOP_OK;
  if (!g_ev_made) {
    for (int i = 0; i < SOP_PROFILE_KINDS; ++i)
      for (int r = 0; r < PROFILE_RING; ++r)
        for (int e = 0; e < 2; ++e) SOP_CUDA_TRY(cudaEventCreate(&g_ev[i][r][e]));
    g_ev_made = true;
  }
  SOP_CUDA_TRY(cudaEventRecord(g_ev[which][g_ev_count[which] % PROFILE_RING][edge], st));
  if (edge == 1) ++g_ev_count[which];
  return SOP_OK;
}

int validate_fmt(const sop_scale_fmt* f, FmtDev* out) {
  if (!f) return SOP_ERR_NULL;
  if (f->exp_bits < 1 || f->exp_bits > 8 || f->man_bits < 0 || f->man_bits > 10) return SOP_ERR_FORMAT;
  if (f->sign_bits < 0 || f->sign_bits > 1 || f->top_exp_reserved < 0 || f->top_exp_reserved > 1) return SOP_ERR_FORMAT;
  if (f->bias < 0 || f->bias > 127) return SOP_ERR_FORMAT;
  const int top = (1 << f->exp_bits) - 1 - f->top_exp_reserved;
  if (top < 1) return SOP_ERR_FORMAT;
  out->y = f->man_bits;
  out->bias = f->bias;
  out->emin = 1 - f->bias;
  out->emax = top - f->bias;
  if (out->emax > 127) return SOP_ERR_FORMAT;  // largest scale must stay finite in fp32
  out->code_max = (top << f->man_bits) | ((1 << f->man_bits) - 1);
  out->sign_bits = f->sign_bits;
  return SOP_OK;
}

int validate_atoms(const sop_atom* atoms, int n_atoms, unsigned dd_mask, const float* dd_lut, AtomsDev* out) {
  if (!atoms) return SOP_ERR_NULL;
  if (n_atoms < 1 || n_atoms > SOP_MAX_ATOMS) return SOP_ERR_ALPHABET;
  if (dd_mask && !dd_lut) return SOP_ERR_NULL;
  if (n_atoms < 32 && (dd_mask >> n_atoms)) return SOP_ERR_ALPHABET;
  memset(out, 0, sizeof(*out));
  out->n_atoms = n_atoms;
  out->dd_mask = dd_mask;
  out->dd_lut = dd_lut;
  for (int i = 0; i < n_atoms; ++i) {
    const sop_atom& a = atoms[i];
    if (!(a.tmax > 0.0f) || !isfinite(a.tmax)) return SOP_ERR_ALPHABET;
    if (a.scope != 0 && a.scope != SOP_G) return SOP_ERR_ALPHABET;
    if (a.negated != 0 && a.negated != 1) return SOP_ERR_ALPHABET;
    if (a.kind == SOP_KIND_LUT) {
      if (a.scope != SOP_G) return SOP_ERR_ALPHABET;
      if (a.n_bits < 1 || a.n_bits > 5) return SOP_ERR_ALPHABET;
      if (a.n_entries < 2 || a.n_entries > (1 << a.n_bits)) return SOP_ERR_ALPHABET;
      if (!((dd_mask >> i) & 1u)) {
        for (int j = 0; j < a.n_entries; ++j) {
          if (!isfinite(a.lut[j])) return SOP_ERR_ALPHABET;
          if (j && a.lut[j] < a.lut[j - 1]) return SOP_ERR_ALPHABET;
        }
      }
    } else if (a.kind == SOP_KIND_FP_E2M3) {
      if (a.n_bits != 6 || a.negated) return SOP_ERR_ALPHABET;
    } else if (a.kind == SOP_KIND_FP_E4M3) {
      if (a.n_bits != 8 || a.negated) return SOP_ERR_ALPHABET;
    } else if (a.kind == SOP_KIND_FP_GRID) {
      if (a.negated || a.n_bits < 2 || a.n_bits > 16) return SOP_ERR_ALPHABET;
      if (a.grid_exp_bits < 0 || a.grid_exp_bits > 8 || a.grid_man_bits < 0 || a.grid_man_bits > 10) return SOP_ERR_ALPHABET;
      if (a.grid_bias < -100 || a.grid_bias > 100) return SOP_ERR_ALPHABET;
      if (a.grid_exp_bits && 1 + a.grid_exp_bits + a.grid_man_bits > a.n_bits) return SOP_ERR_ALPHABET;
      if (!isfinite(a.grid_neg_max) || a.grid_neg_max < a.tmax) return SOP_ERR_ALPHABET;
      // both ends must be values of the grid: a whole number of steps of their binade (or of the subnormal step)
      const float ends[2] = {a.tmax, a.grid_neg_max};
      for (int e = 0; e < 2; ++e) {
        int ex = 0;
        frexp((double)ends[e], &ex);                       // ends[e] = f * 2^ex, f in [1/2, 1)
        const int binade = ex - 1 > 1 - a.grid_bias ? ex - 1 : 1 - a.grid_bias;
        const double steps = ldexp((double)ends[e], a.grid_man_bits - binade);
        if (steps != floor(steps)) return SOP_ERR_ALPHABET;
      }
    } else {
      return SOP_ERR_ALPHABET;
    }
    if (((dd_mask >> i) & 1u) && a.kind != SOP_KIND_LUT) return SOP_ERR_ALPHABET;
    out->atoms[i] = a;
  }
  return SOP_OK;
}

int validate_layer(const void* W, long long M, long long K, long long ldw, const float* c, int g) {
  if (!W || !c) return SOP_ERR_NULL;
  if (g != SOP_G) return SOP_ERR_SHAPE;
  if (M < 1 || K < 1 || (K % SOP_G) != 0 || ldw < K || (ldw % 8) != 0) return SOP_ERR_SHAPE;
  if (((uintptr_t)W & 15u) != 0) return SOP_ERR_SHAPE;
  if (M > (1ll << 31) / (K / SOP_G)) return SOP_ERR_SHAPE;  // block count must fit 31 bits
  return SOP_OK;
}

// ---------------------------------------------------------------------------------------------
// Channel norms.  Two kernels: per-(chunk, column) FP64 partial sums over 64 rows in row order,
// then per column the partials added in chunk order, divided by T, square-rooted, rounded to fp32.
// HBM-bound: X is read exactly once with fully coalesced 128-byte rows per warp.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) norms_partial_kernel(const float* __restrict__ X, long long T, long long K,
                                                            long long ldx, double* __restrict__ part) {
  const long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long chunk = blockIdx.y;
  if (k >= K) return;
  const long long t0 = chunk * 64, t1 = min(T, t0 + 64);
  const float* p = X + t0 * ldx + k;
  double acc = 0.0;
  long long t = t0;
  for (; t + 8 <= t1; t += 8) {
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + (long long)i * ldx);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc = __fma_rn((double)v[i], (double)v[i], acc);
    p += 8 * ldx;
  }
  for (; t < t1; ++t) {
    const double x = (double)__ldg(p);
    acc = __fma_rn(x, x, acc);
    p += ldx;
  }
  part[chunk * K + k] = acc;
}

__global__ void __launch_bounds__(256) norms_final_kernel(const double* __restrict__ part, long long n_chunks, long long K,
                                                          long long T, float* __restrict__ c) {
  const long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  double total = 0.0;
  for (long long ch = 0; ch < n_chunks; ++ch) total = __dadd_rn(total, part[ch * K + k]);
  c[k] = __double2float_rn(__dsqrt_rn(__ddiv_rn(total, (double)T)));
}

}  // namespace sop

extern "C" {

const char* sop_strerror(int code) {
  switch (code) {
    case SOP_OK: return "ok";
    case SOP_ERR_NULL: return "a required pointer is NULL";
    case SOP_ERR_SHAPE: return "bad shape: need M, K, T >= 1, K % 16 == 0, ld >= K (ldw % 8 == 0, W 16-byte aligned), g == 16";
    case SOP_ERR_FORMAT: return "bad scale format or scale-word container";
    case SOP_ERR_ALPHABET: return "bad alphabet: atom count, kind, n_bits, n_entries, tmax or unsorted table";
    case SOP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SOP_ERR_CUDA: return "CUDA runtime error (see sop_last_cuda_error)";
    case SOP_ERR_RANGE: return "argument out of range (k shift, pool_rank, iters or index)";
    case SOP_ERR_TOO_LARGE: return "problem larger than the built-in scratch of the no-allocation entry point";
    default: return "unknown error code";
  }
}

const char* sop_last_cuda_error(void) { return sop::g_cuda_error; }

int sop_version(void) { return 102; }

int sop_profile_enable(int on) {
  sop::g_profile = on != 0;
  for (int i = 0; i < SOP_PROFILE_KINDS; ++i) sop::g_ev_count[i] = 0;
  return SOP_OK;
}

int sop_profile_ms(int which, int back, float* ms) {
  if (!ms) return SOP_ERR_NULL;
  if (which < 0 || which >= SOP_PROFILE_KINDS || back < 0 || back >= sop::PROFILE_RING || back >= sop::g_ev_count[which]) return SOP_ERR_RANGE;
  cudaEvent_t* ev = sop::g_ev[which][(sop::g_ev_count[which] - 1 - back) % sop::PROFILE_RING];
  SOP_CUDA_TRY(cudaEventSynchronize(ev[1]));
  SOP_CUDA_TRY(cudaEventElapsedTime(ms, ev[0], ev[1]));
  return SOP_OK;
}

int sop_profile_last_ms(int which, float* ms) { return sop_profile_ms(which, 0, ms); }
int sop_profile_last_sweep_ms(float* ms) { return sop_profile_ms(SOP_PROFILE_SWEEP, 0, ms); }

int sop_channel_norms_workspace(long long T, long long K, size_t* bytes) {
  if (!bytes) return SOP_ERR_NULL;
  if (T < 1 || K < 1) return SOP_ERR_SHAPE;
  *bytes = (size_t)((T + 63) / 64) * (size_t)K * sizeof(double);
  return SOP_OK;
}

int sop_channel_norms(const float* X_dev, long long T, long long K, long long ldx, float* c_dev,
                      void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!X_dev || !c_dev) return SOP_ERR_NULL;
  if (T < 1 || K < 1 || ldx < K) return SOP_ERR_SHAPE;
  size_t need = 0;
  sop_channel_norms_workspace(T, K, &need);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255u) || workspace_bytes < need) return SOP_ERR_WORKSPACE;
  const long long n_chunks = (T + 63) / 64;
  if (n_chunks > 65535) return SOP_ERR_SHAPE;
  cudaStream_t st = (cudaStream_t)stream;
  dim3 grid((unsigned)((K + 255) / 256), (unsigned)n_chunks);
  int rc;
  if ((rc = sop::profile_mark(SOP_PROFILE_NORMS, 0, st))) return rc;
  sop::norms_partial_kernel<<<grid, 256, 0, st>>>(X_dev, T, K, ldx, (double*)workspace_dev);
  SOP_CUDA_TRY(cudaGetLastError());
  sop::norms_final_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>((const double*)workspace_dev, n_chunks, K, T, c_dev);
  SOP_CUDA_TRY(cudaGetLastError());
  if ((rc = sop::profile_mark(SOP_PROFILE_NORMS, 1, st))) return rc;
  return SOP_OK;
}

// ---------------------------------------------------------------------------------------------
// Channel norms without a caller workspace.  The chunk partials live in a fixed array inside the
// library image: SOP_NORMS_STATIC_DOUBLES doubles (4 MiB) on every GPU that loads the library, held
// until the process exits.  Host code cannot use the array's name as a pointer (on the host it is
// only a handle for the symbol), so its device address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that address is what the kernels get.
// ---------------------------------------------------------------------------------------------
namespace sop {
static __device__ __align__(256) double g_norms_scratch[SOP_NORMS_STATIC_DOUBLES];

constexpr int MAX_DEVICES = 64;
static double* g_norms_scratch_addr[MAX_DEVICES];   // device address of g_norms_scratch, per device ordinal
static bool g_norms_scratch_known[MAX_DEVICES];

// Address of the scratch array on the current device (looked up on the first call per device).
static int norms_scratch_address(double** out) {
  int dev = -1;
  SOP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return SOP_ERR_RANGE;
  if (!g_norms_scratch_known[dev]) {
    void* p = nullptr;
    SOP_CUDA_TRY(cudaGetSymbolAddress(&p, g_norms_scratch));
    g_norms_scratch_addr[dev] = static_cast<double*>(p);
    g_norms_scratch_known[dev] = true;
  }
  *out = g_norms_scratch_addr[dev];
  return SOP_OK;
}
}  // namespace sop

int sop_channel_norms_static(const float* X_dev, long long T, long long K, long long ldx, float* c_dev, void* stream) {
  if (!X_dev || !c_dev) return SOP_ERR_NULL;
  if (T < 1 || K < 1 || ldx < K) return SOP_ERR_SHAPE;
  const long long n_chunks = (T + 63) / 64;
  if (n_chunks > 65535) return SOP_ERR_SHAPE;
  if (n_chunks > SOP_NORMS_STATIC_DOUBLES / K) return SOP_ERR_TOO_LARGE;   // n_chunks * K doubles must fit the array
  double* scratch = nullptr;
  int rc = sop::norms_scratch_address(&scratch);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // every partial that the second kernel reads is written by the first one in this call: nothing has
  // to be cleared, whatever an earlier call left in the array
  dim3 grid((unsigned)((K + 255) / 256), (unsigned)n_chunks);
  sop::norms_partial_kernel<<<grid, 256, 0, st>>>(X_dev, T, K, ldx, scratch);
  SOP_CUDA_TRY(cudaGetLastError());
  sop::norms_final_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>(scratch, n_chunks, K, T, c_dev);
  SOP_CUDA_TRY(cudaGetLastError());
  return SOP_OK;
}

}  // extern "C"
