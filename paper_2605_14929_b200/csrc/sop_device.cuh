// Device-side building blocks of libsop (sm_100a).  Everything here is compiled with -fmad=false:
// a fused multiply-add happens only where __fmaf_rn / __ffma2_rn is written, so every fp32 result
// is one IEEE-754 operation rounded to nearest even and reproducible bit for bit.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sop.h"

#define SOP_MAX_TABLES 8      // distinct LUT contents per call
#define SOP_MAX_CLASSES 8     // distinct (scope, tmax, quantiser) groups per call
#define SOP_HIST_BINS 320     // exponent histogram: ilogb(sigma) + 160, ilogb in [-149, 128]
#define SOP_HIST_OFF 160

namespace sop {

// ---- host-side error plumbing --------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char* where);
#define SOP_CUDA_TRY(expr)                                 \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) {                              \
      ::sop::set_cuda_error(e__, #expr);                   \
      return SOP_ERR_CUDA;                                 \
    }                                                      \
  } while (0)

// What the library remembers about a device, per device ordinal (a process may drive several devices; a call works
// on the device that is current when it is made).  device_facts() returns the entry of the current device, or a
// scratch entry that is never marked as known when the ordinal is beyond the table.
struct DeviceFacts {
  int sms;                    // 0: not asked yet
  int coop_blocks_per_sm;     // resident CTAs of the persistent Lloyd kernel per SM; -1: not asked yet, 0: no cooperative launch
  bool search_attr_set;       // the dynamic shared-memory limits of the search kernels have been raised on this device
  bool lloyd_attr_set;        // the same for the pool cache kernels
};
DeviceFacts* device_facts();
int num_sms();

// Optional timing of one kernel family of a call (CUDA events on the launching stream): edge 0 before
// the first launch, edge 1 after the last.  No-op unless profiling is enabled.
int profile_mark(int which, int edge, cudaStream_t st);

// ---- kernel parameter blocks ---------------------------------------------------------------
struct FmtDev {
  int y;                // mantissa bits
  int bias;
  int emin, emax;       // unbiased exponent range of normal values
  int code_max;         // largest finite magnitude code (E << y | M)
  int sign_bits;
};

struct AtomsDev {
  int n_atoms;
  unsigned dd_mask;         // atoms whose table comes from dd_lut at kernel time
  const float* dd_lut;      // device, SOP_MAX_ENTRIES floats (may be null)
  sop_atom atoms[SOP_MAX_ATOMS];
};

int validate_fmt(const sop_scale_fmt* f, FmtDev* out);
int validate_atoms(const sop_atom* atoms, int n_atoms, unsigned dd_mask, const float* dd_lut, AtomsDev* out);
int validate_layer(const void* W, long long M, long long K, long long ldw, const float* c, int g);

// ---- small device helpers ------------------------------------------------------------------
__device__ __forceinline__ float pow2f_int(int e) {  // 2^e for e in [-126, 127]
  return __uint_as_float((uint32_t)(e + 127) << 23);
}

__device__ __forceinline__ int ilogb_pos(float v) {  // floor(log2 v) for finite v > 0, subnormals included
  const uint32_t b = __float_as_uint(v);
  const int e = (int)(b >> 23);
  if (e != 0) return e - 127;
  return (31 - __clz((int)(b & 0x7FFFFFu))) - 149;
}

__device__ __forceinline__ float bf16lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16hi(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

// value = mant * 2^ex rounded once (only when the result is below the fp32 normal range)
__device__ __forceinline__ float ldexp_once(uint32_t mant, int ex) {
  const int e1 = max(-100, min(100, ex));
  const int e2 = max(-120, min(120, ex - e1));
  return __fmul_rn(__fmul_rn((float)mant, pow2f_int(e1)), pow2f_int(e2));
}

struct QScale { float s_hat; uint32_t code; };  // code = (E << y) | M

// Scale quantisation: sigma * 2^k rounded to nearest even on a y-bit mantissa with gradual
// underflow at E = 0, saturating at code_max, never rounding a positive value to zero; decoded and
// multiplied back by 2^-k.  Pure integer work on the fp32 bit pattern.
__device__ __forceinline__ QScale scale_quantize(float sigma, int k, const FmtDev& f) {
  QScale r;
  r.s_hat = 0.0f;
  r.code = 0;
  if (!(sigma > 0.0f)) return r;
  const uint32_t b = __float_as_uint(sigma);
  int e = (int)(b >> 23);
  {
    // The usual case: the shifted value lies in the format's normal range below its top binade (so that a
    // carry out of the mantissa cannot pass the largest code) and the format keeps at least one mantissa
    // bit.  Rounding to nearest even on y bits is then one integer addition on the fp32 pattern; the shift
    // k moves only the exponent, so the decoded scale is the rounded value itself.
    const int ev0 = e - 127 + k;
    if (e != 0 && f.y >= 1 && ev0 >= f.emin && ev0 < f.emax) {
      const int sh0 = 23 - f.y;
      const uint32_t rb = (b + ((1u << (sh0 - 1)) - 1u) + ((b >> sh0) & 1u)) & ~((1u << sh0) - 1u);
      r.s_hat = __uint_as_float(rb);
      r.code = (uint32_t)(((int)(rb >> 23) - 127 + k + f.bias) << f.y) | ((rb >> sh0) & ((1u << f.y) - 1u));
      return r;
    }
  }
  uint32_t m = b & 0x7FFFFFu;
  if (e == 0) {
    const int sh = __clz((int)m) - 8;
    m <<= sh;
    e = 1 - sh;
  } else {
    m |= 0x800000u;
  }
  const int ev = e - 127 + k;                  // exponent of the shifted value, m in [2^23, 2^24)
  const int sh = 23 - f.y + max(f.emin - ev, 0);
  uint32_t n;
  if (sh > 24) {
    n = 0;
  } else {
    const uint32_t q = m >> sh;
    const uint32_t rem = m & ((1u << sh) - 1u);
    const uint32_t half = 1u << (sh - 1);
    n = q + ((rem > half || (rem == half && (q & 1u))) ? 1u : 0u);
  }
  int code = ev >= f.emin ? ((ev + f.bias) << f.y) + (int)n - (1 << f.y) : (int)n;
  code = min(code, f.code_max);
  code = max(code, 1);
  r.code = (uint32_t)code;
  const int E = code >> f.y;
  const uint32_t M = (uint32_t)code & ((1u << f.y) - 1u);
  const uint32_t mant = E ? ((1u << f.y) + M) : M;
  r.s_hat = ldexp_once(mant, (E ? E : 1) - f.bias - f.y - k);
  return r;
}

// one power-of-two scale per layer: 2^ceil(log2(wmax / tmax))
__device__ __forceinline__ float layer_pot_scale(float wmax, float tmax) {
  if (!(wmax > 0.0f)) return 0.0f;
  const float sigma = __fdiv_rn(wmax, tmax);
  int e = ilogb_pos(sigma);
  const uint32_t b = __float_as_uint(sigma);
  const bool pow2 = (b >> 23) ? ((b & 0x7FFFFFu) == 0u) : (__popc(b) == 1);
  if (!pow2) e += 1;
  return ldexp_once(1u, e);
}

// FP element grids: round |u| to the nearest grid value (ties to even), saturating.
//   E2M3: min_eb = 127 (quantum 2^-3 below 2), vmax = 7.5;  E4M3: min_eb = 121, vmax = 448.
template <int KIND>
__device__ __forceinline__ float fp_quantize(float u) {
  constexpr int min_eb = KIND == SOP_KIND_FP_E2M3 ? 127 : 121;
  constexpr float vmax = KIND == SOP_KIND_FP_E2M3 ? 7.5f : 448.0f;
  const float au = fminf(fabsf(u), vmax);
  // 2^(exponent of au, at least the smallest normal one) * 2^20: adding and subtracting it rounds au to a
  // multiple of the binade's step (3 mantissa bits), ties to even
  const float magic = __uint_as_float(max(__float_as_uint(au) & 0x7F800000u, (uint32_t)min_eb << 23) + (20u << 23));
  const float q = __fsub_rn(__fadd_rn(au, magic), magic);
  return __uint_as_float(__float_as_uint(q) | (__float_as_uint(u) & 0x80000000u));
}

// Element grid given by parameters (SOP_KIND_FP_GRID): min_eb = biased fp32 exponent of the smallest normal
// magnitude (127 + 1 - bias), sh = 23 - man_bits, saturation at vpos above zero and at vneg below.
struct GridDev { int min_eb, sh; float vpos, vneg; };

__device__ __forceinline__ float grid_quantize(float u, const GridDev g) {
  const float au = fminf(fabsf(u), u < 0.0f ? g.vneg : g.vpos);
  const float magic = __uint_as_float(max(__float_as_uint(au) & 0x7F800000u, (uint32_t)g.min_eb << 23) + ((uint32_t)g.sh << 23));
  const float q = __fsub_rn(__fadd_rn(au, magic), magic);     // nearest multiple of the binade's step, ties to even
  return __uint_as_float(__float_as_uint(q) | (__float_as_uint(u) & 0x80000000u));
}

// magnitude number E * 2^y + M of a value already on such a grid, the sign at bit sign_pos
__device__ __forceinline__ uint32_t grid_code(float q, const GridDev g, int sign_pos) {
  const uint32_t b = __float_as_uint(q);
  const int y = 23 - g.sh;
  const int eb = (int)((b >> 23) & 255u);
  uint32_t mag;
  if (eb < g.min_eb) mag = (uint32_t)__float2int_rn(__fmul_rn(fabsf(q), __uint_as_float((uint32_t)(127 + 127 - g.min_eb + y) << 23)));
  else mag = ((uint32_t)(eb - g.min_eb + 1) << y) | ((b >> g.sh) & ((1u << y) - 1u));
  return ((b >> 31) << sign_pos) | mag;
}

// bit pattern sign|E|M of a value already on the grid
template <int KIND>
__device__ __forceinline__ uint32_t fp_code(float q) {
  constexpr int xb = KIND == SOP_KIND_FP_E2M3 ? 2 : 4;
  constexpr int bias = KIND == SOP_KIND_FP_E2M3 ? 1 : 7;
  const uint32_t b = __float_as_uint(q);
  const uint32_t sign = b >> 31;
  const float a = fabsf(q);
  uint32_t mag;
  if (a < pow2f_int(1 - bias)) {
    mag = (uint32_t)__float2int_rn(__fmul_rn(a, pow2f_int(bias - 1 + 3)));   // subnormal: M = a / 2^(1-bias-3)
  } else {
    const int E = (int)((b >> 23) & 255u) - 127 + bias;
    mag = ((uint32_t)E << 3) | ((b >> 20) & 7u);
  }
  return (sign << (xb + 3)) | mag;
}

// Decision thresholds of a table: tau[j] = largest fp32 <= (lut[j] + lut[j+1]) / 2, so that for
// every fp32 u "u > tau[j]" is exactly "u is strictly closer to lut[j+1] than to lut[j]".  A repeated
// entry takes the threshold above it, so its upper copy is never chosen.  tau[j] = +inf for j >= ne-1.
__device__ __forceinline__ void build_thresholds(const float* lut, int ne, float* tau /* 32 */) {
  float next = __int_as_float(0x7F800000);
  for (int j = 31; j >= 0; --j) {
    float t = __int_as_float(0x7F800000);
    if (j < ne - 1) t = (lut[j] == lut[j + 1]) ? next : __double2float_rd(0.5 * ((double)lut[j] + (double)lut[j + 1]));
    tau[j] = t;
    next = t;
  }
}

// number of thresholds strictly below u: branch-free binary search over 2^STEPS - 1 sorted entries (+inf
// padded to 31).  Five steps cover any table; four are enough for a table of at most 16 entries.
template <int STEPS = 5>
__device__ __forceinline__ int count_below(const float* tau, float u) {
  int pos = 0;
#pragma unroll
  for (int step = 1 << (STEPS - 1); step >= 1; step >>= 1)
    if (tau[pos + step - 1] < u) pos += step;
  return pos;
}

// 16-term fp32 sum in the fixed order: four quads of consecutive elements, sequential inside a
// quad, (Q0 + Q1) + (Q2 + Q3).
__device__ __forceinline__ float quad_tree(const float q[4]) {
  return __fadd_rn(__fadd_rn(q[0], q[1]), __fadd_rn(q[2], q[3]));
}

__device__ __forceinline__ float block_cosine(float nw, float nq, float dot) {
  if (nw == 0.0f && nq == 0.0f) return 1.0f;
  if (nw == 0.0f || nq == 0.0f) return 0.0f;
  return __fdiv_rn(dot, __fsqrt_rn(__fmul_rn(nw, nq)));
}

}  // namespace sop
