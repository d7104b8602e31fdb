/* libsop -- C-ABI boundary of the B200 (sm_100a) implementation of the Scaled Outer Product
 * per-layer candidate sweep.
 *
 * One linear layer at a time: W is M x K bf16 (row-major, K contiguous, leading dimension ldw),
 * calibration activations X are T x K fp32, blocks are g = 16 consecutive elements along K
 * (paper Section "Block Scaling": Y = X W^T, scales shared along the contracted dimension K).
 *
 * Conventions for every entry point
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; pointers without the suffix
 *     are HOST pointers read before the call returns.  The library never frees caller memory and
 *     allocates nothing that outlives a call; scratch comes from a caller-provided device
 *     workspace whose size the matching *_workspace() query reports.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     Outputs are valid after the stream has been synchronised.
 *   - Return value: SOP_OK (0) or a negative SOP_ERR_* code; nothing throws, aborts or traps.
 *     Argument errors are detected on the host before anything is launched.
 *   - Required: K % 16 == 0, M, K, T >= 1, ldw >= K, ldx >= K, M*K < 2^31 blocks*16, finite inputs.
 *   - A call works on the CUDA device that is current when it is made.  The library keeps a few facts per
 *     device ordinal (kernel attributes set once, the number of SMs, whether all Lloyd iterations fit one
 *     cooperative launch), so one process may drive several devices; calls are made from one host thread
 *     at a time.
 *   - sop_channel_norms, sop_opq_extract, sop_pair_search, sop_dd4_lloyd, sop_pack and sop_wr_extract can be recorded into a CUDA graph by
 *     stream capture once each has been called normally on the device (the first call does the one-time
 *     set-ups), with profiling off.
 */
#ifndef SOP_H_
#define SOP_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SOP_G 16               /* block size along K */
#define SOP_MAX_ATOMS 16       /* candidates per call, negations and FP formats included */
#define SOP_MAX_ENTRIES 32     /* table entries per LUT atom (n <= 5) */
#define SOP_K_AUTO (-1000)     /* k_mode: choose the F_layer shift on the device */
#define SOP_K_FROM_RESULT (-1001) /* k_mode: take the shift(s) from the result block of a previous search */
#define SOP_FMTA_FROM_RESULT (-1) /* fmta_index of sop_dd4_lloyd: best single LUT candidate of a previous search */
#define SOP_ALL_ATOMS 0xFFFFFFFFu /* eval_mask of sop_pair_search: evaluate every candidate */
#define SOP_SEARCH_SINGLES_ONLY 1 /* flags of sop_pair_search: reduce single candidates only, no pair / signed entries */
#define SOP_SEARCH_SELECT_MSE 2   /* flags of sop_pair_search: the per-block reassignment takes the smaller block error */
#define SOP_SEARCH_KEEP_LOADED_ENTRIES 4 /* flags of sop_pair_search: table entries among loaded candidates are kept, not formed again */
#define SOP_SEARCH_REUSE_PREPASS 8 /* flags of sop_pair_search: the shifts come from the exponent histograms an earlier call left in the workspace */

enum {
  SOP_OK = 0,
  SOP_ERR_NULL = -1,       /* a required pointer is NULL */
  SOP_ERR_SHAPE = -2,      /* M, K, T <= 0, K % 16 != 0, ld < K, g != 16, size beyond the supported range */
  SOP_ERR_FORMAT = -3,     /* bad scale format, or a sign / selector bit requested that the word does not have */
  SOP_ERR_ALPHABET = -4,   /* bad atom: n_entries, unsorted or non-finite table, tmax <= 0, too many atoms */
  SOP_ERR_WORKSPACE = -5,  /* workspace NULL, misaligned (256 B) or too small */
  SOP_ERR_CUDA = -6,       /* a CUDA runtime call failed; see sop_last_cuda_error() */
  SOP_ERR_RANGE = -7,      /* k shift outside [-64, 64], pool_rank outside [1, N_b], iters outside [0, 64] */
  SOP_ERR_TOO_LARGE = -8   /* sop_channel_norms_static: ceil(T/64) * K exceeds the built-in scratch */
};

enum { SOP_KIND_LUT = 0, SOP_KIND_FP_E2M3 = 1, SOP_KIND_FP_E4M3 = 2, SOP_KIND_FP_GRID = 3 };

/* Scale word magnitude format ExMy with optional sign (Section "Scale Format and Metabit
 * Allocation", SwExMy).  bias is 2^(x-1)-1 in every format the paper names.  Rounding is to
 * nearest even with gradual underflow; all exponent codes are finite unless top_exp_reserved;
 * overflow saturates; a positive scale never rounds to zero. */
typedef struct {
  int sign_bits;         /* w: 1 if the deployed word has a sign bit (enables the 4-way signed table) */
  int exp_bits;          /* x in [1, 8] */
  int man_bits;          /* y in [0, 10] */
  int bias;
  int top_exp_reserved;  /* 1: the all-ones exponent code is not used (needed for E8M7) */
} sop_scale_fmt;

/* One candidate codebook ("atom", Section "Per-Layer Pair Search").
 * LUT kind: lut[0..n_entries) ascending (repeats allowed), n_entries <= 2^n_bits <= 32.
 * negated = 1 makes the candidate -(lut): it is evaluated by running the table on -u, so that
 * code_{-a}(-w) == code_a(w) exactly, ties included.
 * FP kinds (E2M3: 6-bit, largest 7.5; E4M3: 8-bit OCP, largest 448) ignore lut.
 * SOP_KIND_FP_GRID: a floating-point element grid given by parameters (Section "Promotion Profiles":
 *   FP8 / FP10 / FP12-class promotion formats; paragraph "HIF7/HIF8 hardware rationale").  Magnitude
 *   number j = E * 2^y + M (y = grid_man_bits) has the value (M / 2^y) 2^(1 - grid_bias) for E = 0 and
 *   (1 + M / 2^y) 2^(E - grid_bias) otherwise.  The grid is the magnitudes up to tmax on the positive
 *   side and up to grid_neg_max >= tmax on the negative side (both must be grid values); rounding is to
 *   nearest, ties to the even magnitude number, saturating.  HIF7 is y = 3, bias = -2, tmax = 120,
 *   grid_neg_max = 128.  grid_exp_bits = x > 0 gives the element code sign | E | M with the sign above
 *   x + y bits; x = 0 marks a grid without such a code (it can be swept but not packed).  lut is ignored.
 * scope = 16: per-block scale in the layer's scale format, s = max|w_block| / tmax
 * ("LUT-scale coupling": the scale is taken against max(LUT)).
 * scope = 0: one power-of-two scale per layer, 2^ceil(log2(max|W| / tmax)) (the "^0" suffix). */
typedef struct {
  int n_bits;
  int kind;
  int negated;
  int scope;
  float tmax;
  int n_entries;
  float lut[SOP_MAX_ENTRIES];
  int grid_exp_bits;     /* SOP_KIND_FP_GRID only (zero otherwise): x in [0, 8] */
  int grid_man_bits;     /* y in [0, 10] */
  int grid_bias;         /* the smallest normal magnitude is 2^(1 - grid_bias) */
  float grid_neg_max;    /* largest magnitude on the negative side, >= tmax */
} sop_atom;

/* Per-layer statistics of one candidate or one candidate pair. */
typedef struct {
  double acos;       /* mean over blocks of the selected c-weighted block cosine (Section "ACos") */
  double mse;        /* sum over blocks of the selected squared error / (M K) */
  long long n_sel1;  /* blocks whose selector bit is 1 (second codebook); -1 marks an undefined entry */
  long long n_neg;   /* signed table only: blocks whose scale sign is negative */
} sop_pair_stat;

/* Device-resident result block of sop_pair_search (read it back with cudaMemcpy). */
typedef struct {
  int k[SOP_MAX_ATOMS];  /* F_layer shift used for each candidate (0 for scope-0 candidates) */
  int best_a, best_b;    /* best two-codebook pair a < b by ACos, ties to the smallest (a, b); -1 if none */
  int best_single;       /* best single LUT candidate by ACos, ties to the lowest index; -1 if none */
  int best_sa, best_sb;  /* best pair of the signed table; -1 if none */
  float layer_absmax;    /* max |W| */
  int reserved[2];
} sop_search_result;

const char* sop_strerror(int code);
/* Text of the last CUDA runtime error seen by this thread inside the library ("" if none). */
const char* sop_last_cuda_error(void);
int sop_version(void);

/* ---- channel norms:  c_k = sqrt((1/T) sum_t X[t,k]^2)   (Section "Channel Norms") ----------
 * X_dev: T x K fp32, row stride ldx.  c_dev: K fp32.  Accumulation in FP64; order: chunks of 64
 * rows, sequential fused multiply-add inside a chunk, chunk partials added in chunk order, so the
 * result is bit-reproducible.  Workspace: ceil(T/64) * K doubles. */
int sop_channel_norms_workspace(long long T, long long K, size_t* bytes);
int sop_channel_norms(const float* X_dev, long long T, long long K, long long ldx, float* c_dev,
                      void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---- channel norms for callers that cannot allocate (the paper has no counterpart: this is a
 *      packaging variant of sop_channel_norms, same arithmetic, same result bit for bit) ---------
 * Who needs it: a caller that may not, or cannot, obtain device memory for the workspace -- a
 * serving process that handed all device memory to its own arena at start-up and treats any later
 * cudaMalloc as a fault, a latency-critical loop that must avoid the device-wide synchronisation
 * that cudaMalloc / cudaFree imply, or a plug-in that is handed only the tensors and owns no
 * allocator.  This entry point takes no workspace and calls no allocation routine: its scratch is
 * a fixed array of SOP_NORMS_STATIC_DOUBLES doubles (4 MiB) that is part of the library image on
 * every GPU that loads the library, for the life of the process.
 *   Limit: ceil(T / 64) * K <= SOP_NORMS_STATIC_DOUBLES, else SOP_ERR_TOO_LARGE (for example
 *   T = 2048 tokens at K = 14336, or T = 1024 at K = 28672, fit; T = 4096 at K = 14336 does not).
 *   First call on a device: looks up the array's device address (one cudaGetSymbolAddress with that
 *   device current) and remembers it; make that first call outside any stream capture.
 *   Sharing: every call on a device uses the same array and finds the previous call's partials in
 *   it.  Nothing needs clearing (each call overwrites every partial it reads), but two calls whose
 *   kernels can overlap on the GPU -- different streams, no ordering between them -- would
 *   overwrite each other's partials: order such calls (one stream, or events).
 * X_dev, T, K, ldx, c_dev, stream: as for sop_channel_norms. */
#define SOP_NORMS_STATIC_DOUBLES (1 << 19)
int sop_channel_norms_static(const float* X_dev, long long T, long long K, long long ldx, float* c_dev, void* stream);

/* ---- the candidate sweep (Sections "Block Scaling", "ACos", "Per-Layer Pair Search" step 4,
 *      "Per-layer scale shift") ----------------------------------------------------------------
 * For every block and every candidate: scale = Q_fmt(absmax / tmax * 2^k) * 2^-k, codes = nearest
 * table entry (or nearest-even FP grid value) of w * (1 / scale), c-weighted block cosine and
 * squared error in fp32 with a fixed summation order; then per layer, in FP64:
 *   pair_table_dev [n_atoms x n_atoms]: [a][a] = candidate a alone; [a][b], a < b, both LUT atoms of
 *     equal n_bits = two-codebook quantisation with per-block selector [cos_b > cos_a];
 *     other entries are marked n_sel1 = -1.
 *   signed_table_dev [n_atoms x n_atoms] (may be NULL; filled only when fmt->sign_bits = 1): for
 *     base atoms i <= j, each immediately followed in `atoms` by its own negation, the per-block
 *     best of {i, -i, j, -j}, ties resolved in that order.
 *   result_dev: shifts, best pair, best single.
 *   block_cos_dev / block_sse_dev (may be NULL): [n_atoms x N_b] per-block values, N_b = M*K/16,
 *     block index = m * (K/16) + j.
 * k_mode: SOP_K_AUTO runs the F_layer search per distinct tmax (maximise the number of blocks whose
 *   shifted scale exponent lies in the format's normal range, k in [-64, 64], ties to the smallest
 *   |k| then to k > 0); SOP_K_FROM_RESULT: see prev_result_dev; any other value in [-64, 64] is used as
 *   the shift for every candidate.
 * dd_lut_dev (may be NULL): device table of SOP_MAX_ENTRIES floats that replaces, at kernel time,
 *   the lut of every atom whose index bit is set in dd_mask (a codebook produced by sop_dd4_lloyd
 *   can be swept without a host round trip).
 * eval_mask / load_mask: the sweep in two calls ("only the new columns").  Candidates in eval_mask
 *   (SOP_ALL_ATOMS: all) are evaluated; candidates in load_mask are not evaluated again: their
 *   per-block cosine and error are read from block_cos_dev / block_sse_dev as an earlier call on
 *   the same layer, alphabet, format and shift wrote them (both arrays are then required).  A
 *   candidate in neither mask is absent: every table entry that involves it is marked undefined and
 *   its shift is reported as 0.  The masks must be disjoint and not both empty.  At most 8 distinct
 *   tables may be evaluated per call (an atom and its negation share one).  The lookup tables of the
 *   evaluated candidates live in shared memory; when a fine-grained alphabet would not fit beside the
 *   staging tile, the lookup grid is coarsened and the tables that then share a cell between thresholds are
 *   searched exactly instead (slower, same results): no alphabet within the limits above is refused for size.
 * flags: SOP_SEARCH_SINGLES_ONLY fills only the diagonal (and best_single): enough to choose the
 *   primary codebook FMTa before the Lloyd refinement.  SOP_SEARCH_SELECT_MSE (paragraph "Pair-search
 *   design axes", axis ii): in every two-way and signed entry the block goes to the candidate with the
 *   smaller block squared error instead of the larger block cosine (ties keep the earlier candidate);
 *   acos, mse and the counts are those of that assignment, the best pair is still ranked by acos.
 *   SOP_SEARCH_REUSE_PREPASS: the exponent histogram of the block scales and max|W| do not depend on the scale
 *   format, so a layer that is swept at several scale formats needs them once.  With this flag the call takes them
 *   from workspace_dev as the last call without the flag (and without SOP_K_FROM_RESULT) left them, and only derives
 *   this format's shifts: the caller guarantees that W, M, K, the alphabet and eval_mask are those of that call
 *   (calls with SOP_K_FROM_RESULT in between leave the histograms alone).  Ignored with SOP_K_FROM_RESULT.
 * prev_result_dev (may be NULL): with k_mode = SOP_K_FROM_RESULT, the result block of the earlier call on
 *   this layer (not result_dev itself).  The shift of every scale class and max|W| are taken from it
 *   instead of reading W once more; every per-block-scaled class of this call must then contain a
 *   candidate of load_mask (SOP_ERR_RANGE otherwise). */
int sop_pair_search_workspace(long long M, long long K, int n_atoms, size_t* bytes);
/* Launch shape of the reduction of the table entries (no counterpart in the paper): reduce_tile_pairs = 1 (the
 * default) lets a CTA work on two tiles of 256 blocks at a time where its shared memory allows, 0 keeps it to one.
 * The additions and their order are the same: results do not depend on it.  SOP_ERR_RANGE for other values. */
int sop_pair_search_tuning(int reduce_tile_pairs);
int sop_pair_search(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                    const sop_scale_fmt* fmt, int k_mode, const sop_atom* atoms, int n_atoms,
                    const float* dd_lut_dev, unsigned dd_mask, unsigned eval_mask, unsigned load_mask, int flags,
                    const sop_search_result* prev_result_dev,
                    sop_pair_stat* pair_table_dev, sop_pair_stat* signed_table_dev,
                    sop_search_result* result_dev, float* block_cos_dev, float* block_sse_dev,
                    void* workspace_dev, size_t workspace_bytes, void* stream);

/* Measurement aid (no counterpart in the paper): with profiling enabled, an entry point records a
 * CUDA event on `stream` directly before the first and after the last launch of its main kernel:
 *   SOP_PROFILE_SWEEP   the sweep kernel of sop_pair_search (one launch; the events coincide when the call evaluates nothing)
 *   SOP_PROFILE_REDUCE  the reduction kernel(s) of sop_pair_search
 *   SOP_PROFILE_LLOYD   the iteration kernel(s) of sop_dd4_lloyd, or the launches of its dynamic programme
 *   SOP_PROFILE_POOL    what sop_dd4_lloyd launches before them: radix select, set-up, pool list, pool cache
 *   SOP_PROFILE_PREPASS the shift prepass of sop_pair_search (the events coincide when the call takes its shifts from a result)
 *   SOP_PROFILE_OPQ     the three kernels of sop_opq_extract
 *   SOP_PROFILE_WR      the kernels of sop_wr_extract
 *   SOP_PROFILE_PACK    the kernel of sop_pack
 *   SOP_PROFILE_NORMS   both kernels of sop_channel_norms
 * sop_profile_ms waits for the second event of a call of that kind (back = 0: the last call, 1: the one
 * before, ... up to 7) and returns the time between its two events in milliseconds (SOP_ERR_RANGE if
 * no such call has run since profiling was enabled).  Not thread-safe. */
enum { SOP_PROFILE_SWEEP = 0, SOP_PROFILE_LLOYD = 1, SOP_PROFILE_PACK = 2, SOP_PROFILE_NORMS = 3, SOP_PROFILE_REDUCE = 4, SOP_PROFILE_POOL = 5,
       SOP_PROFILE_PREPASS = 6, SOP_PROFILE_OPQ = 7, SOP_PROFILE_WR = 8, SOP_PROFILE_KINDS = 9 };
int sop_profile_enable(int on);
int sop_profile_ms(int which, int back, float* ms);
int sop_profile_last_ms(int which, float* ms);    /* = sop_profile_ms(which, 0, ms) */
int sop_profile_last_sweep_ms(float* ms);   /* = sop_profile_last_ms(SOP_PROFILE_SWEEP, ms) */

/* ---- DD-n: per-layer data-derived codebook by Lloyd iteration (pair-search steps 2-3) -------
 * Pool = blocks at least as bad under the primary codebook FMTa as the pool_rank-th worst of the
 * layer (ties all in).  By default "bad" is a small block cosine.  Each iteration assigns every pool
 * element u = w / scale (scale against tmax = 1) to its nearest entry, accumulates per entry
 * sum(omega) and sum(omega u) with omega = c / max(c) in int64 fixed point (2^-24 units, |omega u|
 * clamped to 256), replaces each non-empty entry by its centroid snapped to bf16, and re-sorts.
 *   fmta_index: index into `atoms` of FMTa (its table is the initial codebook), or
 *     SOP_FMTA_FROM_RESULT to use search_dev->best_single.
 *   block_metric_dev: [n_atoms x N_b] as written by sop_pair_search (row fmta is read): the block
 *     cosines, or with SOP_LLOYD_POOL_BY_ERROR the block squared errors.
 *   pool_rank in [1, N_b].  The p % rule of the paper is the rank ceil(N_b (100 - p) / 100); a top-k
 *     pool is the rank k.
 *   flags (paragraph "Pair-search design axes"):
 *     SOP_LLOYD_POOL_BY_ERROR    axis (i): rank the blocks by their squared error (the largest are the worst);
 *     SOP_LLOYD_UNIFORM_WEIGHTS  axis (iii): omega = 1 for every channel;
 *     SOP_LLOYD_POOL_THRESHOLD   axis (iv): the pool is every block whose metric is at least as bad as
 *       pool_threshold (cosine <= threshold, or error >= threshold); pool_rank is ignored.  An empty pool
 *       leaves the table as it is.
 *     SOP_LLOYD_LAUNCH_PER_ITERATION  (no counterpart in the paper) one kernel launch per iteration even
 *       where all iterations could run in one cooperative launch; the results are the same.
 *     SOP_LLOYD_GRID_DP  the grid-constrained construction of pair-search steps 1 and 3 ("histogram-DP cluster
 *       selection on the deployed LUT value format's grid points") instead of Lloyd iterations with a snap: the pool
 *       elements u are binned into cells of width 2^-8 over [-1.25, 1.25] (cell = rint(256 u), clamped) with the
 *       integer sums H = sum fix(omega), S = sum fix(omega u), Q = sum fix((omega u) u) per cell; the cells with
 *       H > 0 are cut, in ascending order, into min(n_entries, cells) runs; a run's code point is the bf16 value
 *       nearest to S / H (clamped to +-1.25) and its cost Q - 2 q S + q^2 H in FP64; a dynamic programme finds the
 *       cut of least total cost (ties to the earliest cut).  iters must be 0; out_lut_dev receives the code points in
 *       ascending order (padded with the last one when there are fewer cells than entries) and distortion_dev[0]
 *       the least total cost.  With fmta_index = SOP_FMTA_FROM_RESULT every table atom must have the same n_entries.
 *   k_mode: a shift in [-64, 64], or SOP_K_FROM_RESULT to use search_dev->k[fmta].
 *   out_lut_dev: SOP_MAX_ENTRIES floats (first n_entries valid, ascending).
 *   distortion_dev: iters + 1 doubles, sum omega (u - q)^2 before each update and after the last.
 *     The last entry doubles as the status of the call: it is set to -1 when the call starts and to the final
 *     distortion (never negative) by the closing iteration.  When the iterations run in one launch, its CTAs
 *     wait for one another between iterations; every wait is bounded (about half a second).  A CTA that gives
 *     up makes all of them leave and the last entry stays (or is set back to) -1: the table is then not valid.
 *     A caller reads distortion_dev[iters] after synchronising and treats a negative value as a failed call.
 *   pool_count_dev: one long long, number of blocks in the pool.
 * Workspace: 8 bytes per weight element (u and omega of every pool element are kept across the
 *   iterations), 4 bytes per block (the pool list) and 4 bytes per channel, plus a fixed header. */
#define SOP_LLOYD_POOL_BY_ERROR 1
#define SOP_LLOYD_UNIFORM_WEIGHTS 2
#define SOP_LLOYD_POOL_THRESHOLD 4
#define SOP_LLOYD_LAUNCH_PER_ITERATION 8
#define SOP_LLOYD_GRID_DP 16
int sop_dd4_lloyd_workspace(long long M, long long K, size_t* bytes);
/* Number of kernel launches one sop_dd4_lloyd call with these sizes and flags makes on the current device
 * (measurement aid, no counterpart in the paper).  All iterations run in one cooperative launch where the
 * device supports such launches (the grid is cut to what is resident at once); otherwise, or with
 * SOP_LLOYD_LAUNCH_PER_ITERATION, there is one launch per iteration.  With SOP_LLOYD_GRID_DP pass the number of
 * table entries as `iters`: the dynamic programme takes one launch per row plus two. */
int sop_dd4_lloyd_launches(long long M, long long K, int iters, int flags, int* launches);
/* Launch-shape parameters of sop_dd4_lloyd for this process (test aid, no counterpart in the paper; results do
 * not depend on them).  cell_spill_tiles in [1, 128]: cache tiles a CTA sorts between two transfers of its
 * per-cell partial sums to the global sums (default 128, the most the 32-bit limbs allow);
 * cache_ctas >= 0: largest grid of the cache kernel (0 = default, three CTAs per SM);
 * tiles_per_warp in [1, 4]: cache tiles one warp of an iteration CTA walks between two folds of its 32-bit partial
 *   sums into 64-bit ones (default 4, the most the partial sums hold).
 * iter_ctas >= 0: largest grid of the iteration kernels (0 = default: one warp per cache tile of the expected pool,
 *   at most eight CTAs per SM and, in one cooperative launch, what is resident at once).
 * SOP_ERR_RANGE outside these ranges. */
int sop_dd4_lloyd_tuning(int cell_spill_tiles, int cache_ctas, int tiles_per_warp, int iter_ctas);
int sop_dd4_lloyd(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                  const sop_scale_fmt* fmt, int k_mode, const sop_search_result* search_dev,
                  const float* block_metric_dev, long long pool_rank, float pool_threshold, int flags,
                  const sop_atom* atoms, int n_atoms,
                  int fmta_index, int iters, float* out_lut_dev, double* distortion_dev,
                  long long* pool_count_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---- materialise: codes + scale words for the chosen codebook(s) (Section "Overview" item 4:
 *      2n bytes of codes per block; Section "Scale Format": bit placement) ---------------------
 * Candidates per block in priority order a, (-a if use_sign), b, (-b if use_sign); the largest
 * block cosine wins, ties keep the earlier.  selector = winner is b or -b; sign = winner is a
 * negated variant.
 *   atoms / n_atoms / dd_lut_dev / dd_mask: the alphabet, as for sop_pair_search.
 *   index_a, index_b: indices into `atoms`; index_b = SOP_NO_ATOM packs a single codebook;
 *     index_a = SOP_PAIR_FROM_RESULT takes the pair from search_dev (best_sa/best_sb when use_sign,
 *     else best_a/best_b) so that the whole layer pipeline runs without a host round trip.
 *   k_mode: a shift in [-64, 64] used for both atoms, or SOP_K_FROM_RESULT (search_dev->k[index]).
 *   codes_dev: N_b * 2n bytes, 16-byte aligned; block payload = one little-endian 16n-bit integer,
 *     element r in bits [r n, r n + n).  LUT atoms: table index (for a negated table: the index found on -u);
 *     FP atoms: the format's bit pattern sign|E|M.
 *   words_dev: ceil(N_b * container_bits / 8) bytes, rounded up to a multiple of 4 (the stream is
 *     written with 32-bit operations; the pointer must be 4-byte aligned), little-endian bit stream
 *     of b-bit words in block order (b = 12: two words per three bytes; b in {8, 12, 16}).  Word layout:
 *     word_sign_bits = 1: sign at bit b-1, selector at bit 0, magnitude E:M above the
 *     m = b-1-x-y metabits; word_sign_bits = 0: selector at bit b-1 (if m >= 1), magnitude above
 *     the remaining m-1 metabits.  Unused metabits are zero.
 *   counts_dev (may be NULL): two long long {n_sel1, n_neg}, overwritten.  With index_a = SOP_PAIR_FROM_RESULT
 *     the search result may hold no pair (a singles-only search, a search without a signed table while
 *     use_sign = 1, an alphabet with one base atom): nothing is packed then, codes_dev is left as it was and
 *     counts_dev receives {-1, -1}; pass counts_dev whenever the pair comes from a result block.
 *   flags: SOP_PACK_SELECT_MSE (paragraph "Pair-search design axes", axis ii): the smallest block squared
 *     error wins instead of the largest block cosine, ties keep the earlier candidate.
 *   block_metric_dev (may be NULL): [n_atoms x N_b] per-block cosines (with SOP_PACK_SELECT_MSE: per-block
 *     errors) written by sop_pair_search for the same layer, alphabet, format and shift.  When every
 *     candidate of the choice has a row there (with use_sign, the negated variant of an atom is the atom
 *     of the alphabet with the same table and the opposite `negated`; from a search result it is the next
 *     atom), the winner of each block is read off these values and only the winner is encoded: the output
 *     is identical, the cost drops to one encode per block.  Otherwise the candidates are evaluated here. */
#define SOP_NO_ATOM (-2)
#define SOP_PAIR_FROM_RESULT (-1)
#define SOP_PACK_SELECT_MSE 1
int sop_pack(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
             const sop_scale_fmt* fmt, const sop_atom* atoms, int n_atoms, const float* dd_lut_dev,
             unsigned dd_mask, int index_a, int index_b, int k_mode, const sop_search_result* search_dev,
             int use_sign, int container_bits, int word_sign_bits, unsigned char* codes_dev,
             unsigned char* words_dev, long long* counts_dev, const float* block_metric_dev, int flags, void* stream);

/* ---- OPQ: outlier extraction before the search (Section "Outlier Per-Quantum Extraction (OPQ)") ----
 * Positions with |w_i| / sigma_b > m are taken out of the codebook input and kept as exact bf16 values in a
 * sparse stream.  sigma_b = sqrt(mean_j w_j^2) over the block's g = 16 elements (the paper names sigma_b
 * without defining it), so the test is w_i^2 g > m^2 sum_j w_j^2; it is taken in binary64 (squares of bf16
 * values are exact, the sum runs in element order, one product on the right), so the decision does not
 * depend on the device.  A zero block has no outlier.
 *
 * sop_opq_threshold (host only): the m with F_M(m) = (2 Phi(m) - 1)^M = q, Phi the standard normal CDF,
 * M = max_order (the paper's default: M = g = 16, q = 0.92).  q in (0, 1), max_order >= 1, else SOP_ERR_RANGE.
 *
 * sop_opq_extract:
 *   W_dev [M x K] bf16, ldw as for sop_pair_search; m: the threshold, in (0, 1e6).
 *   W_out_dev [M x K] bf16 with row stride ldo (16-byte aligned, ldo % 8 == 0, ldo >= K), overwritten: W with
 *     every outlier replaced by +0; it is the input of the search that follows.  Must not be W_dev
 *     (SOP_ERR_RANGE): the stream is read from the untouched input.
 *   Stream: records ascend by (row, column); a record is the column k in bits 0-15 and the bf16 pattern of
 *     the weight in bits 16-31 (32 bits per outlier, as the paper counts them), so K <= 65536 (SOP_ERR_SHAPE
 *     beyond).  row_start_dev [M + 1] unsigned, overwritten: first record of every row, [M] = the number of
 *     records.  records_dev [capacity] unsigned: records beyond `capacity` are counted but not written (compare
 *     *count_dev with the capacity; M * K always suffices).  count_dev: one long long, overwritten.
 *   workspace_dev: sop_opq_workspace bytes, 256-byte aligned.
 * Inference applies the stream as Y[t, m] += sum over the row's records of value * X[t, k]; that step is
 * outside this library. */
int sop_opq_threshold(double q, int max_order, double* m_out);
int sop_opq_workspace(long long M, long long K, size_t* bytes);
int sop_opq_extract(const void* W_dev, long long M, long long K, long long ldw, int g, double m,
                    void* W_out_dev, long long ldo, unsigned* row_start_dev, unsigned* records_dev, long long capacity,
                    long long* count_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---- Wr: sparse correction of the codebook residual (Section "Sparse Residual Correction (Wr)") ----
 * E = W - W_hat for the packed layer, the entries with the largest activation-weighted magnitude |E_mk| c_k
 * are stored as a sparse stream with E3M4 values.  W_hat is decoded from the stream sop_pack wrote (scale
 * word -> sign, selector, scale; codes -> table values), E_i = w_i - s_hat q_i with one rounding, the metric
 * is the binary32 product |E_i| c_k.  The paper fixes neither ties nor the value scaling; here:
 *   n_keep (in [1, M K], the "top sigma" as a rank, e.g. ceil(0.001 M K)): tau = the n_keep-th largest metric
 *     of the layer; an entry is kept when its metric >= tau (ties all in) and > 0;
 *   values: E3M4 = sign, 3 exponent bits (bias 3, the all-ones exponent left out), 4 mantissa bits, largest
 *     15.5; the code is the nearest grid point (ties to the even magnitude number) of E / 2^e with one
 *     exponent e per layer, the smallest e with max |E_kept| / 2^e <= 15.5 (the stream's header).
 *   Arguments W_dev .. words_dev: exactly those given to sop_pack for this layer (codes_dev and words_dev now
 *     inputs); with index_a = SOP_PAIR_FROM_RESULT and a result without a pair nothing was packed: no record
 *     is written and *count_dev = -1.
 *   Stream: as for sop_opq_extract, a record is the column k in bits 0-15 and the E3M4 code in bits 16-23;
 *     row_start_dev [M + 1], records_dev [capacity], count_dev as there.  scale_exp_dev: one int, e (0 when
 *     nothing is kept).  tau_dev (may be NULL): one float, tau.
 *   workspace_dev: sop_wr_workspace bytes, 256-byte aligned.
 * The residual is never stored (W, codes and scale words are 2.6 bytes per element, a stored residual 4): one
 * decode pass histograms the block maxima of the metric, which bounds the threshold from below; a second one
 * collects the elements above that bound (typically a fraction of a per cent) into a candidate list in the
 * workspace, from which the threshold, the kept set and the stream follow.  A layer whose candidates do not fit
 * the list (more than max(65536, M K / 64): metrics nearly all alike) is handled by full decode passes instead;
 * the results are the same. */
int sop_wr_workspace(long long M, long long K, size_t* bytes);
int sop_wr_extract(const void* W_dev, long long M, long long K, long long ldw, const float* c_dev, int g,
                   const sop_scale_fmt* fmt, const sop_atom* atoms, int n_atoms, const float* dd_lut_dev, unsigned dd_mask,
                   int index_a, int index_b, int k_mode, const sop_search_result* search_dev, int use_sign,
                   int container_bits, int word_sign_bits, const unsigned char* codes_dev, const unsigned char* words_dev,
                   long long n_keep, unsigned* row_start_dev, unsigned* records_dev, long long capacity,
                   long long* count_dev, int* scale_exp_dev, float* tau_dev, void* workspace_dev, size_t workspace_bytes,
                   void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SOP_H_ */
