/*
 * vardrop.h -- C ABI of the B200 (sm_100a) implementation of VarDrop's per-batch training path
 * (Kang et al., "VarDrop: Enhancing Training Efficiency by Reducing Variate Redundancy in Periodic Time
 * Series Forecasting", AAAI-25).
 *
 * The path, in the order a training step calls it:
 *   vardrop_hash      k-dominant frequency hashing of a batch (Algorithm 1)
 *   vardrop_select    grouping by hash value and stratified sampling (Eq. 1, Eq. 2)
 *   vardrop_attn_fwd  gather of the kept Q/K/V variate tokens + scaled dot-product attention (Eq. 3)
 *   vardrop_attn_bwd  derivative of Eq. 3 over the kept tokens, gradients scattered to the full layout
 *
 * Conventions shared by every entry point
 *   - Pointers named in the argument lists are DEVICE pointers unless the comment says "host".
 *     Configuration structs are host pointers and are read before the call returns.
 *   - The caller owns every buffer, including the workspace `ws` (size from the matching
 *     *_workspace_bytes query).  The library never allocates or frees device memory, never
 *     synchronises the device and launches only on `stream` (a cudaStream_t passed as void*).
 *   - Device pointers must be 16-byte aligned.
 *   - The return value is a vardrop_status.  Problems found on the host (bad argument, unsupported
 *     shape, short workspace, failed launch) are returned at once and nothing is launched.  Problems
 *     found on the device (non-finite amplitude, a bounded wait that ran out) are written to the
 *     first int32 of `ws` as a vardrop_status; read it with a device-to-host copy after
 *     synchronising the stream.  The word is sticky: the first device-side problem is recorded and stays
 *     until the caller zeroes it, so zero the first int32 of a new workspace (and after handling an
 *     error); the library itself never clears it, which keeps a problem of an earlier queued call
 *     readable after later ones.  vardrop_last_error() gives a thread-local text for the last non-OK return.
 *   - Kernels are launched with programmatic stream serialization: a kernel's set-up may overlap the
 *     tail of the previous kernel on the same stream, its reads and writes do not.
 *   - Calls are thread-safe as long as concurrent calls use different workspaces.
 */
#ifndef VARDROP_H_
#define VARDROP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    VARDROP_OK = 0,
    VARDROP_ERR_INVALID_ARG = 1,   /* null/misaligned pointer, size out of range                       */
    VARDROP_ERR_UNSUPPORTED = 2,   /* e.g. L above 8192, head dimension other than 32/64 */
    VARDROP_ERR_WORKSPACE = 3,     /* ws_bytes below the *_workspace_bytes answer                      */
    VARDROP_ERR_CUDA = 4,          /* a CUDA runtime call or launch failed                             */
    VARDROP_ERR_TIMEOUT = 5,       /* device side: a bounded wait gave up (device status word only)    */
    VARDROP_ERR_NONFINITE = 6      /* device side: a candidate amplitude was NaN or infinite           */
} vardrop_status;

/* Static text for a status code; never freed. */
const char* vardrop_status_string(int status);
/* Thread-local detail of the last non-OK return on this thread ("" if none). */
const char* vardrop_last_error(void);
/* Library version, "major.minor". */
const char* vardrop_version(void);
/* Reads the device status word at the head of workspace `ws` (see "Problems found on the device" above): queues a
 * 4-byte device-to-host copy on `stream`, waits for that stream, and returns the vardrop_status found there
 * (VARDROP_ERR_CUDA when the copy itself fails).  This is the one entry point that synchronises; it never clears
 * the word. */
int vardrop_ws_status(const void* ws, void* stream);

/* Failure-handling check (no counterpart in the paper).  Every wait inside the library's kernels is bounded: when it runs out the
 * kernel records VARDROP_ERR_TIMEOUT in the status word and leaves through its normal exit, so the context stays usable.
 * This call launches one warp that waits `limit_us` microseconds (1 .. 100000) on a barrier nothing ever completes, through
 * that same wait, so that the path can be seen to work: afterwards vardrop_ws_status(ws) is VARDROP_ERR_TIMEOUT and later
 * calls on the stream run normally.  ws: at least 256 bytes. */
int vardrop_probe_bounded_wait(void* ws, size_t ws_bytes, unsigned int limit_us, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Measurement aids (no counterpart in the paper).
 *   vardrop_launch_count          kernels this library has launched in this process so far.
 *   vardrop_profile_enable(on)    arms (1) or disarms (0) the per-kernel timer and drops what it had collected.
 *                                 While armed every kernel launch is bracketed by a pair of CUDA events on its
 *                                 stream (host-side objects owned by the library), which costs a little idle
 *                                 time between kernels: arm it only for profiling passes.
 *   vardrop_profile_kernels       number of distinct kernels; ids are 0 .. count-1.
 *   vardrop_profile_kernel_name   name of kernel `id`.
 *   vardrop_profile_read          waits for the recorded events of kernel `id` and returns the sum of their
 *                                 durations (host pointers: total_ms, launches).
 * ---------------------------------------------------------------------------------------------- */
long long vardrop_launch_count(void);
int vardrop_profile_enable(int on);
int vardrop_profile_kernels(void);
const char* vardrop_profile_kernel_name(int id);
int vardrop_profile_read(int id, double* total_ms, long long* launches);

/* ------------------------------------------------------------------------------------------------
 * k-dominant frequency hashing -- Algorithm 1 ("k-Dominant Frequency Hashing") and Definition 1.
 *
 *   step 1  amplitude spectrum A[b,n,f] = |sum_t x[b,n,t] exp(-2 pi i f t / L)| of every window
 *   step 2  low-pass filter: only the bins f_lo <= f < f_hi are candidates
 *   step 3  scope 0: mean over the batch, Abar[n,f] = (1/B) sum_b A[b,n,f]   (S = 1 hash row)
 *           scope 1: every instance hashed on its own, Abar[b,n,f] = A[b,n,f] (S = B hash rows)
 *   step 4  the k candidate bins of largest Abar in descending-amplitude order; equal amplitudes
 *           rank the lower bin first
 *   step 5  hash value = the ordered k-tuple packed 12 bits per bin, rank-1 bin most significant
 *
 * cfg (host)  B, N, L  shape of x;  1 <= k <= 5;  f_lo/f_hi candidate band, both 0 selects the default
 *             f_lo = 1, f_hi = ceil((L/2+1)/2) (25 at L = 96, the cut-off of Appendix E);
 *             requires 0 <= f_lo, f_lo + k <= f_hi <= L/2+1, f_hi <= 4096 and L <= 8192 (prime factors of L above 7 are
 *             transformed as plain sums, at a cost that grows with the factor).
 * x           [B, N, L] float32, contiguous.
 * keys        [S, N] uint64 out.
 * freqs       [S, N, k] int32 out, the ranked bins; may be NULL.
 * amp_dbg     [S, N, f_hi - f_lo] float32 out, Abar; may be NULL.
 * ws          no scratch is used beyond the status word; pass at least vardrop_hash_workspace_bytes.
 * Device status: VARDROP_ERR_NONFINITE when a candidate amplitude is not finite (keys then unspecified).
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t B, N, L, k;
    int32_t f_lo, f_hi;
    int32_t scope;
} vardrop_hash_cfg;

size_t vardrop_hash_workspace_bytes(const vardrop_hash_cfg* cfg);
int vardrop_hash(const float* x, const vardrop_hash_cfg* cfg, uint64_t* keys, int32_t* freqs, float* amp_dbg,
                 void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Grouping and stratified sampling -- last sentence of "Procedure of k-DFH" (variates with the same
 * hash value form a group), Eq. 1 (|S_i| = min(|G_i|, gs)), Eq. 2 (S = union of the S_i), and the
 * token reduction ratio delta = 1 - n_sel / N of Sec. 3.3.
 *
 * Per hash row s (S rows, independent):
 *   groups    classes of equal key; group ids are dense ranks in ascending key order; members of a
 *             group are ordered by ascending variate index
 *   quota     q_g = min(|G_g|, gs if gs > 0, max(1, ceil(|G_g| * rate_ppm / 10^6))), rate_ppm =
 *             round(rate * 10^6), integer arithmetic; rate = 1 is Eq. 1 itself
 *   sampling  member j of group g gets priority = word 0 of Philox4x32-10(counter (j, g, s, step),
 *             key (seed low, seed high)); the q_g members of smallest (priority, j) are kept
 *
 * cfg (host)    S, N (1 <= N <= 65536), gs (<= 0: no cap), rate in (0, 1], seed, step.
 * keys          [S, N] uint64 in.
 * group_id      [S, N] int32 out.
 * group_offsets [S, N+1] int32 out; entry g is the start of group g in `members`, entries past the
 *               number of groups equal N.
 * members       [S, N] int32 out; variates sorted by (key, index).
 * n_groups      [S] int32 out.
 * sel_idx       [S, N] int32 out; kept variates ascending, first n_sel[s] valid, the rest -1.
 * n_sel         [S] int32 out.
 * inv_idx       [S, N] int32 out; position of variate n in sel_idx, or -1 when dropped.
 * ws            scratch of vardrop_select_workspace_bytes; contents are scratch only.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t S, N, gs;
    double rate;
    uint64_t seed;
    uint32_t step;
} vardrop_select_cfg;

size_t vardrop_select_workspace_bytes(const vardrop_select_cfg* cfg);
int vardrop_select(const uint64_t* keys, const vardrop_select_cfg* cfg, int32_t* group_id, int32_t* group_offsets,
                   int32_t* members, int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx,
                   void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * vardrop_select without a workspace (the paper has no counterpart; this is a packaging variant).
 *
 * For callers that cannot obtain device memory at the point where they select tokens: code running
 * inside a framework whose allocator is locked or already exhausted, plug-ins that are handed
 * input/output buffers and nothing else, or hosts that forbid cudaMalloc after start-up.  The
 * scratch that vardrop_select takes as `ws` lives here in a fixed 400 KiB array that is part of
 * the library image; every GPU that loads the library carries that array until the process ends.
 *
 * Same arguments, outputs and results as vardrop_select, minus ws / ws_bytes.
 * Limit: S * N <= 16384; larger problems return VARDROP_ERR_UNSUPPORTED (use vardrop_select).
 * It never calls cudaMalloc, cudaFree or any allocating routine.  For N <= 2048 it issues one kernel launch
 * and the built-in array is not touched; for larger N it issues one cudaMemsetAsync and three kernel
 * launches on `stream`, all working in that array.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and caches it; make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps whatever the previous call left: the parts
 * that must start at zero are cleared at the head of every call, so back-to-back calls on one stream
 * are fine, but two calls whose GPU work overlaps (different streams, different threads) race and
 * give wrong results.  There is no device status word to read back for this variant.
 * ---------------------------------------------------------------------------------------------- */
int vardrop_select_static(const uint64_t* keys, const vardrop_select_cfg* cfg, int32_t* group_id, int32_t* group_offsets,
                          int32_t* members, int32_t* n_groups, int32_t* sel_idx, int32_t* n_sel, int32_t* inv_idx,
                          void* stream);

/* ------------------------------------------------------------------------------------------------
 * Gather of the kept raw variates -- Sec. 3.3 ("Token Reduction"): the dropped variates are removed from the
 * lookback window itself, before the embedding, so that every later layer works on N' variates:
 *   x_sel[b, j, :] = x[b, sel_idx[s(b), j], :]   for j < n_sel[s(b)],   s(b) = 0 (S = 1) or b (S = B).
 * A pure copy, bit-exact.
 *
 * cfg (host)  B, N, L shape of x; S = 1 (one selection for the batch) or B (one per instance).
 * x           [B, N, L] float32, contiguous.
 * sel_idx     [S, N] int32, n_sel [S] int32: vardrop_select's outputs.
 * x_sel       [B, N, L] float32 out (capacity of all N variates); rows 0 .. n_sel-1 of instance b are written, the
 *             rest is untouched.
 * No workspace and no device status: nothing can go wrong on the device that the host did not check.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t B, N, L, S;
} vardrop_gather_cfg;

int vardrop_gather_rows(const float* x, const int32_t* sel_idx, const int32_t* n_sel, const vardrop_gather_cfg* cfg,
                        float* x_sel, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Attention over the kept tokens -- Sec. 3.3 (token reduction: only the selected variate tokens enter
 * self-attention) and Eq. 3, per batch instance b and head h:
 *   Q' = q[b, sel_idx[0..n_sel), h, :] (same for K', V');  O' = softmax(Q' K'^T * sm_scale) V';
 *   lse_i = log sum_j exp(S_ij).
 * bf16 operands, fp32 accumulation and softmax, P rounded to bf16 before the second product.
 *
 * cfg (host)  B, N, H, D (D = 32 or 64; N <= 65536), sm_scale (0 selects 1/sqrt(D)), S (1 or B), and the element strides
 *             sB, sN, sH of q, k and v (the head dimension is contiguous): element (b, n, h, d) of each lies at
 *             b sB + n sN + h sH + d.  All three 0 selects the contiguous layout sH = D, sN = H D, sB = N H D; otherwise
 *             each must be a multiple of 8 elements (16 bytes), sH >= D, sN >= sH, sB >= sN (views of a fused [B, N, 3, H, D]
 *             projection, padded heads or tokens, slices along N).  o, lse, d_o, dq, dk, dv are always contiguous.
 * q, k, v     [B, N, H, D] bf16 with the strides above.
 * sel_idx     [S, N] int32, ascending kept variates (vardrop_select's output: S = 1 for the paper's batch-wise
 *             grouping, S = B when every instance was hashed and sampled on its own), or NULL for the
 *             all-token path (VarDrop off, the inference / "ground" configuration of the paper).
 * n_sel       [S] int32 on the device, number of valid entries of each row of sel_idx; ignored when sel_idx is NULL.
 * o           [B, N, H, D] bf16 out; rows 0..n_sel[s(b)]-1 of instance b hold O', the rest is untouched.
 * lse         [B, H, N] float32 out; entries 0..n_sel[s(b)]-1 valid.
 * ws          scratch of vardrop_attn_workspace_bytes.  After the call it holds what the backward pass of the same
 *             step needs (staged Q', K', V' where the library stages them, a cleared dQ' accumulator):
 *             vardrop_attn_bwd must be given the same, unmodified workspace, once per forward call.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t B, N, H, D;
    float sm_scale;
    int32_t S;      /* selections: 0 or 1 = one shared by all instances (batch-wise grouping), B = one per instance */
    int64_t sB, sN, sH;   /* element strides of q, k, v; all 0 = contiguous */
} vardrop_attn_cfg;

size_t vardrop_attn_workspace_bytes(const vardrop_attn_cfg* cfg);
int vardrop_attn_fwd(const void* q, const void* k, const void* v, const int32_t* sel_idx, const int32_t* n_sel,
                     const vardrop_attn_cfg* cfg, void* o, float* lse, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Backward of the above (the paper applies VarDrop in training only, Sec. 3.1; the derivative of
 * Eq. 3 is the chain rule):
 *   dV' = P^T dO';  dP = dO' V'^T;  Delta_i = sum_d dO'_id O'_id;  dS = P o (dP - Delta);
 *   dQ' = dS K' sm_scale;  dK' = dS^T Q' sm_scale,
 * then scattered: row sel_idx[i] of dq/dk/dv receives row i of dQ'/dK'/dV'; rows of dropped variates
 * are written as zeros, so every row of dq, dk, dv is written exactly once.
 *
 * q, k, v, sel_idx, n_sel, cfg, ws   as given to vardrop_attn_fwd (ws unmodified since).  Exactly one backward call per forward
 *             call on a workspace: a backward call that finds no unconsumed forward pass in `ws` (called twice, or after another
 *             forward call reused the workspace and was already consumed) sets the device status to VARDROP_ERR_INVALID_ARG.
 * o, lse      outputs of vardrop_attn_fwd.
 * d_o         [B, N, H, D] bf16, gradient of o; rows 0..n_sel-1 are read.
 * inv_idx     [S, N] int32 from vardrop_select (NULL when sel_idx is NULL).
 * dq, dk, dv  [B, N, H, D] bf16 out, full variate layout.
 * With more than two key tiles dQ' is accumulated across key tiles by bulk fp32 reduce-adds that land in no fixed
 * order, so the low-order bits of dq may differ from run to run; dK', dV' are bit-reproducible.
 * ---------------------------------------------------------------------------------------------- */
int vardrop_attn_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* d_o,
                     const int32_t* sel_idx, const int32_t* n_sel, const int32_t* inv_idx, const vardrop_attn_cfg* cfg,
                     void* dq, void* dk, void* dv, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Variate redundancy -- Appendix A ("Variate Redundancy in Multivariate Time Series Benchmark Datasets"),
 * Eq. 4: the Pearson correlation coefficient rho(v, w) of two variates of one window, and per variate
 * its largest coefficient with any other variate (the quantity of the appendix's histograms; Sec. 1
 * quotes the share of variates above 0.9).  A constant variate (zero variance; the paper leaves it
 * undefined) correlates 0 with everything.
 *
 * x          [B, N, L] float32, contiguous, device: every instance is treated on its own.
 * max_rho    [B, N] float32, device: max over w != v of rho(v, w); -2 when N = 1.
 * n_above    [B] int32, device: number of variates of the instance with max_rho >= cfg->threshold.
 * ws         scratch (status word + the normalised windows); vardrop_pearson_workspace_bytes.
 * Accuracy: statistics in fp32, the products on the tensor cores with every value held as two bf16
 * terms (16 mantissa bits) and fp32 accumulation: absolute error of a coefficient below 1e-4.
 * Device status: VARDROP_ERR_NONFINITE when a window's variance is not finite.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t B, N, L;
    float threshold;     /* in [-1, 1] */
} vardrop_pearson_cfg;

size_t vardrop_pearson_workspace_bytes(const vardrop_pearson_cfg* cfg);
int vardrop_pearson_max(const float* x, const vardrop_pearson_cfg* cfg, float* max_rho, int32_t* n_above, void* ws,
                        size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VARDROP_H_ */
