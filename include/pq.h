/*
 * pq.h -- C ABI of the B200 (sm_100a) PermuQuant quantized-linear library.
 *
 * The library implements the per-group quantized linear layer of the PermuQuant method:
 *   offline : channel statistics -> joint second-moment sort candidates (Eq. 9, Prop. 3.2)
 *             -> calibration error of every candidate (Eq. 3) -> acceptance rule (Eq. 10)
 *             -> permuted, quantized weight (Eq. 8, P^T W);
 *   runtime : bf16 activations (already in permuted channel order) -> NVFP4 -> W4A4
 *             block-scaled GEMM with fp32 accumulation and bf16 output (Eq. 8, Q(XP) Q(P^T W)).
 *
 * General rules for every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned unless
 *     stated otherwise.  The library allocates nothing and frees nothing (scratch memory is a
 *     caller-provided workspace sized by pq_workspace_bytes).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns without synchronising.  Device scalars (tensor scales, best, accept)
 *     are read and written by kernels, so a whole pipeline can be enqueued back to back.
 *   - Errors are reported by return code only; argument errors are detected on the host before
 *     anything is launched.  Nothing aborts, throws or prints.
 *   - bf16 tensors are row-major [rows, K] with leading dimension `ld` (elements, multiple of 8),
 *     K contiguous.  Activations are X[M,K]; weights are stored transposed, Wt[N,K] (the
 *     nn.Linear convention), so "input channel i of W" is column i of Wt.
 *   - Permutations use the gather convention of App. C: position j of the reordered tensor
 *     reads channel perm[j] of the original one.  Every order handed to the library must hold
 *     values in [0, K): the gather kernels index a staged row with them and do not check (the
 *     orders the library itself produces always do).
 *   - Inputs must be finite.  Tensor scales must lie in [2^-100, 2^100].
 *
 * NVFP4 storage
 *   codes : uint8 [rows, K/2], channel 2j in the low nibble and 2j+1 in the high nibble;
 *           nibble = sign bit (8) | E2M1 magnitude code 0..7 = {0, .5, 1, 1.5, 2, 3, 4, 6}.
 *   sf    : one unsigned E4M3 byte per 16 channels.  PQ_SF_LINEAR: [rows, K/16] row-major.
 *           PQ_SF_TCGEN05: the tensor-core layout -- rows padded to a multiple of 128 and K/16
 *           padded to a multiple of 4; the tensor is tiled in blocks of 128 rows x 4 scale
 *           columns, blocks ordered [row block][column block], 512 bytes each; inside a block the
 *           byte of (row r, column c) sits at (r % 32) * 16 + (r / 32) * 4 + c.
 *           Size in bytes: pq_sf_bytes(rows, K, layout).
 *   ts    : one fp32 tensor scale; value = E2M1 value * E4M3 scale * ts.
 */
#ifndef PQ_H
#define PQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PQ_OK = 0,
    PQ_ERR_NULL = 1,      /* a required pointer is NULL */
    PQ_ERR_SHAPE = 2,     /* a size is out of range or not divisible as required */
    PQ_ERR_ALIGN = 3,     /* a pointer or leading dimension is misaligned */
    PQ_ERR_FORMAT = 4,    /* unsupported pq_format / scale layout */
    PQ_ERR_WORKSPACE = 5, /* workspace missing or too small */
    PQ_ERR_CUDA = 6,      /* the CUDA runtime reported an error (launch, attribute, driver) */
    PQ_ERR_TIMEOUT = 7    /* a bounded device-side wait expired (see pq_device_status) */
} pq_status;

/* Quantization format of the error / fake-quant entry points.
 *   kind 0: NVFP4 (bits and group ignored: 4 bits, groups of 16).
 *   kind 1: symmetric integer, Eq. 1-2, Q = 2^(bits-1) - 1; bits in 2..8, group in {16,32,64,128,256}. */
typedef struct {
    int kind;
    int bits;
    int group;
} pq_format;

enum { PQ_SF_LINEAR = 0, PQ_SF_TCGEN05 = 1 };

/* Which entry point a workspace is for (argument `op` of pq_workspace_bytes). */
enum {
    PQ_OP_CALIB_STATS = 1,
    PQ_OP_SELECT_PERM = 2,
    PQ_OP_GROUP_ERROR = 3,
    PQ_OP_QUANT_WEIGHT = 4,
    PQ_OP_GEMM = 5,
    PQ_OP_OUTPUT_ERROR = 6
};

/* Row blocking of the sums in pq_calib_stats and pq_group_error (part of the arithmetic
 * definition: results depend on it).  A chunk of PQ_CHUNK_ROWS rows is summed in fp32 in row
 * order; the chunk partials of a slab of PQ_SLAB_ROWS rows are added in fp64 in ascending order
 * starting from zero; slab sums are added to the fp64 total in ascending order. */
#define PQ_CHUNK_ROWS 16
#define PQ_SLAB_ROWS 128

const char *pq_status_string(pq_status s);

/* Library version as major*100 + minor. */
int pq_version(void);

/* Text of the last CUDA runtime failure behind a PQ_ERR_CUDA returned to this host thread
 * ("<cuda error name>: <failed call> (line N)"), or "" if there was none.  The pointer stays valid;
 * the text is overwritten by the next failure on the same thread. */
const char *pq_last_error_detail(void);

/* Bytes of scratch the given entry point needs for these sizes (rows = M / T / N as the entry
 * point calls it, P = number of candidate orders, ignored elsewhere).  Never fails; unknown op
 * returns 0.  The workspace must be 256-byte aligned. */
size_t pq_workspace_bytes(int op, int64_t rows, int64_t K, int64_t N, int P);

/* Bytes of the scale tensor of a [rows, K] NVFP4 tensor in the given layout (0 on bad input). */
size_t pq_sf_bytes(int64_t rows, int64_t K, int sf_layout);

/* Channel statistics (second moment of Assumption 3.1 / Sec. 3.3 before the division by the
 * row count, and the absmax used for the tensor scale).  For every channel i:
 *     sumsq[i] += sum_t T[t,i]^2        amax[i] = max(amax[i], |T[t,i]|)
 * Squares are accumulated in fp32 (fused multiply-add, row order) inside a chunk of
 * PQ_CHUNK_ROWS rows; chunks, slabs and the total combine in fp64 as stated at PQ_SLAB_ROWS.
 * Call once per calibration batch (and once on Wt for the weight side);
 * the caller zeroes sumsq / amax before the first batch.
 *   T     : bf16 [rows, K], ld.  K % 8 == 0.
 *   sumsq : fp64 [K] in/out.  amax : fp32 [K] in/out.
 *   ws    : pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0). */
pq_status pq_calib_stats(const void *T, int64_t rows, int64_t K, int64_t ld, double *sumsq,
                         float *amax, void *ws, size_t ws_bytes, void *stream);

/* pq_calib_stats for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a property of the library, not of the method.)
 *
 * Some users of this library run where cudaMalloc is off limits: inside a serving process whose
 * memory pool was sized at start-up and must not grow, in a plugin that is handed tensors but no
 * allocator, or on a path that must never hit the allocator's implicit device synchronisation.
 * They cannot produce the workspace pq_calib_stats asks for.  This entry point computes exactly
 * what pq_calib_stats computes (same kernels, same arithmetic, same results bit for bit) but
 * keeps the per-slab partial sums in a fixed array that is part of the library image:
 * pq_calib_stats_static_max_bytes() bytes (8 MiB) on every GPU that loads the library, for the
 * life of the process.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   - Limit: pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0) must not exceed
 *     pq_calib_stats_static_max_bytes(); larger problems return PQ_ERR_WORKSPACE before anything
 *     is launched (8 MiB covers e.g. 4608 x 12288 or 18432 x 3072; split bigger batches by rows,
 *     the totals accumulate across calls anyway).
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current) and remembers it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, which simply keeps what the last call left
 *     there.  Nothing in it has to start at zero (every partial a call reads it has written
 *     first), but two calls whose kernels overlap on the GPU (different streams, no dependency
 *     between them) race on it: order them.
 *   T, rows, K, ld, sumsq, amax, stream: as for pq_calib_stats. */
pq_status pq_calib_stats_static(const void *T, int64_t rows, int64_t K, int64_t ld, double *sumsq,
                                float *amax, void *stream);
size_t pq_calib_stats_static_max_bytes(void);

/* fp32 tensor scale from per-channel absmax: *ts = max_i amax[i] / 2688 (= 6 * 448), or 1 if
 * the maximum is 0.  ts is a device scalar. */
pq_status pq_tensor_scale(const float *amax, int64_t K, float *ts, void *stream);

/* Sort candidates of the joint second-moment criterion, Eq. 9, for alpha = j/J, j = 0..J.
 * With a_i = sumsq_a[i]/rows_a and w_i = sumsq_w[i]/rows_w the key of channel i is the
 * left-to-right fp64 product of j factors a_i and J-j factors w_i (ordered like
 * (a_i)^alpha (w_i)^(1-alpha)).  perms[j*K + pos] = channel with the pos-th largest key; equal
 * keys keep ascending channel order.  j = J is the activation-only sort of Prop. 3.2, j = 0 the
 * weight-only sort.
 *   K <= 16384, 1 <= J <= 16.  perms : int32 [J+1, K] out.
 *   ws : pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, J + 1) bytes, 256-byte aligned (the sort keys of
 *        every candidate); a NULL or short workspace returns PQ_ERR_WORKSPACE. */
pq_status pq_select_perm(const double *sumsq_a, int64_t rows_a, const double *sumsq_w,
                         int64_t rows_w, int64_t K, int J, int32_t *perms, void *ws,
                         size_t ws_bytes, void *stream);

/* Calibration quantization error, Eq. 3, per candidate order p and group column k:
 *     err[p*(K/g) + k] += sum_t sum_{j<g} (e_j - ehat_j)^2,   e_j = T[t, perms[p*K + k*g + j]]
 * where ehat is the per-group quantize-dequantize of e in format `fmt` (NVFP4 with tensor scale
 * *ts, or Eq. 1-2 integers).  perms == NULL means P == 1 and the original order.  fp32
 * arithmetic: residual by one fused multiply-add, squares summed in runs of 8 channels, runs
 * combined pairwise; rows in chunks and slabs as in pq_calib_stats; fp64 across slabs and calls.
 *   T : bf16 [rows, K], ld.  K % group == 0, K <= 16384, 1 <= P <= 8.
 *   ts: device fp32 scalar (NVFP4 only, else may be NULL).
 *   err : fp64 [P, K/g] in/out (caller zeroes before the first batch).
 *   ws : pq_workspace_bytes(PQ_OP_GROUP_ERROR, rows, K, 0, P). */
pq_status pq_group_error(const void *T, int64_t rows, int64_t K, int64_t ld, pq_format fmt,
                         const float *ts, const int32_t *perms, int P, double *err, void *ws,
                         size_t ws_bytes, void *stream);

/* Output-side calibration error: "the quantization error on the calibration data" of Sec. 3.3
 * (the E of the acceptance rule, Eq. 10) read on the layer's output instead of its inputs.  For
 * every output column n
 *     err[n] += sum_t (Yref[t,n] - Yq[t,n])^2
 * Yref is the unquantized product X W^T in fp32 (any GEMM the caller trusts), Yq the bf16 output
 * of the quantized layer (pq_linear_w4a4 with the candidate order applied to both operands).
 * The difference is one fp32 subtraction; the squares are accumulated like pq_calib_stats: fp32
 * fused multiply-add in row order inside a chunk of PQ_CHUNK_ROWS rows, chunks, slabs and the
 * total in fp64 as stated at PQ_SLAB_ROWS.  sum_n err[n] of the original order and of each
 * candidate are the E[p] of pq_accept (pass them as err_x with Kg = N and a zero err_w).
 *   Yref : device fp32 [rows, N], ld_ref elements between rows (ld_ref % 4 == 0, 16-byte aligned).
 *   Yq   : device bf16 [rows, N], ld_q (ld_q % 8 == 0, 16-byte aligned).  N % 8 == 0.
 *   err  : device fp64 [N] in/out (the caller zeroes it before the first batch).
 *   ws   : pq_workspace_bytes(PQ_OP_OUTPUT_ERROR, rows, N, 0, 0)  (N in the place of K). */
pq_status pq_output_error(const float *Yref, int64_t ld_ref, const void *Yq, int64_t ld_q,
                          int64_t rows, int64_t N, double *err, void *ws, size_t ws_bytes,
                          void *stream);

/* The absmax criterion of the reordering ablation (Tab. 2(a)) as one more candidate order:
 * perm[pos] = channel with the pos-th largest absmax, equal values in ascending channel order.
 * The row can be appended to the candidate table that pq_group_error / pq_accept evaluate.
 *   amax : device fp32 [K] (as accumulated by pq_calib_stats).  K <= 16384.
 *   perm : device int32 [K] out.  ws : pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, 1). */
pq_status pq_order_by_absmax(const float *amax, int64_t K, int32_t *perm, void *ws, size_t ws_bytes,
                             void *stream);

/* Per-channel first moments, the other ingredient of the variance criterion of the reordering ablation
 * (Tab. 2(a)):  sum[i] += sum_t T[t,i], blocked exactly like the squares of pq_calib_stats (fp32
 * additions in row order inside a chunk of PQ_CHUNK_ROWS rows; chunks, slabs and the total in fp64).
 *   T : bf16 [rows, K], ld.  sum : fp64 [K] in/out (the caller zeroes it before the first batch).
 *   ws : pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0). */
pq_status pq_calib_sum(const void *T, int64_t rows, int64_t K, int64_t ld, double *sum, void *ws,
                       size_t ws_bytes, void *stream);

/* The variance criterion of Tab. 2(a) as one more candidate order: channels by descending
 * var_i = sumsq[i] / rows - (sum[i] / rows)^2 in fp64 (two divisions, one multiplication, one
 * subtraction; may come out slightly negative for a constant channel), equal values in ascending
 * channel order.
 *   sum, sumsq : device fp64 [K] as accumulated by pq_calib_sum / pq_calib_stats over `rows` rows.
 *   perm : device int32 [K] out.  K <= 16384.  ws : pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, 1). */
pq_status pq_order_by_variance(const double *sum, const double *sumsq, int64_t rows, int64_t K,
                               int32_t *perm, void *ws, size_t ws_bytes, void *stream);

/* The "round-robin" order of Tab. 2(a).  The paper names it without defining it; this library's
 * reading: the channels sorted by descending second moment (equal values in ascending channel order)
 * are dealt to the K / group groups one at a time in turn, so every group receives channels of every
 * magnitude: with G = K / group, perm[(r % G) * group + r / G] = channel of sorted rank r.
 *   sumsq : device fp64 [K].  K % group == 0, K <= 16384.  perm, ws : as for pq_order_by_variance. */
pq_status pq_order_round_robin(const double *sumsq, int64_t K, int group, int32_t *perm, void *ws,
                               size_t ws_bytes, void *stream);

/* Relative-error weights for pq_accept: lambda[0] = 1 / sum_i sumsq_a[i], lambda[1] =
 * 1 / sum_i sumsq_w[i] (sequential fp64 sums in channel order).  lambda: device fp64 [2]. */
pq_status pq_error_weights(const double *sumsq_a, const double *sumsq_w, int64_t K, double *lambda,
                           void *stream);

/* Candidate selection and the acceptance rule, Eq. 10.  Row 0 of err_x / err_w is the original
 * order, rows 1..P the candidates.
 *     E[p] = lambda[0] * sum_k err_x[p,k] + lambda[1] * sum_k err_w[p,k]      (fp64, in k order)
 *     best = argmin_{p in 1..P} E[p] (first on ties);   accept = (E[0] - E[best] > tau * E[0]).
 * tau is a fraction (the paper's 2.5 means 0.025); tau = 0 is the paper's default.
 *   lambda : device fp64 [2], or NULL for (1, 1).  best, accept : device int32 scalars out.
 *   E : device fp64 [P+1] out, or NULL. */
pq_status pq_accept(const double *err_x, const double *err_w, const double *lambda, int P,
                    int64_t Kg, double tau, int32_t *best, int32_t *accept, double *E,
                    void *stream);

/* Offline weight path of Eq. 8: gather the input channels by perm (P^T W), compute the weight
 * tensor scale *ts_w = max|Wt| / 2688 and quantize to NVFP4.
 *   Wt : bf16 [N, K], ld.  K % 16 == 0 (K % 64 == 0 for PQ_SF_TCGEN05), K <= 16384.
 *   perm : int32 [K] or NULL (original order).
 *   perm_select : device int32 [2] = {best, accept} as written by pq_accept, or NULL.  When
 *       given, `perm` must be the [J+1, K] candidate table and the row best-1 is used if
 *       accept != 0, the original order otherwise -- so the decision never visits the host.
 *   codes : uint8 [N, K/2] out.  sf : pq_sf_bytes(N, K, sf_layout) bytes out.  ts_w : device out.
 *   ws : pq_workspace_bytes(PQ_OP_QUANT_WEIGHT, N, K, 0, 0). */
pq_status pq_quant_weight(const void *Wt, int64_t N, int64_t K, int64_t ld, const int32_t *perm,
                          const int32_t *perm_select, uint8_t *codes, uint8_t *sf, int sf_layout,
                          float *ts_w, void *ws, size_t ws_bytes, void *stream);

/* Runtime activation quantizer (dynamic per-group scales, static tensor scale *ts_x from
 * calibration).  Per row and 16-channel group: absmax -> E4M3(absmax / (6 ts)) -> 16 E2M1 codes
 * of x / (scale * ts), round to nearest even, saturating.  Channels arrive already permuted.
 *   X : bf16 [M, K], ld.  K % 16 == 0 (K % 64 == 0 for PQ_SF_TCGEN05).
 *   codes : uint8 [M, K/2] out.  sf : pq_sf_bytes(M, K, sf_layout) bytes out (padding bytes of
 *   the tensor-core layout are written as 0). */
pq_status pq_quant_act_nvfp4(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x,
                             uint8_t *codes, uint8_t *sf, int sf_layout, void *stream);

/* The same quantizer with a channel order applied on the way in (codes and scales of X P): the
 * calibration-time form, used to evaluate a candidate order on the layer output (pq_output_error)
 * before any producer has been rewritten to emit permuted activations.  Rows are staged in shared
 * memory and gathered from there (rows of up to 6400 channels four per warp, sharing indices and
 * gathers, when perm is 16-byte aligned; otherwise one block per row; same results);
 * perm == NULL is pq_quant_act_nvfp4.
 *   perm : device int32 [K], values in [0, K) (not checked).  K <= 16384.  Other arguments as for
 *   pq_quant_act_nvfp4. */
pq_status pq_quant_act_nvfp4_perm(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                  const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout,
                                  void *stream);

/* W4A4 block-scaled GEMM, right-hand side of Eq. 8:
 *     Y[m,n] = bf16( ts_x*ts_w * sum_kb sfx[m,kb]*sfw[n,kb] * sum_{j<16} qx[m,16kb+j]*qw[n,16kb+j] )
 * on the tcgen05 tensor cores (E2M1 operands, UE4M3 block scales in tensor memory, fp32
 * accumulation).  Both scale tensors must be in PQ_SF_TCGEN05 layout.
 *   xq [M,K/2], wq [N,K/2] codes;  K % 64 == 0, K >= 64;  N % 8 == 0;  M, N >= 1.
 *   Y : bf16 [M, N], ldy (multiple of 8).
 *   ws : pq_workspace_bytes(PQ_OP_GEMM, M, K, N, 0) bytes holding the device status word.  The
 *        caller zeroes it once (cudaMemset) before the first GEMM that uses it; the kernel only
 *        ever writes a non-zero code there.
 * Every device-side wait is bounded; if one expires the kernel records PQ_ERR_TIMEOUT in the
 * status word (read it with pq_device_status) and returns.
 * Launch: the kernel (like the activation quantizer) is launched as a programmatic dependent of
 * the kernel before it in `stream`: its set-up may overlap that kernel's last thread blocks, and
 * it waits for that kernel to complete before it reads or writes global memory, so what the
 * caller observes is ordinary stream order. */
pq_status pq_gemm_w4a4(const uint8_t *xq, const uint8_t *sfx, const float *ts_x, const uint8_t *wq,
                       const uint8_t *sfw, const float *ts_w, int64_t M, int64_t N, int64_t K,
                       void *Y, int64_t ldy, void *ws, size_t ws_bytes, void *stream);

/* The timed runtime path: pq_quant_act_nvfp4 (tensor-core scale layout) followed by
 * pq_gemm_w4a4.  xq / sfx are caller-provided intermediates of the sizes above. */
pq_status pq_linear_w4a4(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x,
                         uint8_t *xq, uint8_t *sfx, const uint8_t *wq, const uint8_t *sfw,
                         const float *ts_w, int64_t N, void *Y, int64_t ldy, void *ws,
                         size_t ws_bytes, void *stream);

/* The runtime path of Eq. 8 for n independent batches through one layer (image batches, micro-
 * batches): batch i is quantized into intermediates set i % n_sets and multiplied into Y[i].  The
 * quantizer of a batch runs on one internal stream, the GEMMs on another, ordered by events, so the
 * quantization of the following batches overlaps the GEMM of the current one (the quantizer's
 * small thread blocks fit beside the GEMM's one CTA per SM), and every second GEMM is launched as a
 * programmatic dependent of the one before it.  Results are those of n calls of pq_linear_w4a4.
 *   X, Y   : HOST arrays of n device pointers (bf16 [M, K] ld, bf16 [M, N] ldy); read during the call.
 *   xq, sfx: HOST arrays of n_sets device pointers, 2 <= n_sets <= 8, each as in pq_linear_w4a4;
 *            with more sets the quantizer may run further ahead.
 *   ws     : as for pq_gemm_w4a4 (shared by all batches).
 * Ordering: all work is ordered after what `stream` already holds and before what is enqueued in
 * `stream` afterwards; the call may be captured in a CUDA graph.  The first call on a device creates
 * two streams and a few events (host objects, no device memory) that live until the process exits;
 * calls on the same device from several host threads must be serialised by the caller. */
pq_status pq_linear_w4a4_batched(int n, const void *const *X, int64_t M, int64_t K, int64_t ld,
                                 const float *ts_x, uint8_t *const *xq, uint8_t *const *sfx,
                                 int n_sets, const uint8_t *wq, const uint8_t *sfw,
                                 const float *ts_w, int64_t N, void *const *Y, int64_t ldy, void *ws,
                                 size_t ws_bytes, void *stream);

/* The same runtime path for a caller whose tensors live in HOST memory (the end-to-end
 * measurement): copies X_host -> X_dev on `stream`, runs pq_linear_w4a4, copies Y_dev -> Y_host,
 * all asynchronously on `stream` (the caller synchronises the stream before reading Y_host).
 *   X_host : bf16 [M, K] contiguous HOST memory (pinned for the copy to be asynchronous).
 *   Y_host : bf16 [M, N] contiguous HOST memory, out.
 *   X_dev  : bf16 [M, K] contiguous device staging buffer;  Y_dev : bf16 [M, N] contiguous device
 *            staging buffer;  everything else as in pq_linear_w4a4.
 * Returns PQ_ERR_CUDA if a copy cannot be enqueued. */
pq_status pq_linear_w4a4_host(const void *X_host, int64_t M, int64_t K, const float *ts_x,
                              void *X_dev, uint8_t *xq, uint8_t *sfx, const uint8_t *wq,
                              const uint8_t *sfw, const float *ts_w, int64_t N, void *Y_dev,
                              void *Y_host, void *ws, size_t ws_bytes, void *stream);

/* pq_linear_w4a4_host for n independent batches: uploads, the runtime path and downloads run on
 * three internal streams ordered by events, so the copies of neighbouring batches overlap each
 * other (PCIe is full duplex) and the kernels.  Batch i uses staging buffers X_dev[i % n_sets] and
 * Y_dev[i % n_sets]; one set of intermediates xq / sfx serves all batches (the kernels of different
 * batches run in order).  Results are those of n calls of pq_linear_w4a4_host.
 *   X_host, Y_host : HOST arrays of n HOST pointers (bf16 [M, K] / [M, N] contiguous, pinned).
 *   X_dev, Y_dev   : HOST arrays of n_sets device staging buffers, 2 <= n_sets <= 8.
 * Ordering and the internal streams as for pq_linear_w4a4_batched; the caller synchronises
 * `stream` before reading the Y_host buffers. */
pq_status pq_linear_w4a4_host_batched(int n, const void *const *X_host, int64_t M, int64_t K,
                                      const float *ts_x, void *const *X_dev, void *const *Y_dev,
                                      int n_sets, uint8_t *xq, uint8_t *sfx, const uint8_t *wq,
                                      const uint8_t *sfw, const float *ts_w, int64_t N,
                                      void *const *Y_host, void *ws, size_t ws_bytes, void *stream);

/* The producer in front of a quantized linear layer, fused (App. C: the channel reordering absorbed
 * into the normalization kernel; here the NVFP4 quantizer of Eq. 8 is attached as well, so the
 * normalized activations are never written in bf16).  Per token row x of H and output position j
 * reading channel c = perm[j] (perm == NULL: c = j), in fp32:
 *   PQ_NORM_RMS  : out_j = (x_c * inv) * a_j,                    inv = 1 / sqrt(mean_i(x_i^2) + eps)
 *   PQ_NORM_ADALN: out_j = fma((x_c - mu) * inv, 1 + a_j, b_j),  inv = 1 / sqrt(mean_i((x_i - mu)^2) + eps)
 * a (RMSNorm weight or modulation scale) and b (modulation shift) are indexed by OUTPUT position: they
 * arrive reordered, the (1 + Ps) and Pb of App. C; one vector each per call; IEEE division and square
 * root.  The row sums run over the ORIGINAL channel order (so they do not depend on the permutation):
 * element i is added by lane (i / 8) % 32 in ascending i, the 32 lane sums meet in a butterfly of strides
 * 16, 8, 4, 2, 1.  out is quantized in groups of 16 exactly as pq_quant_act_nvfp4 quantizes a bf16
 * tensor holding out, except that out keeps its fp32 precision.
 *   H : bf16 [M, K], ld.  K % 16 == 0 (K % 64 == 0 for PQ_SF_TCGEN05), K <= 32768.
 *   a, b : device fp32 [K], 16-byte aligned (b may be NULL for PQ_NORM_RMS).  perm : int32 [K] or NULL.
 *   codes, sf : as pq_quant_act_nvfp4.  y_out : bf16 [M, K] contiguous or NULL; receives bf16(out),
 *   the tensor the unfused kernel of App. C writes (for calibration or for checking). */
enum { PQ_NORM_RMS = 0, PQ_NORM_ADALN = 1 };
pq_status pq_norm_quant_nvfp4(const void *H, int64_t M, int64_t K, int64_t ld, int kind, const float *a,
                              const float *b, float eps, const int32_t *perm, const float *ts_x,
                              uint8_t *codes, uint8_t *sf, int sf_layout, void *y_out, void *stream);

/* PermuQuant-H producer (App. D: reordering in the Hadamard-transformed basis, x H P): every row of X
 * goes through the Hadamard transform, the transformed channels are read in the order `perm` (the
 * transform itself is unchanged, only the order in which its outputs are consumed), and the result is
 * quantized to NVFP4 exactly as pq_quant_act_nvfp4 quantizes a tensor, except that the quantizer sees
 * the fp32 values.  The same call transforms weight rows (Wt H, written to y_out in bf16 and then fed
 * to pq_calib_stats / pq_group_error / pq_quant_weight), since (x H)(Wt H)^T = x Wt^T.
 *   Transform: K = m * 2^n with m = 1 or m = 12 (2^n >= 8); y = x (H_m (x) H_{2^n}) / sqrt(K), i.e. with
 *   channel i = a * 2^n + b the matrix entry is H_m[a][a'] * (-1)^popcount(b & b'); H_12 = I + S is Paley's
 *   matrix for q = 11: S[0][j] = 1, S[i][0] = -1, S[i][j] = chi(i - j) for i, j >= 1, chi the quadratic
 *   character modulo 11.  (The paper names the transform only; matrix, order and scaling are this
 *   library's reading.)  fp32 arithmetic in this order: the 12 segments combined first, terms added one
 *   by one in ascending segment; then inside every segment the butterflies (x[i], x[i+h]) <-
 *   (x[i] + x[i+h], x[i] - x[i+h]) with strides h = 1, 2, 4, ...; then one multiplication by
 *   fl(1 / sqrt(K)).  Other widths return PQ_ERR_SHAPE.
 *   X : bf16 [M, K], ld.  K % 16 == 0, K <= 16384 (K % 64 == 0 for codes in PQ_SF_TCGEN05).
 *   perm : device int32 [K] or NULL (transformed order).  ts_x : device fp32 scalar (needed with codes).
 *   codes, sf : as pq_quant_act_nvfp4, or both NULL to transform only (then y_out is required).
 *   y_out : bf16 [M, K] contiguous or NULL; receives bf16 of the reordered transformed rows. */
pq_status pq_hadamard_quant_nvfp4(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                  const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout,
                                  void *y_out, void *stream);

/* Integer fake-quant of Eq. 1-2 (quantize, dequantize, round to bf16), optional gather.
 *   T : bf16 [rows, K], ld.  out : bf16 [rows, K], ldo.  perm : int32 [K] or NULL.
 *   fmt.kind must be 1; fmt.group in {16, 32, 64, 128, 256}; K % fmt.group == 0; K <= 16384 when perm != NULL. */
pq_status pq_fakequant_int(const void *T, int64_t rows, int64_t K, int64_t ld, pq_format fmt,
                           const int32_t *perm, void *out, int64_t ldo, void *stream);

/* Rearrange scale bytes from the tensor-core layout into [rows, K/16] row-major (for tests and
 * debugging). */
pq_status pq_sf_to_linear(const uint8_t *sf_tc, int64_t rows, int64_t K, uint8_t *sf_linear,
                          void *stream);

/* Synchronises `stream`, then reads the status word a GEMM workspace holds: PQ_OK, or
 * PQ_ERR_TIMEOUT if a bounded wait inside the kernel expired, PQ_ERR_CUDA if the stream reports
 * an asynchronous error.  HOST call; `ws` is the device workspace passed to pq_gemm_w4a4. */
pq_status pq_device_status(const void *ws, void *stream);

/* Exercises the expiry path of the GEMM's bounded device-side waits without a hang or a fault (the
 * failure-detection path of the library; the paper has no counterpart).  One warp waits, with the same
 * helper every role of the GEMM kernel uses, on a barrier that nobody arrives at; after `limit_cycles`
 * SM clock cycles the wait gives up, raises the kernel's abort flag, writes PQ_ERR_TIMEOUT into the
 * status word at `ws` and the kernel returns normally: the context stays usable.
 *   ws           : a GEMM workspace (device); afterwards pq_device_status(ws) reports PQ_ERR_TIMEOUT
 *                  until the caller zeroes the word again.
 *   limit_cycles : 1 .. 1e8 (a fraction of a second at most).
 *   observed     : device int32 [2] out: {result of the wait (0 = gave up), abort flag}. */
pq_status pq_selftest_wait_expiry(void *ws, size_t ws_bytes, long long limit_cycles, int *observed,
                                  void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PQ_H */
