/*
 * attn.h - C ABI of the BF16 flash-attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes causal or full softmax attention, forward and
 * backward, with the rounding behaviour analysed in "Why Low-Precision
 * Transformer Training Fails: An Analysis on Flash Attention"
 * (arXiv 2510.04212):
 *
 *   mode 0  standard flash attention, Algorithm 1 (forward) and Algorithm 2
 *           (backward): the unnormalised probabilities P-bar = exp(S - m) are
 *           BF16, so every key that attains the row maximum has P-bar == 1;
 *           P-bar V accumulates in FP32 and the unnormalised output is rounded
 *           to BF16 (the "(.)_lp" product of Sec. 3.3.2) before the division
 *           by the row sum.
 *   mode 1  stabilised flash attention, Algorithm 3 / Sec. 4: inside each key
 *           tile, a row whose maximum is attained by more than one entry
 *           (within eps) uses beta*r_m (r_m > 0) or 0 (r_m < 0) as its maximum,
 *           so that no P-bar equals 1.  The backward pass is unchanged.
 *
 * Conventions common to every entry point
 * ---------------------------------------
 *  - Every pointer is a DEVICE pointer unless stated otherwise.  The caller
 *    owns every buffer; the library allocates no device memory, frees
 *    nothing, and never synchronises: work is enqueued on `stream`
 *    (a cudaStream_t passed as void*; NULL is the default stream).
 *    Kernels are launched with programmatic stream serialization: a kernel's
 *    blocks may be set up while the previous kernel of the stream drains, but
 *    touch no global memory before that kernel has completed, so stream order
 *    holds for every buffer as with an ordinary launch.
 *  - Tensors q, k, v, o, dO, dq, dk, dv: BF16 (16-bit storage), row-major
 *    contiguous [B][H][N][d], base address 16-byte aligned.
 *    lse and delta: FP32, [B][H][N].
 *  - Supported shapes: d in {64, 128}; N a multiple of 128, N >= 128;
 *    B, H >= 1; B*H*N < 2^31.  Self-attention only (same N for queries and
 *    keys), no dropout, no bias.
 *  - scale is the softmax scale alpha (Sec. 2.2), finite and > 0.
 *  - Return value: ATTN_OK (0) or a negative ATTN_ERR_* code.  Nothing is
 *    enqueued when an error is returned for bad arguments.  The library
 *    never aborts, throws or prints.  There is no CPU fallback and no other
 *    GPU architecture: on a device that is not compute capability 10.x
 *    every compute entry point returns ATTN_ERR_DEVICE.
 *  - Device-side waits are bounded.  If one runs out (a pipeline fault), the
 *    kernel stops early and records it; attn_last_device_status() reports it
 *    after the caller has synchronised the stream.
 *  - Host threads: every entry point may be called from several host threads
 *    at once, each with its own current device and stream; what the library
 *    caches on the host is per device and published atomically.  The
 *    parameters set by attn_set_mitigation() and attn_set_guard_max_shift()
 *    are process-wide: a compute call uses the values in force when it is
 *    made.  attn_bwd_static() shares one scratch array per device (see there).
 */
#ifndef ATTN_H_
#define ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ATTN_OK               0
#define ATTN_ERR_NULL        -1   /* a required pointer is NULL */
#define ATTN_ERR_SHAPE       -2   /* unsupported B, H, N or d */
#define ATTN_ERR_MODE        -3   /* mode has a bit this entry point does not know */
#define ATTN_ERR_PARAM       -4   /* scale, beta or eps out of range */
#define ATTN_ERR_WORKSPACE   -5   /* workspace missing, misaligned or too small */
#define ATTN_ERR_CUDA        -6   /* a CUDA runtime/driver call or a launch failed */
#define ATTN_ERR_TIMEOUT     -7   /* a bounded device-side wait ran out */
#define ATTN_ERR_DEVICE      -8   /* current device is not sm_100 */
#define ATTN_ERR_ALIGN       -9   /* a tensor base address is not 16-byte aligned */

#define ATTN_MODE_STANDARD    0
#define ATTN_MODE_STABILISED  1
/*
 * Diagnostic variants, OR-ed into `mode`.  They reproduce the paper's isolating experiments; the defaults
 * (flags clear) are the arithmetic the paper analyses.
 *   ATTN_MODE_FLAG_SINGLE_ROUNDING (forward)  the unnormalised output O-bar stays FP32 and only
 *        O = bf16(O-bar / l) is rounded: the rounding of O-bar that Sec. 3.3.2 identifies as the source of
 *        the biased error is left out.  Accepted and ignored by the backward entry points.
 *   ATTN_MODE_FLAG_DELTA_GIVEN (backward)     `delta` is an INPUT: the caller supplies rowsum(dO o O), for
 *        instance computed from a high-precision O (the delta_hp of Sec. 3.2, Eq. 9 discussion), and the
 *        library does not compute it.  Rejected by the forward entry points.
 */
#define ATTN_MODE_FLAG_SINGLE_ROUNDING  2
#define ATTN_MODE_FLAG_DELTA_GIVEN      4
/*
 * Guarded tie rule (forward, only together with ATTN_MODE_STABILISED; otherwise ATTN_ERR_MODE).  An extension, NOT
 * the paper's Algorithm 3, and never the default.  Algorithm 3 looks at one key tile at a time and sets
 * m' = beta * r_m (r_m > 0) or 0 (r_m < 0) when the tile's row maximum r_m is repeated.  Two consequences the paper
 * notes or implies (Sec. 4, App. C): a maximum repeated across two tiles is not seen, and for large |r_m| the shift
 * makes every exponential of the row underflow, so that l = 0 and O is not finite (e.g. a repeated r_m = 110 with
 * beta = 2).  With this flag, per key tile:
 *   repeated = (r_s > 1)  or  |r_m - (largest r_m of the earlier tiles of the row)| <= eps
 *   m'       = the paper's value, unless that lies more than `max_shift` above r_m; then m' = r_m + max_shift
 * so the tile's own maximum keeps an exponent >= -max_shift and l >= exp(-max_shift) > 0.  Where no shift exceeds
 * max_shift and no maximum repeats across tiles the results equal mode 1 bit for bit.
 * max_shift: process-wide, default ATTN_GUARD_DEFAULT_MAX_SHIFT, see attn_set_guard_max_shift.
 */
#define ATTN_MODE_FLAG_GUARDED          8
#define ATTN_GUARD_DEFAULT_MAX_SHIFT    16.0f

/*
 * Forward pass: Algorithm 1 (mode 0) or Algorithm 3 (mode 1).
 *   in : q, k, v      BF16 [B][H][N][d]
 *   out: o            BF16 [B][H][N][d]   O = softmax(scale Q K^T) V
 *        lse          FP32 [B][H][N]      L = m + log(l), the row log-sum-exp
 *   causal != 0 masks keys after the query (key index > query index).
 * Key/query tile sizes are those of attn_get_tiles(); in mode 1 the tie rule
 * is applied per key tile (Algorithm 3 applies it to S_i^(j)), so the key tile
 * size is part of the numerical contract.  beta and eps come from
 * attn_set_mitigation().
 */
int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int H, int N, int d, int causal, float scale, int mode,
             void* stream);

/*
 * attn_fwd plus the paper's leading indicator of the failure (Sec. 3.3.2: rows in which several entries
 * of P-bar are exactly 1):
 *   out: ones   int32 [B][H][N]   per query row, the number of P-bar entries, over all key tiles, that are
 *               exactly 1 after the BF16 rounding (overwritten).
 * Same arguments, checks and results for o and lse as attn_fwd; a separate kernel instantiation, so
 * attn_fwd itself does not pay for the counting.
 */
int attn_fwd_count_ones(const void* q, const void* k, const void* v, void* o, float* lse, int* ones,
                        int B, int H, int N, int d, int causal, float scale, int mode,
                        void* stream);

/*
 * attn_fwd plus the output in FP32, for the paper's "O kept in FP32" experiments (Sec. 3.2: the failure goes away
 * when delta is formed from an O that was not rounded to BF16):
 *   out: o_f32   FP32 [B][H][N][d], device memory, 16-byte aligned, overwritten: O-bar / l, where O-bar is the FP32
 *                accumulator of Algorithm 1 / 3 before either of its BF16 roundings and the division is IEEE
 *                round-to-nearest.  P-bar is still the BF16-rounded matrix (that rounding is the method's).
 * o and lse are written as by attn_fwd, bit for bit.  A separate kernel instantiation (that of
 * attn_fwd_count_ones), so attn_fwd does not pay for it.  Errors as attn_fwd; o_f32 == NULL: ATTN_ERR_NULL.
 * attn_bwd_delta_f32 turns o_f32 into the delta that attn_bwd takes with ATTN_MODE_FLAG_DELTA_GIVEN.
 */
int attn_fwd_o_f32(const void* q, const void* k, const void* v, void* o, float* lse, float* o_f32,
                   int B, int H, int N, int d, int causal, float scale, int mode,
                   void* stream);

/*
 * delta = rowsum(dO o O) with O in FP32 (Algorithm 2's first line, on the output of attn_fwd_o_f32; Sec. 3.2):
 *   in : o_f32  FP32 [B][H][N][d];  dO  BF16 [B][H][N][d]        (device memory, 16-byte aligned)
 *   out: delta  FP32 [B][H][N]      products and sums in FP32, one rounding per fused multiply-add
 * Errors: ATTN_ERR_NULL, ATTN_ERR_SHAPE, ATTN_ERR_ALIGN, ATTN_ERR_DEVICE, ATTN_ERR_CUDA.
 */
int attn_bwd_delta_f32(const float* o_f32, const void* dO, float* delta, int B, int H, int N, int d, void* stream);

/*
 * attn_fwd_count_ones with P-bar rounded to an 8-bit floating-point format instead of BF16: a diagnostic for the
 * question the paper leaves open (Sec. 5 names FP8 training as future work), not part of its method.
 *   pbar_format  ATTN_PBAR_BF16 (0): exactly attn_fwd_count_ones;
 *                ATTN_PBAR_E4M3 (1): 4 exponent bits (bias 7), 3 fraction bits, subnormals down to 2^-9;
 *                ATTN_PBAR_E5M2 (2): 5 exponent bits (bias 15), 2 fraction bits, subnormals down to 2^-16.
 * Each unrounded probability exp(S - m) is rounded to nearest-even in that format; the rounded value (exactly
 * representable in BF16) is what the tensor core multiplies with V, what the row sum l accumulates and what
 * `ones` counts.  Everything else (FP32 scores and statistics, O-bar rounding, modes and flags) is as in
 * attn_fwd.  Only the numerics of an FP8 P-bar are reproduced: the product still runs on the BF16 tensor path.
 * Errors as attn_fwd_count_ones; an unknown pbar_format returns ATTN_ERR_MODE.
 */
#define ATTN_PBAR_BF16 0
#define ATTN_PBAR_E4M3 1
#define ATTN_PBAR_E5M2 2
int attn_fwd_pbar_format(const void* q, const void* k, const void* v, void* o, float* lse, int* ones,
                         int B, int H, int N, int d, int causal, float scale, int mode, int pbar_format,
                         void* stream);

/*
 * The P-bar V product of the forward pass on the 8-bit tensor path: the setting the paper names as future work
 * (Sec. 5: FP8 training), built so that its numerics and its speed can be measured; not part of the paper's method.
 *
 * attn_quantize_v_e4m3:  v_t[b][h][c][n] = e4m3(v[b][h][n][c] * v_scale)   (round to nearest even, saturating at 448)
 *   in : v         BF16 [B][H][N][d];   v_scale > 0 (ATTN_ERR_PARAM otherwise)
 *   out: v_t_e4m3  E4M3 [B][H][d][N]    one byte per element, transposed, 16-byte aligned
 * attn_fwd_fp8pv:  attn_fwd with P-bar = e4m3(exp(S - m)) (instead of BF16) and V taken from v_t_e4m3; the product
 *   O-bar += P-bar V runs as tcgen05.mma kind::f8f6f4 with FP32 accumulation (the products of two E4M3 values are
 *   exact in FP32).  S = Q K^T stays BF16 x BF16, all statistics stay FP32, l sums the rounded P-bar, and
 *   O = bf16(bf16(v_descale * O-bar) / l): pass v_descale = 1 / v_scale.  mode: 0 or ATTN_MODE_STABILISED only
 *   (other bits: ATTN_ERR_MODE).  The result equals attn_fwd_pbar_format(..., ATTN_PBAR_E4M3) run on the
 *   dequantised V, up to the order of the FP32 sums.  Other arguments, checks and errors as attn_fwd.
 */
int attn_quantize_v_e4m3(const void* v, void* v_t_e4m3, int B, int H, int N, int d, float v_scale, void* stream);
int attn_fwd_fp8pv(const void* q, const void* k, const void* v_t_e4m3, void* o, float* lse,
                   int B, int H, int N, int d, int causal, float scale, int mode, float v_descale, void* stream);

/*
 * delta = rowsum(dO o O), the preprocessing step of Algorithm 2 (Sec. 2.2).
 *   in : o, dO   BF16 [B][H][N][d]
 *   out: delta   FP32 [B][H][N]
 */
int attn_bwd_preprocess(const void* o, const void* dO, float* delta,
                        int B, int H, int N, int d, void* stream);

/*
 * delta = rowsum(dP o P) with dP = dO V^T and P = exp(scale Q K^T - L): the alternative formulation of Sec. 3.2,
 * mathematically the same number as rowsum(dO o O) but computed without O (the paper uses it to show that the
 * error of the BF16 O is what breaks training).  S and dP are FP32 sums of the exact BF16 products, P is not
 * rounded, the row sum is FP32.  A diagnostic, not a step of the hot path, and deliberately slow: it runs the two
 * contractions on the ordinary FP32 pipes so that every product is exact and every sum a plain FP32 sum in a fixed
 * order (1.45 ms on B=16, H=12, N=1024, d=64 causal, six times the forward + backward step).  Pass its result to
 * attn_bwd with ATTN_MODE_FLAG_DELTA_GIVEN.  The cheaper route to a delta free of the rounding of O is
 * attn_fwd_o_f32 followed by attn_bwd_delta_f32.
 *   in : q, k, v, dO  BF16 [B][H][N][d];  lse FP32 [B][H][N] as written by attn_fwd
 *   out: delta        FP32 [B][H][N]
 * Same shape, scale, alignment and device checks and error codes as attn_fwd; asynchronous on `stream`.
 */
int attn_bwd_delta_dp(const void* q, const void* k, const void* v, const void* dO, const float* lse, float* delta,
                      int B, int H, int N, int d, int causal, float scale, void* stream);

/*
 * Backward pass, Algorithm 2: computes delta (as attn_bwd_preprocess), then
 * dQ, dK, dV.  `mode` is validated but does not change the arithmetic
 * (Sec. 4: the stabilised forward leaves the backward pass unaltered).
 *   in : q, k, v, o, dO   BF16 [B][H][N][d];  lse FP32 [B][H][N] from attn_fwd
 *   out: dq, dk, dv       BF16 [B][H][N][d]  (overwritten, not accumulated into)
 *        delta            FP32 [B][H][N]     (overwritten)
 *   scratch: workspace, at least attn_bwd_workspace_bytes(B,H,N,d) bytes,
 *        256-byte aligned.  It holds the FP32 dQ accumulator, in a layout
 *        that is private to the library; the library clears it itself.  Two attn_bwd calls that may overlap on the GPU
 *        must not share a workspace.
 */
int attn_bwd(const void* q, const void* k, const void* v, const void* o,
             const void* dO, const float* lse,
             void* dq, void* dk, void* dv,
             float* delta, void* workspace, size_t workspace_bytes,
             int B, int H, int N, int d, int causal, float scale, int mode,
             void* stream);

/*
 * One stage of attn_bwd, same arguments and checks.  attn_bwd is stages 1, 2, 3 in order on
 * `stream`; running them as three calls gives the same result and lets a caller put its own
 * CUDA events between the kernels (the benchmark times each kernel this way).
 *   ATTN_BWD_STAGE_PREPROCESS  delta = rowsum(dO o O) and clearing of the workspace; it also leaves, in the first
 *                              1040 bytes of every 128-row tile of the dQ OUTPUT buffer, scratch that MAIN reads
 *                              (an arrival counter and the tile's per-row -L*log2(e) and -delta as FP32)
 *   ATTN_BWD_STAGE_MAIN        the loops of Algorithm 2: dK, dV, FP32 dQ accumulated in the workspace.  At both head
 *                              widths it must follow a PREPROCESS with the same call arguments, with nothing
 *                              else writing dq, the workspace, lse or delta in between.
 *   ATTN_BWD_STAGE_FINALIZE    dQ = bf16(scale * accumulator), overwriting the scratch; launches nothing for
 *                              d = 64, where the main kernel finishes every dQ tile itself (the CTA whose
 *                              contribution completes a tile converts it)
 *   ATTN_BWD_STAGE_ALL         all three (what attn_bwd does)
 * Any other stage value returns ATTN_ERR_PARAM.
 */
#define ATTN_BWD_STAGE_ALL         0
#define ATTN_BWD_STAGE_PREPROCESS  1
#define ATTN_BWD_STAGE_MAIN        2
#define ATTN_BWD_STAGE_FINALIZE    3
int attn_bwd_stage(int stage,
                   const void* q, const void* k, const void* v, const void* o,
                   const void* dO, const float* lse,
                   void* dq, void* dk, void* dv,
                   float* delta, void* workspace, size_t workspace_bytes,
                   int B, int H, int N, int d, int causal, float scale, int mode,
                   void* stream);

/*
 * attn_bwd without a caller-provided workspace.  (The paper has no counterpart to this entry
 * point; it exists for the sake of callers, not of the method.)
 *
 * Who needs it: code that has to run the backward pass at a point where it cannot obtain device
 * memory - a callback inside a host framework that owns the allocator, a serving or training loop
 * that must not hit cudaMalloc's implicit device-wide synchronisation, a process whose memory
 * budget was handed out in full at start-up.  Such a caller still passes every input and output
 * buffer; only the FP32 dQ accumulator that attn_bwd takes as `workspace` is replaced by an array
 * built into the library.
 *
 *   - The built-in scratch is ATTN_BWD_STATIC_MAX_BYTES (32 MiB) of static device memory per GPU
 *     that loads the library, held until the process exits.  A call needs
 *     attn_bwd_workspace_bytes(B,H,N,d) = 4*B*H*N*d bytes of it, i.e. B*H*N*d <= 8,388,608 elements;
 *     larger problems return ATTN_ERR_WORKSPACE and enqueue nothing (use attn_bwd instead).
 *   - No cudaMalloc, cudaFree or other allocating call is made, on any call.
 *   - The first call on each device looks up the device address of the scratch
 *     (cudaGetSymbolAddress) with that device current; make that first call outside any stream
 *     capture.  Later calls on the same device only launch kernels.
 *   - All calls on a device share the one scratch array, which keeps whatever the previous call
 *     left in it; each call clears the part it uses before accumulating.  Two calls that can
 *     overlap on the GPU (different streams, or different host threads without ordering) race on
 *     it and produce wrong dQ: serialise them, or give the concurrent ones attn_bwd with their own
 *     workspace.
 *   - Arguments, results, error codes and numerics are otherwise those of attn_bwd.
 */
#define ATTN_BWD_STATIC_MAX_BYTES  (32u << 20)
int attn_bwd_static(const void* q, const void* k, const void* v, const void* o,
                    const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta,
                    int B, int H, int N, int d, int causal, float scale, int mode,
                    void* stream);

/*
 * Grouped-query attention (not in the paper, whose experiments use multi-head attention; its method applies per query
 * head unchanged): H query heads share H_kv key/value heads, H a multiple of H_kv (else ATTN_ERR_SHAPE); query head h
 * attends to key/value head h / (H / H_kv).
 *   q, o, dO, dq   BF16 [B][H][N][d];      lse, delta  FP32 [B][H][N]
 *   k, v, dk, dv   BF16 [B][H_kv][N][d]
 * Forward: Algorithm 1 / 3 per query head, as attn_fwd.  Backward: Algorithm 2 per query head; dK and dV of a
 * key/value head accumulate the contributions of its H / H_kv query heads in FP32 (in the same TMEM accumulators, one
 * query head after the other) and are rounded to BF16 once.  Workspace: attn_bwd_workspace_bytes(B, H, N, d).
 * All other arguments, checks, modes and error codes as attn_fwd / attn_bwd; H_kv == H is exactly those functions.
 */
int attn_fwd_gqa(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream);
int attn_bwd_gqa(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                 void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                 int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream);

/*
 * Sequences whose length is not a multiple of 128 (the paper's experiments use N = 1024; nothing in the method
 * depends on it): the tensors keep N rows per head in memory, N a multiple of 128 as everywhere else, of which the
 * first `seqlen` (1 <= seqlen <= N, else ATTN_ERR_SHAPE) are the sequence and the rest is padding.
 *   - keys >= seqlen are masked out (they get probability 0), queries >= seqlen take part in nothing;
 *   - rows >= seqlen of o, lse, dq, dk, dv, delta are unspecified on return (rows of tiles that hold no sequence row
 *     are not written at all; padding rows of dk, dv inside the last tile come back as zeros);
 *   - the padding rows of q, k, v, dO must hold finite values (zeros, say): they go through the tensor cores with
 *     weight 0, and 0 * NaN would not be 0.
 * The result on the first seqlen rows is that of the algorithms on a sequence of length seqlen, with the same tiles
 * (the key tile that contains row seqlen - 1 is simply shorter).  H_kv as for attn_fwd_gqa (pass H_kv = H for
 * multi-head attention); all other arguments, checks, modes and error codes as attn_fwd / attn_bwd;
 * workspace: attn_bwd_workspace_bytes(B, H, N, d).  seqlen == N is exactly attn_fwd_gqa / attn_bwd_gqa.
 */
int attn_fwd_padded(const void* q, const void* k, const void* v, void* o, float* lse,
                    int B, int H, int H_kv, int N, int seqlen, int d, int causal, float scale, int mode, void* stream);
int attn_bwd_padded(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                    int B, int H, int H_kv, int N, int seqlen, int d, int causal, float scale, int mode, void* stream);

/*
 * One sequence length per batch element (a padded batch of sequences of different lengths): as attn_fwd_padded /
 * attn_bwd_padded, with `seqlens`, an array of B 32-bit integers in DEVICE memory (read by the kernels; NULL gives
 * ATTN_ERR_NULL), in place of the single seqlen.  Batch element b uses its first seqlens[b] rows (values are clamped
 * to [0, N]; 0 leaves every output row of that batch element unwritten).  Tiles that hold only padding are skipped by
 * the kernels, so the cost follows the actual lengths.  Everything else as for the padded entry points.
 */
int attn_fwd_varlen(const void* q, const void* k, const void* v, void* o, float* lse, const int* seqlens,
                    int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream);
int attn_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                    const int* seqlens, int B, int H, int H_kv, int N, int d, int causal, float scale, int mode,
                    void* stream);

/*
 * Packed variable-length batches: B sequences stored one after the other with no padding rows, addressed by
 * cumulative offsets (the layout training frameworks use for batches of documents of different lengths; the paper's
 * experiments use a fixed context of 1024, nothing in its method depends on that).
 *   cu_seqlens  int32 [B + 1], DEVICE memory: sequence b occupies tokens [cu_seqlens[b], cu_seqlens[b + 1]);
 *               cu_seqlens[0] = 0, non-decreasing, cu_seqlens[B] = T.  A length of 0 is allowed (nothing is written
 *               for that sequence); a length above N_max is the caller's error (the tokens beyond N_max are ignored).
 *   q, o, dO, dq   BF16 [T][H][d]      (token-major: the heads of a token are contiguous)
 *   k, v, dk, dv   BF16 [T][H_kv][d]
 *   lse, delta     FP32 [H][T]
 *   T           total number of tokens;  N_max: a multiple of 128, >= every sequence length (it sizes the workspace)
 * The result for sequence b is that of attn_fwd / attn_bwd (attn_fwd_gqa / attn_bwd_gqa when H_kv < H) on that
 * sequence alone, with the same tiles, modes and flags; every output row of every token is written, nothing else is.
 * How: a layout adapter around the per-batch-length kernels (attn_fwd_varlen / attn_bwd_varlen).  The call copies the
 * packed inputs into padded [B][H][N_max][d] tensors inside `workspace` (streaming kernels, zeros in the unused rows
 * of partly used tiles), runs those kernels, which skip the tiles that hold only padding, and copies the results
 * back; all on `stream`, no synchronisation.  The copies move every tensor once more each way (about 8 x the size
 * of q for a forward + backward); the attention kernels themselves do no work on padding tiles.
 *   workspace   device memory, 256-byte aligned, at least attn_packed_workspace_bytes(B, H, H_kv, N_max, d, backward)
 *               bytes (backward = 0 for attn_fwd_packed, 1 for attn_bwd_packed); contents undefined on entry and on
 *               return.  Too small, NULL or misaligned: ATTN_ERR_WORKSPACE.
 * With ATTN_MODE_FLAG_DELTA_GIVEN, delta is an input in the packed layout.  Other errors as attn_fwd_varlen /
 * attn_bwd_varlen; cu_seqlens == NULL: ATTN_ERR_NULL; T < 1 or T * H >= 2^31: ATTN_ERR_SHAPE.
 */
size_t attn_packed_workspace_bytes(int B, int H, int H_kv, int N_max, int d, int backward);
int attn_fwd_packed(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_seqlens,
                    void* workspace, size_t workspace_bytes, int B, int H, int H_kv, int T, int N_max, int d,
                    int causal, float scale, int mode, void* stream);
int attn_bwd_packed(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, const int* cu_seqlens,
                    void* workspace, size_t workspace_bytes, int B, int H, int H_kv, int T, int N_max, int d,
                    int causal, float scale, int mode, void* stream);

/* Bytes of scratch attn_bwd needs for this shape; 0 if the shape is unsupported. */
size_t attn_bwd_workspace_bytes(int B, int H, int N, int d);

/* Query-tile (Br) and key-tile (Bc) sizes the forward kernel uses for head
 * width d (the B_r, B_c of Algorithms 1 and 3).  Host-only, needs no GPU. */
int attn_get_tiles(int d, int* Br, int* Bc);

/* Limit on the upward shift of m under ATTN_MODE_FLAG_GUARDED (> 0, finite; else ATTN_ERR_PARAM and no change).
 * Process-wide; read by attn_fwd at call time.  Host-only. */
int attn_set_guard_max_shift(float max_shift);
float attn_get_guard_max_shift(void);

/* Parameters of the tie rule of Sec. 4 (beta > 1, eps > 0); defaults 2.0 and
 * 1e-3.  Process-wide; read by attn_fwd at call time.  Host-only. */
int attn_set_mitigation(float beta, float eps);
int attn_get_mitigation(float* beta, float* eps);

/* After the caller has synchronised `stream`: ATTN_OK, or ATTN_ERR_TIMEOUT if a
 * kernel enqueued by this library on the current device gave up on a bounded
 * wait since the last call of this function (which clears the record), or
 * ATTN_ERR_CUDA if a kernel found its shared-memory layout out of bounds. */
int attn_last_device_status(void* stream);

/*
 * Self-test of the bounded-wait path (the paper has no counterpart: this belongs to the error contract of the
 * library, not to the method).  Enqueues on `stream` a one-block kernel built like the compute kernels (barriers in
 * shared memory, a TMEM allocation, one single-thread role and one whole-warp role, the common teardown) in which
 * nothing ever arrives on the barriers the roles wait for.  Their waits are bounded at one millisecond instead of the
 * compute kernels' two seconds, so the kernel gives up after about a millisecond through the path a pipeline fault
 * would take: abort flag, every role leaves its wait, TMEM is freed, the device status word is set.  After the caller
 * has synchronised, attn_last_device_status() returns ATTN_ERR_TIMEOUT once; the context is intact and later calls
 * behave normally.  No fault, trap or unbounded loop is involved.  Returns ATTN_OK once enqueued, ATTN_ERR_DEVICE /
 * ATTN_ERR_CUDA as the compute entry points.
 */
int attn_selftest_wait_timeout(void* stream);

/* Static, human-readable text for a return code. */
const char* attn_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_H_ */
