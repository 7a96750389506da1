/*
 * ak.h - C ABI of libak: row-reduction kernels for NVIDIA B200 (sm_100a).
 *
 * Forward ops over contiguous row-major bf16 [rows, D] tensors:
 *   RMSNorm            (paper Table 3, row "rmsnorm";   Table 4 rows "rmsnorm")
 *   last-dim softmax   (paper Table 3, row "softmax";   Table 4 rows "softmax")
 *   fused cross-entropy(paper Table 3, row "cross_ent": online log-sum-exp fused with
 *                       the NLL gather; Table 4 rows "cross_ent")
 * and, built on the same skeletons: LayerNorm ("layernorm"), row-sum ("reduce"), rotary
 * embedding ("rotary_emb"), fp16 / fp32 variants of the first three (*_dt) and the
 * vocabulary-parallel form of the cross-entropy (ak_xent_vp_*).
 * Semantics are those of the PyTorch reference ops the paper uses as its correctness
 * oracle (Section 6): F.rms_norm, F.softmax(dim=-1), F.cross_entropy(ignore_index).
 *
 * Conventions for every entry point unless stated otherwise
 *   - Pointers named *_dev / without suffix in the device entry points are DEVICE
 *     pointers valid on the current CUDA device.  The caller owns them for the whole
 *     asynchronous lifetime of the call; the library neither frees nor retains them.
 *   - Tensors are dense row-major, row stride == D (or V) elements; bf16 = the upper 16
 *     bits of an IEEE-754 binary32.  Any D >= 1 and any 2-byte-aligned bf16 pointer is
 *     accepted; the fastest paths need 16-byte aligned base pointers and D % 8 == 0.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Device entry points only enqueue work; they never synchronise.
 *   - The return value is an ak_status.  Arguments are validated on the host before any
 *     launch.  Data-dependent problems (an out-of-range target) cannot be reported
 *     synchronously and are encoded in the output (NaN); no kernel ever traps.  The one
 *     device-side failure that is not encoded in the output, a bounded wait that gave up, is
 *     reported by ak_wait_timeouts().
 *   - Calls act on the CURRENT CUDA device: pointers must belong to it, and a process that
 *     drives several GPUs makes the tensors' device current before each call (the Python
 *     binding does).  Function attributes, occupancy figures, scratch pools, the host-buffer
 *     arena and the static scratch are kept per device.
 *   - Kernels are launched as programmatic dependents (programmatic stream serialisation): their
 *     CTAs may become resident while the previous kernel of the stream drains, but every read and
 *     write comes after griddepcontrol.wait, i.e. after that kernel has completed and flushed;
 *     before the wait they only prefetch their first inputs into L2 (AK_DISABLE_PREFETCH=1 in
 *     the environment, read once, switches that prefetch off).  Stream order is therefore
 *     observed exactly as for ordinary launches, with any kernel before or after.
 *   - Stream-ordered scratch, where an entry point says it uses some, comes from a CUDA
 *     memory pool of the library's own (one per device, created at first use, keeps up to
 *     256 MiB cached between calls) through cudaMallocFromPoolAsync / cudaFreeAsync on the
 *     call's stream; such calls may be captured in CUDA graphs.
 *   - Thread-block clusters: AK_PATH_CLUSTER kernels need the device to co-schedule up to eight
 *     CTAs.  Where a cluster launch is refused (a partition of a device with too few SMs per
 *     GPC), the dispatcher falls back to one CTA per row or the multi-pass kernels; setting
 *     AK_DISABLE_CLUSTERS=1 in the environment (read once) makes that the choice from the start.
 *   - rows == 0 is legal: nothing is launched (cross-entropy still writes loss_mean = NaN).
 *   - Determinism: same inputs, shape, pointer alignment, library build and GPU model
 *     give bit-identical outputs.  Path selection is a pure function of
 *     (rows, D, pointer alignment); no float atomics, no order-dependent reductions.
 *   - y may alias x exactly (in-place) for RMSNorm and softmax; partial overlap is
 *     undefined.
 *   - Re-entrant; safe to call concurrently on different streams.
 */
#ifndef AK_H_
#define AK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AK_OK = 0,
    AK_ERR_NULL = 1,   /* a required pointer is NULL */
    AK_ERR_SHAPE = 2,  /* rows < 0, D <= 0, or a size the chosen path cannot take */
    AK_ERR_ALIGN = 3,  /* pointer not aligned to its element type (or to 16 B where a forced path needs it) */
    AK_ERR_ARG = 4,    /* eps negative or not finite; bad base or position offset; unknown path id or dtype; bad nsplit */
    AK_ERR_CUDA = 5,   /* a CUDA runtime call or launch failed */
    AK_ERR_NOMEM = 6,  /* scratch allocation failed or caller workspace too small */
    AK_ERR_CAPACITY = 7 /* problem larger than the fixed scratch of ak_xent_fwd_static */
} ak_status;

/* Path ids for the *_path entry points (testing / tuning).  0 always means "let the
 * dispatcher choose", which is what the plain entry points do. */
enum {
    AK_PATH_AUTO = 0,
    /* Size limits are in row BYTES (bf16: D = bytes / 2); the register and shared-memory paths
     * need 16-byte aligned pointers and rows that are a multiple of 16 bytes. */
    AK_PATH_WARP = 1,     /* one (or two) warps per row, row held in registers; rows <= 4 KiB (bf16 D <= 2048) */
    AK_PATH_CTA = 2,      /* one CTA per row, row held in registers; rows <= 64 KiB (bf16 D <= 32768) */
    AK_PATH_GENERIC = 3,  /* any D, any element alignment; the row is kept in registers or staged in shared memory (of one CTA, or of a cluster of up to eight for rows beyond 224 KiB and for a few long rows) in its 16-byte phase: a single DRAM pass; else re-read from L1/L2 */
    AK_PATH_SMEM = 4,     /* one CTA per row, row staged in shared memory by bulk (TMA) copies; rows <= 224 KiB (bf16 D <= 114688) */
    AK_PATH_CLUSTER = 5   /* a thread-block cluster of 2, 4 or 8 CTAs per row, each staging a slice in its shared memory, partial results exchanged through distributed shared memory; rows of 32 bytes and more.  The dispatcher takes it for aligned rows longer than 64 KiB, in slices of at most 32 KiB where eight CTAs can do that, and for at most 64 rows of 32 KiB or more (eight CTAs each); rows beyond 1792 KiB (bf16 D > 917504) do not fit eight CTAs' shared memory and are streamed from global memory by the eight CTAs instead (two or three reads, the later ones from the caches where they still hold the slice) */
};
/* Element types of the *_dt entry points.  The plain entry points are bf16. */
enum {
    AK_DTYPE_BF16 = 0,
    AK_DTYPE_F16 = 1,     /* IEEE binary16 */
    AK_DTYPE_F32 = 2
};
enum {
    AK_XENT_AUTO = 0,
    AK_XENT_ROW = 1,      /* one CTA streams a whole row (online max / sum-exp), loss written directly */
    AK_XENT_SPLIT = 2     /* nsplit CTAs per row write partial (max, sum-exp); a merge kernel finishes */
};

/* ---------------------------------------------------------------------------------
 * RMSNorm forward (Table 3 "rmsnorm": warp-shuffle reduction, fast rsqrt; the weight
 * multiply is fused into the epilogue as in Section 7.3, Tier 3).
 *   y[r, j] = bf16_rne( x[r, j] * w[j] * rsqrt( (1/D) sum_k x[r, k]^2 + eps ) )
 * x, y: device bf16 [rows, D]; w: device bf16 [D]; accumulation in fp32.
 * eps must be finite and >= 0.
 * Range: the squares are added in fp32, so a row whose sum of squares exceeds 3.4e38 (|x| of
 * about 1e19 / sqrt(D) and more; bf16 itself reaches 3.4e38) gives inf, rstd = 0 and an output
 * row of exact zeros where the definition gives about +-w.  (LayerNorm likewise returns beta for
 * a row whose squared deviations overflow.)  Softmax and cross-entropy have no such limit.
 */
int ak_rmsnorm_fwd(const void* x, const void* w, void* y,
                   int64_t rows, int64_t D, float eps, void* cuda_stream);
int ak_rmsnorm_fwd_path(const void* x, const void* w, void* y,
                        int64_t rows, int64_t D, float eps, void* cuda_stream, int path);

/* ---------------------------------------------------------------------------------
 * Element-type variants of the three ops (the paper measures in FP16 and its benchmark
 * harness sweeps FP16 / BF16 / FP32: Section 6 and the Table 4 caption).  Same definitions
 * as the bf16 entry points; `dtype` (AK_DTYPE_*) is the type of x, w, y / logits; losses
 * stay fp32; accumulation is fp32; outputs are rounded once, to nearest even (fp32
 * outputs carry the fp32 arithmetic's own rounding).  Pointers must be aligned to the
 * element size; the fast paths need 16-byte aligned bases and rows that are a multiple of
 * 16 bytes (D % 8 == 0 for 16-bit types, D % 4 == 0 for fp32); the path limits of AK_PATH_*
 * scale with the row's BYTES (4 KiB / 64 KiB / 224 KiB; clusters stage up to 1792 KiB).  fp16 outputs beyond 65504
 * become inf, as the type dictates.  `path` (and `nsplit`) as in the *_path entry points;
 * 0 = automatic.  An unknown dtype gives AK_ERR_ARG.
 */
int ak_rmsnorm_fwd_dt(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                      int dtype, void* cuda_stream, int path);
int ak_softmax_fwd_dt(const void* x, void* y, int64_t rows, int64_t D,
                      int dtype, void* cuda_stream, int path);
int ak_xent_fwd_dt(const void* logits, const int64_t* targets, int64_t ignore_index,
                   float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                   int dtype, void* cuda_stream, int path, int nsplit);
/* LayerNorm and row-sum in the element type `dtype` (x, gamma, beta, y; the sums stay fp32);
 * same rules as the *_dt entry points above. */
int ak_layernorm_fwd_dt(const void* x, const void* gamma, const void* beta, void* y,
                        int64_t rows, int64_t D, float eps, int dtype, void* cuda_stream, int path);
int ak_rowsum_fwd_dt(const void* x, float* out, int64_t rows, int64_t D, int dtype, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Rotary position embedding forward (Table 3 "rotary_emb": interleaved rotation; Table 4
 * rows "rotary": batch x heads x sequence x head_dim).
 *   x, y: device [n_seq, S, Dh] of `dtype`, n_seq = batch * heads, dense; y may alias x.
 *   The head vector at sequence index s has position p = pos_offset + s; its pair
 *   i = elements (2i, 2i + 1) turns by theta = p * base^(-2i / Dh):
 *     y[2i]     = rne( x[2i] cos(theta) - x[2i + 1] sin(theta) )
 *     y[2i + 1] = rne( x[2i] sin(theta) + x[2i + 1] cos(theta) )
 * Dh even, 2 <= Dh <= 512 (else AK_ERR_SHAPE); base finite and > 0 (typically 10000);
 * 0 <= pos_offset < 2^52.  Frequencies f_i = base^(-2i / Dh) are formed in double on the host;
 * the angle is the double product fl(p * f_i), reduced to [-pi, pi] in double on the device, so
 * cos / sin of that angle are right to fp32 rounding at any accepted position.  The double
 * product itself is within p * f_i * 2^-53 rad of the real one: below fp32's rounding while
 * p * f_i < 2^28, 6e-5 rad at 2^40.  Products and sums in fp32.  Fast path: 16-byte aligned x and y and Dh a multiple of the elements in
 * 16 bytes; anything else takes an element-wise kernel.  One launch, no scratch.
 */
int ak_rope_fwd(const void* x, void* y, int64_t n_seq, int64_t S, int64_t Dh, float base,
                int64_t pos_offset, int dtype, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Vocabulary-parallel cross-entropy (the fused cross_ent of Table 3 with the vocabulary
 * dimension sharded over ranks, as in tensor-parallel language-model heads).  Rank k holds
 * logits_shard: device [rows, V_local] of `dtype`, the columns
 * [vocab_start, vocab_start + V_local) of the full [rows, V_total] logits; targets index the
 * FULL vocabulary and are the same on every rank.
 *   1. ak_xent_vp_partial on every rank: writes `partial` = rows * (nsplit + 1) pairs of fp32
 *      (ak_xent_vp_partial_bytes): per row, nsplit online (max, sum-exp) pairs of the shard's
 *      slices, then (x[r, t], 1) if this shard owns column t, else (0, 0).  Rows whose target
 *      is ignore_index or outside [0, V_total) are neither read nor written.
 *   2. the caller all-gathers the partial buffers in rank order into [nranks][rows][nsplit+1]
 *      pairs (16 * (nsplit + 1) bytes per row and rank; the only exchange).
 *   3. ak_xent_vp_merge on every rank: merges in (rank, slice) order and writes loss_rows
 *      [rows] and, if not NULL, loss_mean [1], with the conventions of ak_xent_fwd; identical
 *      bits on all ranks.  A valid target owned by no shard or by several gives NaN.
 * nsplit (1..64) must be the same on all ranks; ak_xent_vp_nsplit gives the dispatcher's
 * choice for (rows, V_local) (1 when rows alone fill the GPU).  All buffers are caller-owned;
 * nothing is allocated; each call enqueues one or two kernels on `cuda_stream`.
 */
int ak_xent_vp_nsplit(int64_t rows, int64_t V_local);
size_t ak_xent_vp_partial_bytes(int64_t rows, int nsplit);
int ak_xent_vp_partial(const void* logits_shard, const int64_t* targets, int64_t ignore_index,
                       int64_t vocab_start, int64_t V_total, void* partial,
                       int64_t rows, int64_t V_local, int nsplit, int dtype, void* cuda_stream);
int ak_xent_vp_merge(const void* partials, int nranks, int nsplit, const int64_t* targets,
                     int64_t ignore_index, int64_t V_total, float* loss_rows, float* loss_mean,
                     int64_t rows, void* cuda_stream);

/* Path the dispatcher picks for op (0 = RMSNorm, 1 = softmax, 2 = LayerNorm) at this shape, alignment and
 * element type; -1 for an unknown op or dtype.  Pure function; no CUDA calls. */
int ak_choose_path_dt(int op, int64_t rows, int64_t D, int aligned16, int dtype);

/* ---------------------------------------------------------------------------------
 * LayerNorm forward (Table 3 "layernorm"; Table 4 rows "layernorm").
 *   mu = (1/D) sum_k x[r, k];  var = (1/D) sum_k (x[r, k] - mu)^2   (biased)
 *   y[r, j] = bf16_rne( (x[r, j] - mu) * rsqrt(var + eps) * gamma[j] + beta[j] )
 * x, y: device bf16 [rows, D] (y may alias x); gamma, beta: device bf16 [D]; moments in
 * fp32 and fixed order over the on-chip copy of the row, shifted by a value K taken from the
 * row itself (its first element, or the mean of its first 16 bytes): mu = K + mean(x - K),
 * so a constant row gives exactly beta.  Short rows and unaligned rows held in registers then
 * sum x - mu and (x - mu)^2 in a second pass: var = mean((x - mu)^2) - mean(x - mu)^2, and
 * mean(x - mu) is added to mu, which removes what a shift far from the mean (an outlier as
 * first element) had cost it.  The other layouts take sum((x - K)^2) in the first sweep and use
 * var = mean((x - K)^2) - (mu - K)^2 when (mu - K)^2 <= var (the subtraction then costs at
 * most a factor three in the relative error of var); otherwise they make that second pass
 * too.  With fp32 elements (ak_layernorm_fwd_dt) the mean is kept as a sum of two floats and
 * the output subtracts them one after the other, so a mean far above the spread (1024 +- 8)
 * costs no accuracy either.  eps finite, >= 0.
 * Same path ids, size limits and alignment rules as RMSNorm (gamma and beta together play
 * the part of w).  Status codes as for RMSNorm.  One launch and no scratch, except for many
 * rows that are not 16-byte aligned (1024 or more of D <= about 4090, 256 or more longer ones
 * up to 1792 KiB): then a small kernel first writes gamma and beta in all eight 2-byte shifts to
 * about 32 * D bytes of stream-ordered scratch obtained and released on `cuda_stream`, and
 * the row kernel runs as its programmatic dependent; if the scratch cannot be had the
 * single-launch kernel runs instead (same results).
 */
int ak_layernorm_fwd(const void* x, const void* gamma, const void* beta, void* y,
                     int64_t rows, int64_t D, float eps, void* cuda_stream);
int ak_layernorm_fwd_path(const void* x, const void* gamma, const void* beta, void* y,
                          int64_t rows, int64_t D, float eps, void* cuda_stream, int path);

/* ---------------------------------------------------------------------------------
 * Row-sum reduce (Table 3 "reduce").
 *   out[r] = fp32( sum_k x[r, k] ),  fp32 accumulation in a fixed order
 * x: device bf16 [rows, D], 2-byte aligned, any D >= 1; out: device fp32 [rows], caller
 * owned.  One launch and no scratch, except for a few long rows (rows < 4 * SMs = 592 and D >= 16384; a
 * vector sum is rows == 1): then nsplit CTAs per row write partial sums and a second launch
 * adds them in a fixed order, with rows * nsplit * 4 bytes of stream-ordered scratch obtained
 * and released on `cuda_stream` (AK_ERR_NOMEM if that fails).  inf/NaN propagate per IEEE-754.
 */
int ak_rowsum_fwd(const void* x, float* out, int64_t rows, int64_t D, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Softmax forward over the last dimension (Table 3 "softmax").
 *   m = max_k x[r, k];  y[r, j] = bf16_rne( exp(x[r, j] - m) / sum_k exp(x[r, k] - m) )
 * -inf entries (a causal mask lives in the data) give exactly 0.  A row that is all
 * -inf, or contains +inf or NaN, gives NaN (IEEE / PyTorch convention).
 */
int ak_softmax_fwd(const void* x, void* y, int64_t rows, int64_t D, void* cuda_stream);
int ak_softmax_fwd_path(const void* x, void* y, int64_t rows, int64_t D,
                        void* cuda_stream, int path);

/* ---------------------------------------------------------------------------------
 * Fused cross-entropy forward (Table 3 "cross_ent": online log-sum-exp, fused NLL).
 *   t = targets[r]
 *   t == ignore_index        : loss_rows[r] = 0, row not counted (its logits are not read)
 *   t < 0 or t >= V          : loss_rows[r] = NaN, row counted (so the mean is NaN)
 *   otherwise                : loss_rows[r] = (m - x[r, t]) + log(sum_k exp(x[r, k] - m))
 *   loss_mean[0] = (sum of counted loss_rows, fp64, fixed order) / n_counted   (0/0 = NaN)
 * logits: device bf16 [rows, V]; targets: device int64 [rows]; loss_rows: device fp32
 * [rows] (required); loss_mean: device fp32 [1] or NULL (mean skipped).
 * Rows with very long vocabularies or too few rows to fill the GPU take the split-row
 * two-phase path, which needs rows * nsplit * 8 bytes of scratch: ak_xent_fwd obtains and
 * releases it stream-ordered on `cuda_stream` (AK_ERR_NOMEM on failure); ak_xent_fwd_ws takes
 * it from the caller instead.
 */
int ak_xent_fwd(const void* logits, const int64_t* targets, int64_t ignore_index,
                float* loss_rows, float* loss_mean,
                int64_t rows, int64_t V, void* cuda_stream);

/* Bytes of scratch ak_xent_fwd_ws needs for this shape (0 when the dispatcher picks the
 * one-CTA-per-row path).  Pure function of (rows, V). */
size_t ak_xent_workspace_bytes(int64_t rows, int64_t V);

/* Same as ak_xent_fwd but never allocates: `workspace` is a device buffer of at least
 * ak_xent_workspace_bytes(rows, V) bytes, 8-byte aligned, owned by the caller and free
 * to reuse once the work enqueued on `cuda_stream` has finished.  May be NULL when the
 * required size is 0. */
int ak_xent_fwd_ws(const void* logits, const int64_t* targets, int64_t ignore_index,
                   float* loss_rows, float* loss_mean,
                   int64_t rows, int64_t V, void* workspace, size_t workspace_bytes,
                   void* cuda_stream);

/* Testing / tuning variant: force the path and, for AK_XENT_SPLIT, the number of splits
 * per row (1..64; 0 = dispatcher's choice).  Scratch is obtained as in ak_xent_fwd. */
int ak_xent_fwd_path(const void* logits, const int64_t* targets, int64_t ignore_index,
                     float* loss_rows, float* loss_mean,
                     int64_t rows, int64_t V, void* cuda_stream, int path, int nsplit);

/* ---------------------------------------------------------------------------------
 * Cross-entropy forward that never allocates.  (The paper has no counterpart: this entry
 * point exists for the library's users, not for parity with anything the paper describes.)
 *
 * For callers that cannot obtain device memory at call time - a process whose whole memory
 * budget went to its own arena at start-up, a job under a hard GPU quota, a latency-critical
 * loop that must stay out of the allocator.  Same arguments, outputs and conventions as
 * ak_xent_fwd, computed with the split-row layout (the split count the dispatcher would pick
 * for (rows, V)), but the per-slice scratch lives in a fixed 1 MiB array inside the library's
 * device image: every GPU that loads the library holds that 1 MiB until the process exits, and
 * the call performs no cudaMalloc, cudaFree or other allocating routine.
 *   - Limit: rows <= 65535 and rows * nsplit * 8 bytes <= 1 MiB (131072 slices), otherwise
 *     AK_ERR_CAPACITY is returned and nothing is launched.  (4096 rows of any vocabulary, or
 *     2048 rows split 64 ways, fit.)
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device current) and caches it; make that first call before any stream capture.
 *   - All calls on a device share the array and inherit its previous contents.  Nothing needs
 *     clearing (every slot read is written earlier in the same call), but calls whose kernels
 *     overlap on the GPU (different streams) race on it: serialise them, or give each its own
 *     buffer through ak_xent_fwd_ws.
 */
int ak_xent_fwd_static(const void* logits, const int64_t* targets, int64_t ignore_index,
                       float* loss_rows, float* loss_mean,
                       int64_t rows, int64_t V, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Row-sharded cross-entropy (one process per GPU, each holding a block of rows).  Per-row
 * losses need no exchange; the scalar mean needs one: every rank computes its pair
 * {sum of counted loss_rows (fp64, fixed order), number of counted rows (as a double)} with
 * ak_xent_sum_count, the 16-byte pairs are all-gathered in rank order by the caller (NCCL),
 * and ak_xent_mean_merge adds them in index order and writes sum / count (0/0 = NaN), which
 * is bit-identical on every rank.  The paper's system is single-GPU (Section "Limitations");
 * this is the row-shard extension of the mean in ak_xent_fwd.
 * sum_count: device double[2]; sum_count_pairs: device double[2 * n]; loss_mean: device fp32[1].
 * An empty block (rows == 0: loss_rows and targets may be NULL) contributes {0, 0}; n == 0
 * (sum_count_pairs may be NULL) gives NaN.  Both calls only enqueue work on cuda_stream: the
 * all-gather between them has to be ordered on that same stream by the caller.
 */
int ak_xent_sum_count(const float* loss_rows, const int64_t* targets, int64_t ignore_index,
                      int64_t rows, double* sum_count, void* cuda_stream);
int ak_xent_mean_merge(const double* sum_count_pairs, int64_t n, float* loss_mean, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Host-buffer variants: the same ops for callers whose tensors live in HOST memory
 * (pinned memory gives full PCIe speed; pageable works).  Each call copies its inputs to
 * a library-owned device arena in row chunks, runs the device kernels, copies results
 * back, and returns after everything has completed (it synchronises its own internal
 * streams only).  Copy-in, compute and copy-out of successive chunks overlap.  The arena
 * is cached per device and grows on demand; ak_host_arena_release frees it.  Calls are
 * serialised by an internal lock.  All pointers here are HOST pointers.
 */
int ak_rmsnorm_fwd_host(const void* x_host, const void* w_host, void* y_host,
                        int64_t rows, int64_t D, float eps);
int ak_softmax_fwd_host(const void* x_host, void* y_host, int64_t rows, int64_t D);
int ak_xent_fwd_host(const void* logits_host, const int64_t* targets_host, int64_t ignore_index,
                     float* loss_rows_host, float* loss_mean_host, int64_t rows, int64_t V);
int ak_host_arena_release(void);

/* ---------------------------------------------------------------------------------
 * Speed-of-light measurement aids (no op arithmetic): a streaming device-to-device copy and
 * a streaming read, built from the same 16-byte streaming accesses and small one-shot CTAs
 * as the row kernels, so the benchmark can report each op against the bandwidth this GPU
 * actually delivers for 1:1 read/write traffic (RMSNorm, softmax; the paper's GB/s accounting
 * for Table 4) and for read-only traffic (cross-entropy).  src / dst: device pointers,
 * 16-byte aligned, `bytes` a multiple of 16; sink4: 4 writable device bytes (left untouched
 * for ordinary data).
 */
int ak_sol_copy(const void* src, void* dst, size_t bytes, void* cuda_stream);
int ak_sol_read(const void* src, size_t bytes, void* sink4, void* cuda_stream);

/* ---------------------------------------------------------------------------------
 * Introspection.
 */
/* Path id the dispatcher picks for (rows, D) with fully aligned pointers (`aligned16` != 0)
 * or not.  Pure functions of their arguments and of the current device's SM count (which decides
 * when few rows are split over more CTAs); they launch nothing. */
int ak_rmsnorm_choose_path(int64_t rows, int64_t D, int aligned16);
int ak_layernorm_choose_path(int64_t rows, int64_t D, int aligned16);
int ak_softmax_choose_path(int64_t rows, int64_t D, int aligned16);
/* Returns AK_XENT_ROW or AK_XENT_SPLIT and stores the split count (1 for ROW). */
int ak_xent_choose_path(int64_t rows, int64_t V, int* nsplit_out);

/* Number of kernel launches this library has enqueued in this process so far. */
int64_t ak_launch_count(void);

/* SMs of the current device as the dispatch rules see them (148 on a full B200; also 148 when
 * no device can be queried).  The split rules are stated in multiples of it: cross-entropy
 * splits rows when rows < 4 * SMs, the row sum when rows < 4 * SMs as well. */
int ak_sm_count(void);

/* Bounded waits.  The kernels that stage rows through shared memory wait for their own bulk
 * copies (and, in the cluster layouts, for their cluster partners' mailbox posts) on mbarriers,
 * polling at most 2^20 times; they never spin without a limit and never trap.  A wait that gives
 * up is not expected on a healthy device; the threads that hit it stop and leave their part of
 * the output unwritten, and a flag is set on the device.  The status of the call that launched
 * the kernel cannot show this (calls only enqueue): this function reads the flags of the
 * current device, synchronising with it, and returns 0 if no wait ever gave up, the number of
 * kernel families (RMSNorm, softmax, LayerNorm) that saw one otherwise, -1 if the flags cannot be
 * read (no device).  The flags stay set until the process ends. */
int ak_wait_timeouts(void);

/* Static, never-freed description of a status code. */
const char* ak_status_string(int status);

/* Library version, major * 10000 + minor * 100 + patch. */
int ak_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AK_H_ */
