/*
 * reflex.h -- C ABI of the B200 (sm_100a) hot path of Reflex streaming inference: the
 * per-denoising-step action-expert layer. Flow-phase-gated AdaRMSNorm, attention of the dynamic
 * action-token queries over a KV context held in three regions (pinned static prefix, sliding
 * ring, dynamic suffix), and the Euler flow update of the action chunk.
 *
 * Conventions
 *   - Every function returns an int status: REFLEX_OK (0) or a negative REFLEX_ERR_* code. Nothing
 *     throws, aborts or exits. reflex_last_error_string() gives a thread-local description of the
 *     last failure on the calling thread.
 *   - Arguments are validated on the host before anything is launched: a failing call launches
 *     nothing and leaves cache state unchanged.
 *   - All work is enqueued asynchronously on the caller's CUDA stream, passed as void*
 *     (a cudaStream_t; NULL = the legacy default stream). Calls on one stream are ordered.
 *   - The five hot-path calls allocate no memory ("zero dynamic allocations during the control
 *     loop", Sec. 3.4). Device memory -- cache slabs, workspace, tensors -- is allocated by the
 *     caller and lent as raw pointers; the library owns only the host-side handle.
 *   - "device" / "host" beside a pointer says where the memory lives. Device tensors are dense,
 *     row-major in the index order written, and must be 16-byte aligned (REFLEX_ERR_ALIGN).
 *   - dtype is the storage type of K, V, Q, x, weights: REFLEX_DTYPE_BF16 or REFLEX_DTYPE_F32.
 *     Accumulation, softmax state and normalisation statistics are always fp32.
 *   - Symbols: B streams, L layers, Hq / Hkv query / KV heads (G = Hq/Hkv), d head_dim,
 *     S static-prefix tokens (capacity S_max), N ring capacity in tokens, T dynamic action tokens
 *     (capacity T_max), D norm width, Cd conditioning width, Hd gate-MLP hidden width, A action width,
 *     K denoising steps.
 */
#ifndef REFLEX_H
#define REFLEX_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define REFLEX_OK                    0
#define REFLEX_ERR_INVALID_ARG      (-1)  /* NULL pointer, bad enum, id out of range or duplicated   */
#define REFLEX_ERR_SHAPE            (-2)  /* a size outside the range the call or the handle accepts  */
#define REFLEX_ERR_ALIGN            (-3)  /* a device pointer or row pitch not 16-byte aligned        */
#define REFLEX_ERR_STATE            (-4)  /* e.g. attention on a stream whose prefix was never set    */
#define REFLEX_ERR_CUDA             (-5)  /* a CUDA runtime/driver call failed                        */
#define REFLEX_ERR_TIMEOUT          (-6)  /* a bounded device-side wait ran out (status word)         */
#define REFLEX_ERR_NOT_IMPLEMENTED  (-7)

#define REFLEX_DTYPE_BF16 0
#define REFLEX_DTYPE_F32  1

/* attention kernel selection (reflex_cache_set_attention_impl) */
#define REFLEX_ATTN_AUTO   0   /* a tensor-core kernel when the shape qualifies, else the SIMT kernel */
#define REFLEX_ATTN_SIMT   1   /* fp32-FMA split-K kernel, any supported shape and dtype            */
#define REFLEX_ATTN_TC     2   /* tcgen05 kernel, one CTA per 128-row query tile, key split when the grid is small;
                                  REFLEX_ERR_NOT_IMPLEMENTED if the shape does not qualify             */
#define REFLEX_ATTN_TC2    3   /* tcgen05 cta_group::2 kernel: a CTA pair per 256 query rows (batched serving)  */

typedef struct reflex_cache reflex_cache_t; /* opaque, host-side */

/* Geometry of a partitioned KV cache (Sec. 3.1: static prefix / sliding history / dynamic suffix;
 * Sec. 3.4: one monolithic pre-allocated buffer, here with a stream axis added). */
typedef struct {
    int32_t L, B, Hq, Hkv, d;
    int32_t S_max;   /* capacity of the static-prefix region, tokens            */
    int32_t N;       /* capacity of the sliding ring, tokens                    */
    int32_t T_max;   /* largest number of dynamic (action) tokens per call      */
    int32_t dtype;   /* REFLEX_DTYPE_*                                           */
    int32_t static_banks; /* 0 or 1: one static region; 2: two banks, so that a new prefix can be staged while the
                             current one is being read (reflex_cache_stage_static / reflex_cache_commit_static) */
} reflex_cache_desc;

const char *reflex_last_error_string(void);
const char *reflex_version(void);
/* Kernels launched by this library in this process so far (all entry points, all threads). */
unsigned long long reflex_kernel_launch_count(void);

/* ---- helpers around the five hot-path calls -------------------------------------------------- */

/* Bytes of ONE slab (K or V; the caller allocates two): [L][B][banks * S_max + N][Hkv][d] elements of
 * dtype (banks = 2 with static_banks == 2, else 1). Rows [0, banks * S_max) of a (layer, stream) block are
 * the static region (bank k at rows [k S_max, (k + 1) S_max)), the N rows after them the ring in physical
 * slot order. The dynamic suffix is never copied into the slab: attention
 * reads it from the caller's tensors in place. Returns 0 for an invalid descriptor. */
size_t reflex_cache_slab_bytes(const reflex_cache_desc *desc);

/* Bytes of the workspace the caller lends: per-stream ring state, split-K partials, tickets,
 * status word. Returns 0 for an invalid descriptor. */
size_t reflex_workspace_bytes(const reflex_cache_desc *desc);

/* Create a handle over caller-owned device memory. k_slab, v_slab (device, slab_bytes each, contents
 * kept as found -- zero them for the paper's zero-initialised buffer) and workspace (device,
 * workspace_bytes; its state part is initialised by this call on `stream`). ring_head0: host [B]
 * initial write positions in [0, N), or NULL for 0. The handle keeps the pointers; the memory must
 * outlive it. Requirements: Hq % Hkv == 0, d % 32 == 0, d <= 256, all sizes >= 1 (S_max may be 0). */
int reflex_cache_create(const reflex_cache_desc *desc, void *k_slab, void *v_slab, void *workspace,
                        const int32_t *ring_head0, void *stream, reflex_cache_t **out);
int reflex_cache_destroy(reflex_cache_t *cache);

/* Copy the device-side ring state to host arrays (each [B], any may be NULL) and refresh the
 * handle's host mirror. static_len is -1 for a stream whose prefix was never set. Synchronises
 * `stream`. The device copy is what kernels read, so replaying a captured CUDA graph of appends
 * advances it without the host mirror; call this afterwards to resynchronise. */
int reflex_cache_get_state(reflex_cache_t *cache, int32_t *static_len, int32_t *head, int32_t *count,
                           int64_t *total_appended, void *stream);

/* slot_of_age (host, [N]): physical ring slot of the token of age j (0 = oldest) for stream b,
 * -1 beyond the live count, from the host mirror: slot = (head - count + j) mod N. */
int reflex_cache_slot_map(reflex_cache_t *cache, int b, int32_t *slot_of_age);

int reflex_cache_set_attention_impl(reflex_cache_t *cache, int impl);

/* Every device-side wait in the kernels is bounded; a wait that runs out raises a status word in the
 * workspace instead of hanging the GPU. Reads that word (synchronises `stream`): REFLEX_OK, or
 * REFLEX_ERR_TIMEOUT with the wait site in the error string. The word stays set until the cache is
 * created again. */
int reflex_cache_check_status(reflex_cache_t *cache, void *stream);

/* Self-test of that convention, safe by construction: launches one thread that waits on a barrier nothing will ever
 * complete, gives up after limit_us microseconds (1..100000) and raises the cache's status word (wait site 127) exactly as
 * a real kernel would. reflex_cache_check_status then returns REFLEX_ERR_TIMEOUT; the CUDA context stays usable, and a
 * cache created anew over the same memory starts with a clear status word. */
int reflex_cache_selftest_wait_limit(reflex_cache_t *cache, int limit_us, void *stream);

/* ---- the five hot-path calls ------------------------------------------------------------------ */

/* Sec. 3.1 "Static Prefix ... computed once and permanently pinned"; timestep invariance of the
 * encoder makes it valid for every denoising step. Writes K,V of the perception/language prefix of
 * n_streams streams into rows [0, S[i]) of every layer and sets static_len. Nothing else changes
 * (ring kept; rows beyond S[i] keep stale bytes and are masked by static_len).
 *   stream_ids  host [n_streams], distinct, each in [0, B)
 *   k_static, v_static  device [n_streams][L][S_src][Hkv][d]
 *   S           host [n_streams], 0 <= S[i] <= min(S_src, S_max); NULL = S_src for all */
int reflex_cache_init_static(reflex_cache_t *cache, const int32_t *stream_ids, int n_streams,
                             const void *k_static, const void *v_static, int S_src, const int32_t *S,
                             void *stream);

/* Sec. 3.4 "Stream Throughput: Asynchronous Pipeline": the vision thread (producer) pushes the K,V of a new observation
 * while the policy thread (consumer) keeps denoising against the current one. With static_banks == 2:
 *   reflex_cache_stage_static   writes a new prefix into the bank that attention is NOT reading (arguments as
 *                               reflex_cache_init_static) and records its length as staged; attention launched
 *                               before or after it on any stream still reads the current prefix, so this call may
 *                               run on the producer's stream concurrently with the consumer's denoising steps;
 *   reflex_cache_commit_static  makes the staged prefix of the listed streams the current one: an index flip and
 *                               a length update by a tiny kernel on `stream`, no copy. Order it after the staging
 *                               (an event wait on the consumer's stream) and between two chunks.
 * The host mirror follows the calls (static_len as returned by reflex_cache_get_state is the committed length).
 * Errors: REFLEX_ERR_STATE when the cache has one bank or nothing is staged for a listed stream; else as
 * reflex_cache_init_static. */
int reflex_cache_stage_static(reflex_cache_t *cache, const int32_t *stream_ids, int n_streams,
                              const void *k_static, const void *v_static, int S_src, const int32_t *S,
                              void *stream);
int reflex_cache_commit_static(reflex_cache_t *cache, const int32_t *stream_ids, int n_streams, void *stream);

/* Sec. 3.1 "Sliding History ... FIFO queue of the last N"; Sec. 3.4 circular pointer arithmetic into
 * the pre-allocated buffer; App. B.1 "returns eviction count". Appends m tokens per stream in place,
 * in every layer: token i goes to slot (head + i) mod N; head <- (head + m) mod N;
 * count <- min(count + m, N). O(m) whatever the history length.
 *   k_new, v_new  device [n_streams][L][m][Hkv][d]
 *   m             1..N
 *   evicted       host [n_streams] out, may be NULL: max(0, count + m - N) per stream (host mirror) */
int reflex_cache_append_sliding(reflex_cache_t *cache, const int32_t *stream_ids, int n_streams,
                                const void *k_new, const void *v_new, int m, int32_t *evicted,
                                void *stream);

/* Eq. 2 / App. B.3: y = x * rsqrt(mean_i x_i^2 + eps) * (1 + W2 SiLU(W1 c + b1) + b2), statistics
 * and gate accumulation in fp32, one rounding to dtype on store. One gate vector per stream.
 *   x, y     device [B][R][D], may alias
 *   cond     device [B][Cd] dtype, or NULL when gate_buf holds a precomputed gate
 *   W1 [Hd][Cd], b1 [Hd], W2 [D][Hd], b2 [D]  device, dtype (ignored when cond == NULL)
 *   gate_buf device fp32 or NULL.
 *            cond != NULL, gate_buf == NULL: one fused launch, every block recomputes its stream's gate
 *                                            (fine for a single stream, wasteful for a batch).
 *            cond != NULL, gate_buf != NULL: gate_buf holds B*(D+Hd) floats (the gate [B][D] is written to
 *                                            the first B*D; the rest is reserved scratch). Two launches:
 *                                            the gate MLP, weights read once per 8 streams, and the row
 *                                            kernel, which overlaps it (programmatic dependent launch).
 *            cond == NULL: gate_buf [B][D] is an input (a gate computed earlier, e.g. once per tick).
 * Requirements: D % 8 == 0, Cd % 8 == 0, Hd % 8 == 0, D <= 16384, Cd, Hd <= 4096. */
int reflex_adarmsnorm(const void *x, void *y, const void *cond, const void *W1, const void *b1,
                      const void *W2, const void *b2, float *gate_buf, int B, int R, int D, int Cd,
                      int Hd, float eps, int dtype, void *stream);

/* Eq. 2, the part that does not depend on x: gamma_l(c) = 1 + W2_l SiLU(W1_l c + b1_l) + b2_l for every stream and
 * for L layers at once (the layers' parameters stacked along a leading axis), fp32, into gate_buf.
 * c = [emb(t_k), s_t] is fixed for a whole denoising step and known before any layer's input exists, so the gates of
 * all layers of the step can be produced by one call (two launches whatever L is) ahead of the layer loop; each
 * layer then calls reflex_adarmsnorm with cond == NULL and its slice gate_buf + l*B*D. L = 1 is the single-layer case.
 *   cond [B][Cd]; W1 [L][Hd][Cd], b1 [L][Hd], W2 [L][D][Hd], b2 [L][D]   device, dtype
 *   gate_buf  device fp32, L*B*(D+Hd) floats: gates [L][B][D] first, then scratch for the hidden activations
 * Requirements: D % 8 == 0, Cd and Hd multiples of 8 in [8, 1024], 1 <= L <= 65535. Widths above 632 do not fit the
 * staged kernels' shared memory and take a per-stream kernel, one launch per layer.
 * bf16 with Cd, Hd multiples of 16 up to 320 runs on the tensor cores; should one of that kernel's bounded waits run
 * out, its part of the gates is written as NaN (there is no cache handle to carry a status word), so the failure
 * shows in everything computed from them. */
int reflex_adarmsnorm_gate(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2,
                           float *gate_buf, int L, int B, int D, int Cd, int Hd, int dtype, void *stream);

/* No counterpart in the paper: a convenience for callers that cannot hand the library any scratch memory.
 * Same result as reflex_adarmsnorm(x, y, cond, W1, b1, W2, b2, gate_buf, ...) with a gate_buf, but the gate
 * and hidden-layer scratch lives in an array built into the library image (96 Ki floats = 384 KiB of device
 * memory on every GPU that loads the library, held until the process exits), so nothing is allocated: not by
 * this call, not by the caller. Meant for code that must not call cudaMalloc where it runs -- a control loop
 * with a latency bound (an allocation can synchronise the whole device), a plug-in inside a host program that
 * owns all device memory through its own pool, a callback that may not block -- and that has no spare buffer
 * of its own to lend.
 *   Limit: B*(D+Hd) <= 98304 floats and D <= 2048 (e.g. 64 streams x (1024 + 256)); larger shapes return
 *   REFLEX_ERR_SHAPE and must use reflex_adarmsnorm with a caller-provided gate_buf.
 *   The first call on each device looks up the array's device address (with that device current); make that
 *   first call outside any stream capture.
 *   All calls on a device share the one array and it keeps the previous call's contents (every value that is read
 *   is rewritten first, nothing needs clearing): two calls that overlap on the GPU, e.g. on different streams, race.
 *   x, y, cond, W1, b1, W2, b2, B, R, D, Cd, Hd, eps, dtype, stream: as in reflex_adarmsnorm; cond is required. */
int reflex_adarmsnorm_noalloc(const void *x, void *y, const void *cond, const void *W1, const void *b1,
                              const void *W2, const void *b2, int B, int R, int D, int Cd, int Hd, float eps,
                              int dtype, void *stream);

/* Sec. 3.3 "System Optimizations" (the query, key and value projections as one packed matrix W_QKV = [W_Q; W_K; W_V])
 * with the adaptive norm of Eq. 2 folded in (Sec. 4 "Operator Fusion Impact": the norm combined with the linear layer
 * after it, the norm output never written to memory). For every row r of stream b:
 *   y = x[r] / RMS(x[r]) * gamma_b,   [q | k_dyn | v_dyn][r] = W_QKV y
 * One launch; the outputs have the layouts reflex_partitioned_attention reads.
 *   cache    a cache whose status word records a device-side wait that ran out (reflex_cache_check_status), or NULL
 *   x        device [B][R][D] dtype
 *   gate     device fp32 [B][D]: gamma of every stream, as reflex_adarmsnorm_gate writes it
 *   Wqkv     device [(Hq + 2 Hkv) d][D] dtype: one row per output feature; rows of W_Q (head-major) first, then W_K, then W_V
 *   q        device [B][R][Hq][d] dtype;   k_dyn, v_dyn  device [B][R][Hkv][d] dtype   (written; all rows)
 *   impl     0: tensor cores when dtype is bf16, D % 64 == 0 and the gates of the streams under 128 consecutive rows fit in
 *               shared memory ((127 / R + 2) * D * 4 bytes <= 64 KiB), else the plain kernel; 1: the plain kernel (fp32 FMAs);
 *               2: like 0 but never the 512-column tiles that 0 picks for large problems
 * Arithmetic on the tensor-core path: products of bf16(x * gamma) and W_QKV accumulated in fp32, the row's 1/RMS applied
 * to the accumulator, one rounding to bf16 at the end.
 * Requirements: D % 8 == 0, D <= 8192; d % 8 == 0; Hq % Hkv == 0; (Hq + 2 Hkv) d <= 65536; 16-byte aligned pointers.
 * Errors: REFLEX_ERR_INVALID_ARG (NULL pointer, unknown dtype or impl, eps < 0), REFLEX_ERR_SHAPE, REFLEX_ERR_ALIGN;
 * nothing is launched and nothing written on error. */
int reflex_adarmsnorm_qkv(reflex_cache_t *cache, const void *x, const float *gate, const void *Wqkv, void *q,
                          void *k_dyn, void *v_dyn, int B, int R, int D, int Hq, int Hkv, int d, float eps,
                          int dtype, int impl, void *stream);

/* Sec. 3.3 "System Optimizations" (the Gate and Up projections of a SwiGLU block combined into one kernel), again with the
 * adaptive norm of Eq. 2 folded in. For every row r of stream b:
 *   y = x[r] / RMS(x[r]) * gamma_b,   h[r] = SiLU(W_gate y) * (W_up y),   SiLU(z) = z / (1 + e^-z)
 * One launch; neither y nor the two projections reach memory.
 *   cache    as in reflex_adarmsnorm_qkv (status word), or NULL
 *   x        device [B][R][D] dtype;   gate  device fp32 [B][D]
 *   Wgu      device [2F][D] dtype: rows [0, F) = W_gate, rows [F, 2F) = W_up (row f of each = hidden feature f)
 *   h        device [B][R][F] dtype (written)
 *   impl     0: tensor cores when dtype is bf16, D % 64 == 0 and (127 / R + 2) * D * 4 bytes <= 28 KiB, else the plain
 *               kernel; 1: the plain kernel
 * Arithmetic on the tensor-core path: as reflex_adarmsnorm_qkv; both fp32 accumulators are scaled by 1/RMS, the activation
 * and the product are computed in fp32 and rounded to bf16 once.
 * Requirements: D % 8 == 0, D <= 8192; F % 8 == 0; 16-byte aligned pointers. Errors as reflex_adarmsnorm_qkv. */
int reflex_adarmsnorm_swiglu(reflex_cache_t *cache, const void *x, const float *gate, const void *Wgu, void *h,
                             int B, int R, int D, int F, float eps, int dtype, int impl, void *stream);

/* Sec. 3.3 "System Optimizations" lists the linear layers of the action expert; the two that close a residual branch --
 * the attention output projection and the down projection of the SwiGLU block -- are this call:
 *   out[r][n] = res[r][n] + sum_i a[r][i] * W[n][i]
 * One launch; products of bf16 operands accumulated in fp32, the residual added in fp32, one rounding to dtype.
 *   cache    a cache whose status word records a device-side wait that ran out (reflex_cache_check_status), or NULL
 *            (without a cache such a failure shows as NaN in the tile it hit)
 *   a        device [M][K] dtype (M = streams x tokens)
 *   W        device [N][K] dtype: one row per output feature
 *   res      device [M][N] dtype, or NULL for a projection without residual
 *   out      device [M][N] dtype (written); may be the same buffer as res (in-place update of the residual stream),
 *            must not overlap a
 *   impl     0: tensor cores when dtype is bf16 (256 x 256 output tiles per pair of SMs; 256 x 128 where those would leave
 *               most pairs idle, a contraction of 4096 or more then split over two pairs of a cluster while they fit;
 *               a kernel with the weights as the stationary operand when K % 64 == 0 and M <= 128, or M <= 256 in groups
 *               of 64 rows for K >= 2048),
 *               else the plain kernel; 1: the plain kernel (fp32 FMAs, K <= 12288); 2: like 0 but always the 256-row tiles
 * Requirements: K % 8 == 0, 8 <= K <= 12288; N % 8 == 0; 16-byte aligned pointers.
 * Errors: REFLEX_ERR_INVALID_ARG (NULL pointer, unknown dtype or impl, out == a), REFLEX_ERR_SHAPE, REFLEX_ERR_ALIGN;
 * nothing is launched and nothing written on error. */
int reflex_linear_residual(reflex_cache_t *cache, const void *a, const void *W, const void *res, void *out, int M,
                           int K, int N, int dtype, int impl, void *stream);

/* Eq. 1 / App. A Prop. 1: for every stream b, KV head j and its G*T query rows,
 *   out = softmax(scale * Q [K_pin; K_slide; K_dyn]^T) [V_pin; V_slide; V_dyn]
 * over static rows [0, static_len[b]), the live ring slots (physical order; softmax does not depend
 * on key order) and the T dynamic tokens, which are read from k_dyn/v_dyn in place and are new at
 * every denoising step. Cached regions are only read.
 *   q, out         device [B][T][Hq][d] dtype
 *   k_dyn, v_dyn   device [B][T][Hkv][d] dtype
 *   T              1..T_max
 *   scale          <= 0 selects 1/sqrt(d)
 *   dyn_mask       0: every query sees all T dynamic keys (Eq. 1 as printed);
 *                  1: dynamic key j hidden from dynamic query i when j > i (causal suffix, Prop. 1)
 * Calls on one cache must be ordered on a single stream (or by events): when the keys are split, all layers share the
 * cache's one area of partial results in the workspace, and two calls that overlap on the GPU would race in it.
 * Kernel attributes are set up the first time a kernel is used on each device, so one process may drive several
 * devices (each with its own caches). */
int reflex_partitioned_attention(reflex_cache_t *cache, int layer, const void *q, const void *k_dyn,
                                 const void *v_dyn, void *out, int T, float scale, int dyn_mask,
                                 void *stream);

/* Sec. 2.1 / App. C: forward Euler step k of K of the flow ODE, x <- x + dt * v with dt = -1/K
 * (t runs from 1 to 0).
 *   x       device [B][T][A] fp32 master copy, updated in place
 *   v       device [B][T][A] dtype
 *   x_lowp  device [B][T][A] dtype mirror of the updated x, or NULL
 *   k, K    0 <= k < K (k only validated: dt does not depend on it) */
int reflex_flow_step(void *x, const void *v, void *x_lowp, int B, int T, int A, int k, int K,
                     int dtype, void *stream);

/* ---- Sec. 3.4 "Stream Throughput: Asynchronous Pipeline", Algorithm 1 (future-conditional overlap scheduling), Eq. 3 ----
 * Host logic only; no device work. A control loop calls reflex_overlap_tick once per control period:
 *   - the event names the action to execute (chunk index, position in the chunk; Algorithm 1 line 5);
 *   - launch_now = 1 on the tick of action C - K (1-based; line 6), K = ceil(mean inference latency / control period)
 *     fixed at the start of the chunk (line 3) from the last 8 measured latencies (the initial estimate before the
 *     first) and clamped to [0, C - 1]: the caller then starts the next chunk's inference conditioned on the action
 *     just commanded (Eq. 3: s_hat = a_cmd) and reports its completion with reflex_overlap_inference_done;
 *   - when a chunk is used up and the next has not been reported, the tick is a stall (stalled = 1, the last action
 *     is held) and the loop resumes with the first action of the new chunk on the first tick after the report.
 * reflex_overlap_simulate runs the same policy over a trace of inference latencies in continuous time (one loop
 * iteration = one control period, the launch at the end of the period of action C - K) and returns stall and
 * staleness figures; mode 0 = adaptive K (Algorithm 1), 1 = synchronous (inference only after the chunk has ended),
 * 2 = fixed K. Errors: REFLEX_ERR_INVALID_ARG, REFLEX_ERR_STATE (completion reported with nothing in flight). */
typedef struct reflex_overlap reflex_overlap_t;
typedef struct reflex_overlap_event {
    int32_t chunk, action;      /* chunk index (from 0) and 0-based position of the action executed on this tick */
    int32_t launch_now;         /* start the next chunk's inference now */
    int32_t stalled;            /* no action available: the previous one is held */
    int32_t lookahead;          /* K of the current chunk */
    int32_t reserved;
    int64_t stalls_total;       /* stalled ticks so far */
} reflex_overlap_event;
typedef struct reflex_overlap_stats {
    int64_t chunks, stall_ticks;            /* chunks executed; control periods lost waiting (each stall rounded up) */
    double stall_time_s, total_time_s;      /* time lost waiting; time until the last chunk's successor is available */
    double mean_staleness_s;                /* mean age of the conditioning state when a chunk's first action runs */
    double mean_lookahead;
    int32_t min_lookahead, max_lookahead;
} reflex_overlap_stats;
int reflex_overlap_create(int C, double tau_step_s, double tau_inf_init_s, reflex_overlap_t **out);
int reflex_overlap_destroy(reflex_overlap_t *sched);
int reflex_overlap_tick(reflex_overlap_t *sched, reflex_overlap_event *ev);
int reflex_overlap_inference_done(reflex_overlap_t *sched, double latency_s);
int reflex_overlap_simulate(int C, double tau_step_s, double tau_inf_init_s, const double *tau_inf_s, int n_chunks,
                            int mode, int fixed_K, reflex_overlap_stats *out);

#ifdef __cplusplus
}
#endif
#endif /* REFLEX_H */
