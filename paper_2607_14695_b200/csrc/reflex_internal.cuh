// Internal declarations shared by the translation units of libreflex_b200 (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cuda.h>

#include <atomic>

#include "reflex.h"

namespace reflex {

// Per-stream cache state as the kernels read it (device memory, one int4-sized record per stream).
struct StreamState {
    int32_t static_len;  // valid prefix rows, -1 = never initialised
    int32_t head;        // next ring slot to write
    int32_t count;       // live ring tokens
    int32_t ticket;      // arrival counter of the append kernel (always 0 between launches)
    int32_t bank;        // which static bank attention reads (0 unless the cache has two banks)
    int32_t staged_len;  // rows written to the other bank by the last stage call, -1 = nothing staged
};

// Layout of the caller-lent workspace.
struct WorkspaceLayout {
    size_t state_off;     // StreamState[B]
    size_t total_off;     // int64 total_appended[B]
    size_t status_off;    // uint32 status word (bounded-wait failures)
    size_t partial_off;   // split-K partials
    size_t partial_bytes;
    size_t bytes;
};

constexpr int kMaxSplits = 32;
constexpr int kStreamsPerLaunch = 64;  // stream ids / lengths passed by value per launch

struct StreamBatch {
    int32_t id[kStreamsPerLaunch];
    int32_t len[kStreamsPerLaunch];
};

WorkspaceLayout workspace_layout(const reflex_cache_desc &d);

inline size_t elem_size(int dtype) { return dtype == REFLEX_DTYPE_BF16 ? 2 : 4; }

// Geometry every attention kernel needs.
struct AttnParams {
    const void *k_slab, *v_slab;   // [L][B][S_max+N][Hkv][d]
    const void *q, *k_dyn, *v_dyn; // [B][T][Hq][d], [B][T][Hkv][d]
    void *out;
    const StreamState *state;
    float *partials;               // split-K scratch
    int L, B, Hq, Hkv, d, S_max, N, T, layer;
    int ring_off;                  // first ring row of a (layer, stream) block: S_max times the number of static banks
    int dyn_mask;
    float scale;
    int nsplit;
    int dtype;
};

// Split-K partials in the workspace: for n = B * rows * nsplit (row, split) slots, first n rows of d floats with the
// unnormalised O (16-byte aligned), then n (m, l) pairs (m in natural-log units; m = -inf, l = 0 for an empty slice).
__host__ __device__ inline size_t partial_slot(int b, int rows, int r, int nsplit, int s) { return ((size_t)b * rows + r) * nsplit + s; }
__host__ __device__ inline float *partial_o(float *base, size_t slot, int d) { return base + slot * (size_t)d; }
__host__ __device__ inline float *partial_ml(float *base, size_t n_slots, size_t slot, int d) { return base + n_slots * (size_t)d + slot * 2; }

// Records a failure for reflex_last_error_string() and returns `code` (printf-style message).
int api_fail(int code, const char *fmt, ...);

// Kernel attributes (the dynamic shared-memory limit) belong to a device's context, not to the process: a launcher runs its
// set-up the first time it is used on each device. `done` is the launcher's function-local bit mask of devices (ordinals
// modulo 64); several host threads may race to run the same idempotent set-up.
template <typename F>
inline cudaError_t once_per_device(std::atomic<unsigned long long> &done, F &&setup)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
    e = setup();
    if (e != cudaSuccess) return e;
    done.fetch_or(bit, std::memory_order_release);
    return cudaSuccess;
}

// Number of kernels this library has launched in this process (every launcher bumps it).
void count_launch(int n = 1);

// ---- launchers (each returns the cudaError_t of its launch) ----
cudaError_t launch_state_init(StreamState *state, int64_t *total, uint32_t *status, const int32_t *head0_dev_or_null,
                              int B, int N, cudaStream_t st);
cudaError_t launch_init_static(void *k_slab, void *v_slab, const void *k_src, const void *v_src, StreamState *state,
                               const StreamBatch &batch, int n, int src_stream0, int L, int B, int S_max, int ring_off, int N, int S_src, int to_other_bank,
                               size_t row_bytes, cudaStream_t st);
cudaError_t launch_wait_limit_probe(uint32_t *status, unsigned long long limit_ns, cudaStream_t st);
cudaError_t launch_commit_static(StreamState *state, const StreamBatch &batch, int n, cudaStream_t st);
cudaError_t launch_append_sliding(void *k_slab, void *v_slab, const void *k_src, const void *v_src, StreamState *state,
                                  int64_t *total, const StreamBatch &batch, int n, int src_stream0, int L, int B, int ring_off,
                                  int N, int m, size_t row_bytes, cudaStream_t st);
cudaError_t launch_adarmsnorm(const void *x, void *y, const void *cond, const void *W1, const void *b1, const void *W2,
                              const void *b2, float *gate_buf, int B, int R, int D, int Cd, int Hd, float eps, int dtype,
                              cudaStream_t st);
cudaError_t launch_adarmsnorm_gate(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2, float *gate_buf,
                                   int L, int B, int D, int Cd, int Hd, int dtype, cudaStream_t st);
cudaError_t launch_flow_step(float *x, const void *v, void *x_lowp, size_t n, float dt, int dtype, cudaStream_t st);
cudaError_t launch_attention_simt(const AttnParams &p, cudaStream_t st);
int simt_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count);
cudaError_t launch_attention_merge(const AttnParams &p, cudaStream_t st);  // combines nsplit (m, l, acc) partials
bool tc_supported(const AttnParams &p);
bool tensor_map_2d_bf16(CUtensorMap *out, const void *ptr, int inner, int rows, int box_rows);
int tc_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count);
bool tc2_supported(const AttnParams &p);
int tc2_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count);
cudaError_t launch_attention_tc(const AttnParams &p, uint32_t *status, bool two_cta, int sm_count, cudaStream_t st);
// gate MLP of AdaRMSNorm on tcgen05 (bf16): false when the shapes or the driver do not allow it (the caller falls back)
// adaptive norm + packed Q/K/V projection (qkv_tc.cu). impl: 0 = tensor cores where supported, 1 = plain kernel,
// 2 = tensor cores with 256-column tiles only
bool norm_qkv_tc_supported(int dtype, int B, int R, int D, int nq, int nk);
// swiglu_F > 0: W = [W_gate; W_up] and q receives SiLU(gate) * up, [B*R][F]
cudaError_t launch_adarmsnorm_qkv(const void *x, const float *gate, const void *W, void *q, void *k, void *v, int B, int R, int D, int nq, int nk,
                                  int swiglu_F, float eps, int dtype, int impl, int sm_count, uint32_t *status, cudaStream_t st);
// plain projection with residual (linear_tc.cu): out [M][N] = res + a [M][K] W [N][K]^T. impl: 0 = tensor cores where supported,
// 1 = plain kernel, 2 = tensor cores with 256-row tiles whatever M is
cudaError_t launch_linear_residual(const void *a, const void *W, const void *res, void *out, int M, int K, int N, int dtype, int impl,
                                   uint32_t *status, cudaStream_t st);
bool linear_small_takes(int M, int K, int N);
cudaError_t launch_linear_small(const void *a, const void *W, const void *res, void *out, int M, int K, int N, uint32_t *status, cudaStream_t st);
bool gate_tc_supported(int B, int D, int Cd, int Hd);
cudaError_t launch_gate_tc(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2, float *gate_buf, int L, int B,
                           int D, int Cd, int Hd, cudaStream_t st);

}  // namespace reflex
