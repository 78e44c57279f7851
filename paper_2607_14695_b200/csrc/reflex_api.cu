// Host side of the C ABI declared in reflex.h: argument validation, the host mirror of the ring state,
// kernel selection and launches. No call below allocates device memory.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "reflex_internal.cuh"

using namespace reflex;

struct reflex_cache {
    reflex_cache_desc desc;
    void *k_slab, *v_slab;
    char *ws;
    WorkspaceLayout lay;
    std::vector<int32_t> static_len, head, count;
    std::vector<int64_t> total;
    std::vector<int32_t> staged_len;   // host mirror of the length staged in the other static bank, -1 = none
    int attn_impl;
    int sm_count;
};

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t e, const char *what)
{
    return fail(REFLEX_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool desc_ok(const reflex_cache_desc *d)
{
    if (!d) return false;
    if (d->L < 1 || d->B < 1 || d->Hq < 1 || d->Hkv < 1 || d->N < 1 || d->T_max < 1 || d->S_max < 0) return false;
    if (d->Hq % d->Hkv != 0) return false;
    if (!(d->d == 32 || d->d == 64 || d->d == 128 || d->d == 256)) return false;
    if (d->dtype != REFLEX_DTYPE_BF16 && d->dtype != REFLEX_DTYPE_F32) return false;
    if (d->static_banks < 0 || d->static_banks > 2) return false;
    return true;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline int ring_off(const reflex_cache_desc &d) { return (d.static_banks == 2 ? 2 : 1) * d.S_max; }

int check_stream_ids(const reflex_cache *c, const int32_t *ids, int n)
{
    if (!ids) return fail(REFLEX_ERR_INVALID_ARG, "stream_ids is NULL");
    if (n < 1 || n > c->desc.B) return fail(REFLEX_ERR_SHAPE, "n_streams=%d outside [1, B=%d]", n, c->desc.B);
    std::vector<char> seen(c->desc.B, 0);
    for (int i = 0; i < n; ++i) {
        if (ids[i] < 0 || ids[i] >= c->desc.B) return fail(REFLEX_ERR_INVALID_ARG, "stream id %d outside [0, %d)", ids[i], c->desc.B);
        if (seen[ids[i]]) return fail(REFLEX_ERR_INVALID_ARG, "stream id %d listed twice", ids[i]);
        seen[ids[i]] = 1;
    }
    return REFLEX_OK;
}

}  // namespace

namespace reflex {

int api_fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

WorkspaceLayout workspace_layout(const reflex_cache_desc &d)
{
    WorkspaceLayout w;
    size_t off = 0;
    w.state_off = off;  off = align_up(off + sizeof(StreamState) * (size_t)d.B, 256);
    w.total_off = off;  off = align_up(off + sizeof(int64_t) * (size_t)d.B, 256);
    w.status_off = off; off = align_up(off + 256, 256);
    // split-K partials: (m, l, acc[d]) fp32 per (stream, query row, split)
    const size_t rows = (size_t)d.T_max * d.Hq;
    const size_t blocks = ((rows + 3) / 4) * (size_t)d.B;
    size_t splits = (8 * 148 + blocks - 1) / blocks;
    if (splits < 2) splits = 2;     // the batched two-CTA kernel may split the keys when streams alone do not fill the SM pairs
    if (d.Hkv > 0 && d.Hq % d.Hkv == 0 && d.Hq / d.Hkv <= 128) {
        // ... up to one unit per SM pair: (stream, KV head, pair of query tiles) units times key slices
        const size_t tile_tokens = 128 / (size_t)(d.Hq / d.Hkv);
        const size_t units = (((size_t)d.T_max + tile_tokens - 1) / tile_tokens + 1) / 2 * (size_t)d.Hkv * (size_t)d.B;
        const size_t fill = units > 0 ? 74 / units : 0;
        if (fill > splits) splits = fill;
    }
    if (splits > (size_t)kMaxSplits) splits = kMaxSplits;
    w.partial_off = off;
    w.partial_bytes = align_up(splits * (size_t)d.B * rows * (size_t)(d.d + 2) * sizeof(float), 256);
    off += w.partial_bytes;
    w.bytes = off;
    return w;
}

}  // namespace reflex

extern "C" {

const char *reflex_last_error_string(void) { return g_err; }
const char *reflex_version(void) { return "reflex-b200 0.1 (sm_100a)"; }
unsigned long long reflex_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t reflex_cache_slab_bytes(const reflex_cache_desc *d)
{
    if (!desc_ok(d)) return 0;
    return (size_t)d->L * d->B * (size_t)(ring_off(*d) + d->N) * d->Hkv * d->d * elem_size(d->dtype);
}

size_t reflex_workspace_bytes(const reflex_cache_desc *d)
{
    if (!desc_ok(d)) return 0;
    return workspace_layout(*d).bytes;
}

int reflex_cache_create(const reflex_cache_desc *desc, void *k_slab, void *v_slab, void *workspace,
                        const int32_t *ring_head0, void *stream, reflex_cache_t **out)
{
    if (!out) return fail(REFLEX_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!desc_ok(desc)) return fail(REFLEX_ERR_SHAPE, "invalid cache descriptor (need Hq %% Hkv == 0, d in {32,64,128,256}, sizes >= 1)");
    if (!k_slab || !v_slab || !workspace) return fail(REFLEX_ERR_INVALID_ARG, "k_slab, v_slab and workspace must be non-NULL");
    if (!aligned16(k_slab) || !aligned16(v_slab) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(REFLEX_ERR_ALIGN, "slabs must be 16-byte aligned and the workspace 256-byte aligned");
    if (ring_head0)
        for (int b = 0; b < desc->B; ++b)
            if (ring_head0[b] < 0 || ring_head0[b] >= desc->N)
                return fail(REFLEX_ERR_INVALID_ARG, "ring_head0[%d]=%d outside [0, N=%d)", b, ring_head0[b], desc->N);
    reflex_cache *c = new (std::nothrow) reflex_cache();
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "out of host memory");
    c->desc = *desc;
    c->k_slab = k_slab; c->v_slab = v_slab; c->ws = (char *)workspace;
    c->lay = workspace_layout(*desc);
    c->static_len.assign(desc->B, -1);
    c->staged_len.assign(desc->B, -1);
    c->head.assign(desc->B, 0);
    c->count.assign(desc->B, 0);
    c->total.assign(desc->B, 0);
    if (ring_head0) for (int b = 0; b < desc->B; ++b) c->head[b] = ring_head0[b];
    c->attn_impl = REFLEX_ATTN_AUTO;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "device query"); }
    cudaStream_t st = (cudaStream_t)stream;
    // initial ring positions travel through the (not yet used) partial area
    int32_t *head0_dev = nullptr;
    if (ring_head0) {
        head0_dev = (int32_t *)(c->ws + c->lay.partial_off);
        e = cudaMemcpyAsync(head0_dev, ring_head0, sizeof(int32_t) * (size_t)desc->B, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) { delete c; return cuda_fail(e, "copy of ring_head0"); }
    }
    e = launch_state_init((StreamState *)(c->ws + c->lay.state_off), (int64_t *)(c->ws + c->lay.total_off),
                          (uint32_t *)(c->ws + c->lay.status_off), head0_dev, desc->B, desc->N, st);
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "state init launch"); }
    *out = c;
    return REFLEX_OK;
}

int reflex_cache_destroy(reflex_cache_t *c)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    delete c;
    return REFLEX_OK;
}

int reflex_cache_get_state(reflex_cache_t *c, int32_t *static_len, int32_t *head, int32_t *count,
                           int64_t *total_appended, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    const int B = c->desc.B;
    std::vector<StreamState> s(B);
    std::vector<int64_t> tot(B);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(s.data(), c->ws + c->lay.state_off, sizeof(StreamState) * (size_t)B, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(tot.data(), c->ws + c->lay.total_off, sizeof(int64_t) * (size_t)B, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "state read-back");
    for (int b = 0; b < B; ++b) {
        c->static_len[b] = s[b].static_len; c->head[b] = s[b].head; c->count[b] = s[b].count; c->total[b] = tot[b];
        c->staged_len[b] = s[b].staged_len;
        if (static_len) static_len[b] = s[b].static_len;
        if (head) head[b] = s[b].head;
        if (count) count[b] = s[b].count;
        if (total_appended) total_appended[b] = tot[b];
    }
    return REFLEX_OK;
}

int reflex_cache_slot_map(reflex_cache_t *c, int b, int32_t *slot_of_age)
{
    if (!c || !slot_of_age) return fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (b < 0 || b >= c->desc.B) return fail(REFLEX_ERR_INVALID_ARG, "stream %d outside [0, %d)", b, c->desc.B);
    const int N = c->desc.N;
    for (int j = 0; j < N; ++j) {
        if (j < c->count[b]) {
            int s = (c->head[b] - c->count[b] + j) % N;
            if (s < 0) s += N;
            slot_of_age[j] = s;
        } else {
            slot_of_age[j] = -1;
        }
    }
    return REFLEX_OK;
}

int reflex_cache_check_status(reflex_cache_t *c, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    uint32_t word = 0;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(&word, c->ws + c->lay.status_off, sizeof(word), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "status read-back");
    if (word != 0u)
        return fail(REFLEX_ERR_TIMEOUT, "a device-side wait ran out (status 0x%08x: wait site %u, block %u); results of that launch are invalid",
                    word, (word >> 16) & 0x7FFFu, word & 0xFFFFu);
    return REFLEX_OK;
}

int reflex_cache_selftest_wait_limit(reflex_cache_t *c, int limit_us, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    if (limit_us < 1 || limit_us > 100000) return fail(REFLEX_ERR_INVALID_ARG, "limit_us=%d outside [1, 100000]", limit_us);
    cudaError_t e = launch_wait_limit_probe((uint32_t *)(c->ws + c->lay.status_off), (unsigned long long)limit_us * 1000ull, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "wait-limit probe launch");
    return REFLEX_OK;
}

int reflex_cache_set_attention_impl(reflex_cache_t *c, int impl)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    if (impl != REFLEX_ATTN_AUTO && impl != REFLEX_ATTN_SIMT && impl != REFLEX_ATTN_TC && impl != REFLEX_ATTN_TC2)
        return fail(REFLEX_ERR_INVALID_ARG, "unknown attention implementation %d", impl);
    c->attn_impl = impl;
    return REFLEX_OK;
}

static int write_static(reflex_cache_t *c, const int32_t *stream_ids, int n_streams, const void *k_static, const void *v_static, int S_src,
                        const int32_t *S, int to_other_bank, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    int rc = check_stream_ids(c, stream_ids, n_streams);
    if (rc) return rc;
    const reflex_cache_desc &d = c->desc;
    if (to_other_bank && d.static_banks != 2) return fail(REFLEX_ERR_STATE, "the cache was created with one static bank (static_banks = 2 needed)");
    if (S_src < 0) return fail(REFLEX_ERR_SHAPE, "S_src=%d is negative", S_src);
    bool any = false;
    for (int i = 0; i < n_streams; ++i) {
        const int s = S ? S[i] : S_src;
        if (s < 0 || s > d.S_max || s > S_src)
            return fail(REFLEX_ERR_SHAPE, "S[%d]=%d outside [0, min(S_src=%d, S_max=%d)]", i, s, S_src, d.S_max);
        any |= s > 0;
    }
    if (any && (!k_static || !v_static)) return fail(REFLEX_ERR_INVALID_ARG, "k_static / v_static is NULL");
    if (!aligned16(k_static) || !aligned16(v_static)) return fail(REFLEX_ERR_ALIGN, "k_static / v_static not 16-byte aligned");
    const size_t row_bytes = (size_t)d.Hkv * d.d * elem_size(d.dtype);
    cudaStream_t st = (cudaStream_t)stream;
    for (int i0 = 0; i0 < n_streams; i0 += kStreamsPerLaunch) {
        const int n = (n_streams - i0 < kStreamsPerLaunch) ? n_streams - i0 : kStreamsPerLaunch;
        StreamBatch batch;
        memset(&batch, 0, sizeof(batch));
        for (int i = 0; i < n; ++i) { batch.id[i] = stream_ids[i0 + i]; batch.len[i] = S ? S[i0 + i] : S_src; }
        cudaError_t e = launch_init_static(c->k_slab, c->v_slab, k_static, v_static, (StreamState *)(c->ws + c->lay.state_off),
                                           batch, n, i0, d.L, d.B, d.S_max, ring_off(d), d.N, S_src, to_other_bank, row_bytes, st);
        if (e != cudaSuccess) return cuda_fail(e, "init_static launch");
        for (int i = 0; i < n; ++i) (to_other_bank ? c->staged_len : c->static_len)[batch.id[i]] = batch.len[i];
    }
    return REFLEX_OK;
}

int reflex_cache_init_static(reflex_cache_t *c, const int32_t *stream_ids, int n_streams, const void *k_static,
                             const void *v_static, int S_src, const int32_t *S, void *stream)
{
    return write_static(c, stream_ids, n_streams, k_static, v_static, S_src, S, 0, stream);
}

int reflex_cache_stage_static(reflex_cache_t *c, const int32_t *stream_ids, int n_streams, const void *k_static,
                              const void *v_static, int S_src, const int32_t *S, void *stream)
{
    return write_static(c, stream_ids, n_streams, k_static, v_static, S_src, S, 1, stream);
}

int reflex_cache_commit_static(reflex_cache_t *c, const int32_t *stream_ids, int n_streams, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    int rc = check_stream_ids(c, stream_ids, n_streams);
    if (rc) return rc;
    if (c->desc.static_banks != 2) return fail(REFLEX_ERR_STATE, "the cache was created with one static bank (static_banks = 2 needed)");
    for (int i = 0; i < n_streams; ++i)
        if (c->staged_len[stream_ids[i]] < 0) return fail(REFLEX_ERR_STATE, "stream %d: nothing staged", stream_ids[i]);
    cudaStream_t st = (cudaStream_t)stream;
    for (int i0 = 0; i0 < n_streams; i0 += kStreamsPerLaunch) {
        const int n = (n_streams - i0 < kStreamsPerLaunch) ? n_streams - i0 : kStreamsPerLaunch;
        StreamBatch batch;
        memset(&batch, 0, sizeof(batch));
        for (int i = 0; i < n; ++i) batch.id[i] = stream_ids[i0 + i];
        cudaError_t e = launch_commit_static((StreamState *)(c->ws + c->lay.state_off), batch, n, st);
        if (e != cudaSuccess) return cuda_fail(e, "commit_static launch");
        for (int i = 0; i < n; ++i) { c->static_len[batch.id[i]] = c->staged_len[batch.id[i]]; c->staged_len[batch.id[i]] = -1; }
    }
    return REFLEX_OK;
}

int reflex_cache_append_sliding(reflex_cache_t *c, const int32_t *stream_ids, int n_streams, const void *k_new,
                                const void *v_new, int m, int32_t *evicted, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    int rc = check_stream_ids(c, stream_ids, n_streams);
    if (rc) return rc;
    const reflex_cache_desc &d = c->desc;
    if (m < 1 || m > d.N) return fail(REFLEX_ERR_SHAPE, "m=%d outside [1, N=%d]", m, d.N);
    if (!k_new || !v_new) return fail(REFLEX_ERR_INVALID_ARG, "k_new / v_new is NULL");
    if (!aligned16(k_new) || !aligned16(v_new)) return fail(REFLEX_ERR_ALIGN, "k_new / v_new not 16-byte aligned");
    const size_t row_bytes = (size_t)d.Hkv * d.d * elem_size(d.dtype);
    cudaStream_t st = (cudaStream_t)stream;
    for (int i0 = 0; i0 < n_streams; i0 += kStreamsPerLaunch) {
        const int n = (n_streams - i0 < kStreamsPerLaunch) ? n_streams - i0 : kStreamsPerLaunch;
        StreamBatch batch;
        memset(&batch, 0, sizeof(batch));
        for (int i = 0; i < n; ++i) batch.id[i] = stream_ids[i0 + i];
        cudaError_t e = launch_append_sliding(c->k_slab, c->v_slab, k_new, v_new, (StreamState *)(c->ws + c->lay.state_off),
                                              (int64_t *)(c->ws + c->lay.total_off), batch, n, i0, d.L, d.B, ring_off(d), d.N, m,
                                              row_bytes, st);
        if (e != cudaSuccess) return cuda_fail(e, "append_sliding launch");
        for (int i = 0; i < n; ++i) {
            const int b = batch.id[i];
            const int over = c->count[b] + m - d.N;
            if (evicted) evicted[i0 + i] = over > 0 ? over : 0;
            c->head[b] = (c->head[b] + m) % d.N;
            c->count[b] = (c->count[b] + m < d.N) ? c->count[b] + m : d.N;
            c->total[b] += m;
        }
    }
    return REFLEX_OK;
}

int reflex_adarmsnorm(const void *x, void *y, const void *cond, const void *W1, const void *b1, const void *W2,
                      const void *b2, float *gate_buf, int B, int R, int D, int Cd, int Hd, float eps, int dtype,
                      void *stream)
{
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (!x || !y) return fail(REFLEX_ERR_INVALID_ARG, "x / y is NULL");
    if (!cond && !gate_buf) return fail(REFLEX_ERR_INVALID_ARG, "need cond (with the gate MLP parameters) or a precomputed gate_buf");
    if (B < 1 || R < 1) return fail(REFLEX_ERR_SHAPE, "B=%d, R=%d must be >= 1", B, R);
    if (D < 8 || D % 8 != 0 || D > 16384) return fail(REFLEX_ERR_SHAPE, "D=%d must be a multiple of 8 in [8, 16384]", D);
    if (!(eps >= 0.f)) return fail(REFLEX_ERR_INVALID_ARG, "eps must be >= 0");
    if (cond) {
        if (!W1 || !b1 || !W2 || !b2) return fail(REFLEX_ERR_INVALID_ARG, "gate MLP parameter is NULL");
        if (Cd < 8 || Cd % 8 != 0 || Cd > 4096 || Hd < 8 || Hd % 8 != 0 || Hd > 4096)
            return fail(REFLEX_ERR_SHAPE, "Cd=%d, Hd=%d must be multiples of 8 in [8, 4096]", Cd, Hd);
        if (!aligned16(cond) || !aligned16(W1) || !aligned16(W2) || !aligned16(b1) || !aligned16(b2))
            return fail(REFLEX_ERR_ALIGN, "cond / W1 / b1 / W2 / b2 not 16-byte aligned");
    }
    if (!aligned16(x) || !aligned16(y) || !aligned16(gate_buf)) return fail(REFLEX_ERR_ALIGN, "x / y / gate_buf not 16-byte aligned");
    cudaError_t e = launch_adarmsnorm(x, y, cond, W1, b1, W2, b2, gate_buf, B, R, D, Cd, Hd, eps, dtype, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "adarmsnorm launch");
    return REFLEX_OK;
}

int reflex_adarmsnorm_gate(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2, float *gate_buf,
                           int L, int B, int D, int Cd, int Hd, int dtype, void *stream)
{
    if (L < 1 || L > 65535) return fail(REFLEX_ERR_SHAPE, "L=%d must be in [1, 65535]", L);
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (!cond || !W1 || !b1 || !W2 || !b2 || !gate_buf) return fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (B < 1) return fail(REFLEX_ERR_SHAPE, "B=%d must be >= 1", B);
    if (D < 8 || D % 8 != 0 || D > 16384) return fail(REFLEX_ERR_SHAPE, "D=%d must be a multiple of 8 in [8, 16384]", D);
    if (Cd < 8 || Cd % 8 != 0 || Cd > 1024 || Hd < 8 || Hd % 8 != 0 || Hd > 1024)
        return fail(REFLEX_ERR_SHAPE, "Cd=%d, Hd=%d must be multiples of 8 in [8, 1024]", Cd, Hd);
    if (!aligned16(cond) || !aligned16(W1) || !aligned16(W2) || !aligned16(b1) || !aligned16(b2) || !aligned16(gate_buf))
        return fail(REFLEX_ERR_ALIGN, "cond / W1 / b1 / W2 / b2 / gate_buf not 16-byte aligned");
    cudaError_t e = launch_adarmsnorm_gate(cond, W1, b1, W2, b2, gate_buf, L, B, D, Cd, Hd, dtype, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "adarmsnorm gate launch");
    return REFLEX_OK;
}

int reflex_adarmsnorm_qkv(reflex_cache_t *c, const void *x, const float *gate, const void *Wqkv, void *q, void *k_dyn, void *v_dyn,
                          int B, int R, int D, int Hq, int Hkv, int d, float eps, int dtype, int impl, void *stream)
{
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (impl < 0 || impl > 2) return fail(REFLEX_ERR_INVALID_ARG, "impl must be 0 (auto), 1 (plain kernel) or 2 (tensor cores, 256-column tiles)");
    if (!x || !gate || !Wqkv || !q || !k_dyn || !v_dyn) return fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (B < 1 || R < 1 || (long long)B * R > 0x7FFFFFFF / 2) return fail(REFLEX_ERR_SHAPE, "B=%d, R=%d", B, R);
    if (D < 8 || D % 8 != 0 || D > 8192) return fail(REFLEX_ERR_SHAPE, "D=%d must be a multiple of 8 in [8, 8192]", D);
    if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || d < 8 || d % 8 != 0 || (long long)(Hq + 2 * Hkv) * d > 65536)
        return fail(REFLEX_ERR_SHAPE, "Hq=%d, Hkv=%d, d=%d: need Hq %% Hkv == 0, d a multiple of 8, (Hq + 2 Hkv) d <= 65536", Hq, Hkv, d);
    if (!(eps >= 0.f)) return fail(REFLEX_ERR_INVALID_ARG, "eps must be >= 0");
    if (!aligned16(x) || !aligned16(gate) || !aligned16(Wqkv) || !aligned16(q) || !aligned16(k_dyn) || !aligned16(v_dyn))
        return fail(REFLEX_ERR_ALIGN, "x / gate / Wqkv / q / k_dyn / v_dyn not 16-byte aligned");
    uint32_t *status = c ? (uint32_t *)(c->ws + c->lay.status_off) : nullptr;
    cudaError_t e = launch_adarmsnorm_qkv(x, gate, Wqkv, q, k_dyn, v_dyn, B, R, D, Hq * d, Hkv * d, 0, eps, dtype, impl, c ? c->sm_count : 0, status,
                                          (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "adarmsnorm qkv launch");
    return REFLEX_OK;
}

int reflex_adarmsnorm_swiglu(reflex_cache_t *c, const void *x, const float *gate, const void *Wgu, void *h, int B, int R, int D, int F,
                             float eps, int dtype, int impl, void *stream)
{
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (impl != 0 && impl != 1) return fail(REFLEX_ERR_INVALID_ARG, "impl must be 0 (auto) or 1 (plain kernel)");
    if (!x || !gate || !Wgu || !h) return fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (B < 1 || R < 1 || (long long)B * R > 0x7FFFFFFF / 2) return fail(REFLEX_ERR_SHAPE, "B=%d, R=%d", B, R);
    if (D < 8 || D % 8 != 0 || D > 8192) return fail(REFLEX_ERR_SHAPE, "D=%d must be a multiple of 8 in [8, 8192]", D);
    if (F < 8 || F % 8 != 0 || F > (1 << 20)) return fail(REFLEX_ERR_SHAPE, "F=%d must be a multiple of 8 in [8, 2^20]", F);
    if (!(eps >= 0.f)) return fail(REFLEX_ERR_INVALID_ARG, "eps must be >= 0");
    if (!aligned16(x) || !aligned16(gate) || !aligned16(Wgu) || !aligned16(h)) return fail(REFLEX_ERR_ALIGN, "x / gate / Wgu / h not 16-byte aligned");
    uint32_t *status = c ? (uint32_t *)(c->ws + c->lay.status_off) : nullptr;
    cudaError_t e = launch_adarmsnorm_qkv(x, gate, Wgu, h, nullptr, nullptr, B, R, D, 0, 0, F, eps, dtype, impl, c ? c->sm_count : 0, status,
                                          (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "adarmsnorm swiglu launch");
    return REFLEX_OK;
}

int reflex_linear_residual(reflex_cache_t *c, const void *a, const void *W, const void *res, void *out, int M, int K, int N, int dtype,
                           int impl, void *stream)
{
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (impl < 0 || impl > 2) return fail(REFLEX_ERR_INVALID_ARG, "impl must be 0 (auto), 1 (plain kernel) or 2 (tensor cores, 256-row tiles)");
    if (!a || !W || !out) return fail(REFLEX_ERR_INVALID_ARG, "NULL argument");
    if (M < 1 || (long long)M * N > 0x3FFFFFFF) return fail(REFLEX_ERR_SHAPE, "M=%d, N=%d", M, N);
    if (K < 8 || K % 8 != 0 || K > 12288) return fail(REFLEX_ERR_SHAPE, "K=%d must be a multiple of 8 in [8, 12288]", K);
    if (N < 8 || N % 8 != 0) return fail(REFLEX_ERR_SHAPE, "N=%d must be a multiple of 8", N);
    if (!aligned16(a) || !aligned16(W) || !aligned16(out) || (res && !aligned16(res))) return fail(REFLEX_ERR_ALIGN, "a / W / res / out not 16-byte aligned");
    if (a == out) return fail(REFLEX_ERR_INVALID_ARG, "out may alias res, not a");
    uint32_t *status = c ? (uint32_t *)(c->ws + c->lay.status_off) : nullptr;
    cudaError_t e = launch_linear_residual(a, W, res, out, M, K, N, dtype, impl, status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "linear residual launch");
    return REFLEX_OK;
}

int reflex_partitioned_attention(reflex_cache_t *c, int layer, const void *q, const void *k_dyn, const void *v_dyn,
                                 void *out, int T, float scale, int dyn_mask, void *stream)
{
    if (!c) return fail(REFLEX_ERR_INVALID_ARG, "cache is NULL");
    const reflex_cache_desc &d = c->desc;
    if (layer < 0 || layer >= d.L) return fail(REFLEX_ERR_INVALID_ARG, "layer=%d outside [0, %d)", layer, d.L);
    if (T < 1 || T > d.T_max) return fail(REFLEX_ERR_SHAPE, "T=%d outside [1, T_max=%d]", T, d.T_max);
    if (dyn_mask != 0 && dyn_mask != 1) return fail(REFLEX_ERR_INVALID_ARG, "dyn_mask must be 0 or 1");
    if (!q || !k_dyn || !v_dyn || !out) return fail(REFLEX_ERR_INVALID_ARG, "q / k_dyn / v_dyn / out is NULL");
    if (!aligned16(q) || !aligned16(k_dyn) || !aligned16(v_dyn) || !aligned16(out))
        return fail(REFLEX_ERR_ALIGN, "q / k_dyn / v_dyn / out not 16-byte aligned");
    if (scale != scale) return fail(REFLEX_ERR_INVALID_ARG, "scale is NaN");
    for (int b = 0; b < d.B; ++b)
        if (c->static_len[b] < 0)
            return fail(REFLEX_ERR_STATE, "stream %d: static prefix never initialised (reflex_cache_init_static, S = 0 allowed)", b);
    AttnParams p;
    p.k_slab = c->k_slab; p.v_slab = c->v_slab; p.q = q; p.k_dyn = k_dyn; p.v_dyn = v_dyn; p.out = out;
    p.state = (const StreamState *)(c->ws + c->lay.state_off);
    p.partials = (float *)(c->ws + c->lay.partial_off);
    p.L = d.L; p.B = d.B; p.Hq = d.Hq; p.Hkv = d.Hkv; p.d = d.d; p.S_max = d.S_max; p.N = d.N; p.T = T; p.layer = layer;
    p.ring_off = ring_off(d);
    p.dyn_mask = dyn_mask;
    p.scale = scale > 0.f ? scale : 1.0f / sqrtf((float)d.d);
    p.dtype = d.dtype;
    p.nsplit = 1;
    const bool tc_ok = tc_supported(p);
    const bool tc2_ok = tc2_supported(p);
    if ((c->attn_impl == REFLEX_ATTN_TC && !tc_ok) || (c->attn_impl == REFLEX_ATTN_TC2 && !tc2_ok))
        return fail(REFLEX_ERR_NOT_IMPLEMENTED, "tensor-core attention needs bf16, 128 %% (Hq/Hkv) == 0 and d in {64,128,256} (two-CTA form: {128,256})");
    cudaError_t e;
    uint32_t *status = (uint32_t *)(c->ws + c->lay.status_off);
    if (c->attn_impl == REFLEX_ATTN_SIMT || !tc_ok) {
        p.nsplit = simt_choose_splits(p, c->lay.partial_bytes, c->sm_count);
        e = launch_attention_simt(p, (cudaStream_t)stream);
    } else {
        // Batched shapes take the two-CTA kernel (with a key split when the streams alone do not fill the SM pairs);
        // a single stream or a few take one CTA per query tile with a finer key split.
        const int split2 = tc2_ok ? tc2_choose_splits(p, c->lay.partial_bytes, c->sm_count) : 0;
        const bool two = c->attn_impl == REFLEX_ATTN_TC2 || (c->attn_impl == REFLEX_ATTN_AUTO && split2 >= 1);
        p.nsplit = two ? (split2 >= 1 ? split2 : 1) : tc_choose_splits(p, c->lay.partial_bytes, c->sm_count);
        e = launch_attention_tc(p, status, two, c->sm_count, (cudaStream_t)stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "attention launch");
    return REFLEX_OK;
}

int reflex_flow_step(void *x, const void *v, void *x_lowp, int B, int T, int A, int k, int K, int dtype, void *stream)
{
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (!x || !v) return fail(REFLEX_ERR_INVALID_ARG, "x / v is NULL");
    if (B < 1 || T < 1 || A < 1) return fail(REFLEX_ERR_SHAPE, "B, T, A must be >= 1");
    if (K < 1 || k < 0 || k >= K) return fail(REFLEX_ERR_INVALID_ARG, "step k=%d outside [0, K=%d)", k, K);
    if (!aligned16(x) || !aligned16(v) || !aligned16(x_lowp)) return fail(REFLEX_ERR_ALIGN, "x / v / x_lowp not 16-byte aligned");
    const float dt = -1.0f / (float)K;
    cudaError_t e = launch_flow_step((float *)x, v, x_lowp, (size_t)B * T * A, dt, dtype, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "flow_step launch");
    return REFLEX_OK;
}

}  // extern "C"
