// Cache maintenance kernels: state initialisation, static-prefix write (Sec. 3.1) and the in-place
// sliding-ring append with circular pointer arithmetic (Sec. 3.4, App. B.2). Byte movers: rows are
// opaque 16-byte units, so one kernel serves bf16 and fp32 storage.
#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

__global__ void state_init_kernel(StreamState *state, int64_t *total, uint32_t *status, const int32_t *head0, int B, int N)
{
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) *status = 0u;
    if (b >= B) return;
    StreamState s;
    s.static_len = -1;
    int h = head0 ? head0[b] : 0;
    s.head = ((h % N) + N) % N;
    s.count = 0;
    s.ticket = 0;
    s.bank = 0;
    s.staged_len = -1;
    state[b] = s;
    total[b] = 0;
}

cudaError_t launch_state_init(StreamState *state, int64_t *total, uint32_t *status, const int32_t *head0, int B, int N,
                              cudaStream_t st)
{
    state_init_kernel<<<(B + 127) / 128, 128, 0, st>>>(state, total, status, head0, B, N);
    count_launch();
    return cudaGetLastError();
}

// One (stream, layer) prefix is a single contiguous run of S*row_bytes bytes on both sides.
// grid = (chunks, L, n); 16-byte units, grid-stride over the run.
__global__ void __launch_bounds__(256)
init_static_kernel(uint4 *__restrict__ k_slab, uint4 *__restrict__ v_slab, const uint4 *__restrict__ k_src,
                   const uint4 *__restrict__ v_src, StreamState *state, StreamBatch batch, int src_stream0, int L, int B,
                   int rows_per_block /* ring_off + N */, int S_max, int S_src, int row_units, int to_other_bank)
{
    const int i = blockIdx.z, l = blockIdx.y;
    const int b = batch.id[i];
    const int S = batch.len[i];
    const size_t units = (size_t)S * row_units;
    const size_t src_off = ((size_t)(src_stream0 + i) * L + l) * S_src * row_units;
    // the bank attention reads, or (staging a new prefix while the current one is in use) the other one
    const int bank = ((const volatile StreamState *)state)[b].bank ^ (to_other_bank ? 1 : 0);
    const size_t dst_off = (((size_t)l * B + b) * rows_per_block + (size_t)bank * S_max) * row_units;
    for (size_t u = (size_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (size_t)gridDim.x * blockDim.x) {
        k_slab[dst_off + u] = k_src[src_off + u];
        v_slab[dst_off + u] = v_src[src_off + u];
    }
    if (blockIdx.x == 0 && l == 0 && threadIdx.x == 0) {
        if (to_other_bank) state[b].staged_len = S;
        else state[b].static_len = S;
    }
}

cudaError_t launch_init_static(void *k_slab, void *v_slab, const void *k_src, const void *v_src, StreamState *state,
                               const StreamBatch &batch, int n, int src_stream0, int L, int B, int S_max, int ring_off, int N, int S_src, int to_other_bank,
                               size_t row_bytes, cudaStream_t st)
{
    const int row_units = (int)(row_bytes / 16);
    size_t max_units = (size_t)S_src * row_units;
    int chunks = (int)((max_units + 256 * 8 - 1) / (256 * 8));
    if (chunks < 1) chunks = 1;
    if (chunks > 64) chunks = 64;
    dim3 grid(chunks, L, n);
    init_static_kernel<<<grid, 256, 0, st>>>((uint4 *)k_slab, (uint4 *)v_slab, (const uint4 *)k_src, (const uint4 *)v_src,
                                             state, batch, src_stream0, L, B, ring_off + N, S_max, S_src, row_units, to_other_bank);
    count_launch();
    return cudaGetLastError();
}

// grid = (chunks, n). Every block reads (head, count) of its stream, copies its share of the
// L*m rows to slots (head + i) mod N, then takes a ticket; the last block to arrive publishes the new
// state. No block waits for another, so there is no spin and nothing to time out.
__global__ void __launch_bounds__(256)
append_sliding_kernel(uint4 *__restrict__ k_slab, uint4 *__restrict__ v_slab, const uint4 *__restrict__ k_src,
                      const uint4 *__restrict__ v_src, StreamState *state, int64_t *total, StreamBatch batch,
                      int src_stream0, int L, int B, int ring_off, int N, int m, int row_units)
{
    const int i = blockIdx.y;
    const int b = batch.id[i];
    __shared__ int s_head;
    if (threadIdx.x == 0) s_head = ((volatile StreamState *)state)[b].head;
    __syncthreads();
    const int head = s_head;
    const size_t units = (size_t)L * m * row_units;
    const size_t src_base = (size_t)(src_stream0 + i) * L * m * row_units;
    const int rows_per_block = ring_off + N;
    for (size_t u = (size_t)blockIdx.x * blockDim.x + threadIdx.x; u < units; u += (size_t)gridDim.x * blockDim.x) {
        const int off = (int)(u % row_units);
        const size_t r = u / row_units;
        const int tok = (int)(r % m);
        const int l = (int)(r / m);
        int slot = head + tok;
        if (slot >= N) slot -= N;
        const size_t dst = (((size_t)l * B + b) * rows_per_block + ring_off + slot) * row_units + off;
        k_slab[dst] = k_src[src_base + u];
        v_slab[dst] = v_src[src_base + u];
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int arrived = atomicAdd(&state[b].ticket, 1);
        if (arrived == (int)gridDim.x - 1) {
            // every block of this launch has read `head` and finished its copies: publish the new state
            const int count_old = ((volatile StreamState *)state)[b].count;
            state[b].head = (head + m) % N;
            state[b].count = min(count_old + m, N);
            total[b] += m;
            __threadfence();
            state[b].ticket = 0;
        }
    }
}

cudaError_t launch_append_sliding(void *k_slab, void *v_slab, const void *k_src, const void *v_src, StreamState *state,
                                  int64_t *total, const StreamBatch &batch, int n, int src_stream0, int L, int B, int ring_off,
                                  int N, int m, size_t row_bytes, cudaStream_t st)
{
    const int row_units = (int)(row_bytes / 16);
    const size_t units = (size_t)L * m * row_units;
    int chunks = (int)((units + 256 * 4 - 1) / (256 * 4));
    if (chunks < 1) chunks = 1;
    if (chunks > 32) chunks = 32;
    dim3 grid(chunks, n);
    append_sliding_kernel<<<grid, 256, 0, st>>>((uint4 *)k_slab, (uint4 *)v_slab, (const uint4 *)k_src,
                                                (const uint4 *)v_src, state, total, batch, src_stream0, L, B, ring_off, N, m,
                                                row_units);
    count_launch();
    return cudaGetLastError();
}

// The staged prefix becomes the one attention reads: flip the bank, take over the staged length.
__global__ void commit_static_kernel(StreamState *state, StreamBatch batch, int n)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int b = batch.id[i];
    StreamState s = state[b];
    if (s.staged_len >= 0) {
        s.bank ^= 1;
        s.static_len = s.staged_len;
        s.staged_len = -1;
        state[b] = s;
    }
}

cudaError_t launch_commit_static(StreamState *state, const StreamBatch &batch, int n, cudaStream_t st)
{
    commit_static_kernel<<<(n + 127) / 128, 128, 0, st>>>(state, batch, n);
    count_launch();
    return cudaGetLastError();
}

// Self-test of the bounded-wait convention every kernel of the library follows: one thread waits on an mbarrier that
// nothing will ever complete, with a time limit, and on expiry records the wait site in the status word and returns.
// Nothing here can hang: the limit is clamped by the launcher, and the loop leaves on its own.
__global__ void wait_limit_probe_kernel(uint32_t *status, unsigned long long limit_ns, uint32_t code)
{
    __shared__ __align__(8) unsigned long long probe_bar;
    using namespace ptx;
    const uint32_t bar = smem_u32(&probe_bar);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        fence_mbar_init();
        const unsigned long long t_start = globaltimer_ns();
        bool done = false;
        for (uint32_t n = 1; !done; ++n) {
            if (mbar_try_wait(bar, 0)) done = true;                                   // (never: nothing arrives)
            else if ((n & 63u) == 0u && globaltimer_ns() - t_start > limit_ns) break;
        }
        if (!done) atomicCAS(status, 0u, 0x80000000u | (code << 16) | (blockIdx.x & 0xFFFFu));
    }
}

cudaError_t launch_wait_limit_probe(uint32_t *status, unsigned long long limit_ns, cudaStream_t st)
{
    wait_limit_probe_kernel<<<1, 32, 0, st>>>(status, limit_ns, 127u);
    count_launch();
    return cudaGetLastError();
}

}  // namespace reflex
