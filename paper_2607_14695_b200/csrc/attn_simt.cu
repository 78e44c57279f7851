// Partitioned attention (Eq. 1), SIMT form: fp32 FMA, one warp per query row, online softmax over 32-key
// tiles, optional split over the key range with a merge of (m, l, acc) partials. Serves every supported
// shape and storage type; the tensor-core kernel takes over where the query tile is large enough.
//
// Keys are enumerated in one logical index space per stream:
//   [0, S)            static rows (S = static_len)
//   [S, S+N)          ring slots in PHYSICAL order; slot p is live iff ((p - (head-count)) mod N) < count
//   [S+N, S+N+T)      dynamic tokens, read in place from the caller's tensors
// Softmax does not depend on key order, so the ring is never unrolled or gathered.
#include <math.h>

#include "reflex_internal.cuh"

namespace reflex {

template <typename T, int DPL> struct RowIO;
template <int DPL> struct RowIO<__nv_bfloat16, DPL> {
    // lane-owned slice of DPL consecutive elements
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[DPL]) {
        if constexpr (DPL == 8) {
            uint4 u = *reinterpret_cast<const uint4 *>(p);
            const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
            for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
        } else {
#pragma unroll
            for (int i = 0; i < DPL; ++i) f[i] = __bfloat162float(p[i]);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&f)[DPL]) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) p[i] = __float2bfloat16_rn(f[i]);
    }
};
template <int DPL> struct RowIO<float, DPL> {
    static __device__ __forceinline__ void load(const float *p, float (&f)[DPL]) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) f[i] = p[i];
    }
    static __device__ __forceinline__ void store(float *p, const float (&f)[DPL]) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) p[i] = f[i];
    }
};

template <typename T> __device__ __forceinline__ float ld_f(const T *p);
template <> __device__ __forceinline__ float ld_f<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

// dot of a K row (global, storage type) with a query row (shared, fp32), 8 elements per step
template <typename T>
__device__ __forceinline__ float dot_row(const T *__restrict__ k, const float *__restrict__ q_s, int d)
{
    float acc0 = 0.f, acc1 = 0.f;
    for (int e = 0; e < d; e += 8) {
        float f[8];
        RowIO<T, 8>::load(k + e, f);
        const float4 qa = *reinterpret_cast<const float4 *>(q_s + e);
        const float4 qb = *reinterpret_cast<const float4 *>(q_s + e + 4);
        acc0 = fmaf(f[0], qa.x, acc0); acc1 = fmaf(f[1], qa.y, acc1);
        acc0 = fmaf(f[2], qa.z, acc0); acc1 = fmaf(f[3], qa.w, acc1);
        acc0 = fmaf(f[4], qb.x, acc0); acc1 = fmaf(f[5], qb.y, acc1);
        acc0 = fmaf(f[6], qb.z, acc0); acc1 = fmaf(f[7], qb.w, acc1);
    }
    return acc0 + acc1;
}

constexpr int kSimtWarps = 4;

// grid = (ceil(T*Hq / kSimtWarps), B, nsplit)
template <typename T, int DPL>
__global__ void __launch_bounds__(kSimtWarps * 32)
attn_simt_kernel(AttnParams p)
{
    constexpr int d = DPL * 32;
    __shared__ __align__(16) float q_s[kSimtWarps][d];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.y, split = blockIdx.z;
    const int rows = p.T * p.Hq;
    const int r = blockIdx.x * kSimtWarps + warp;
    if (r >= rows) return;  // no block-wide barrier below
    const int t = r / p.Hq, h = r % p.Hq;
    const int kv = h / (p.Hq / p.Hkv);

    const StreamState st = p.state[b];
    const int S = st.static_len > 0 ? st.static_len : 0;
    const int N = p.N;
    const int n_keys = S + N + p.T;
    const int n_tiles = (n_keys + 31) / 32;
    const int per = (n_tiles + p.nsplit - 1) / p.nsplit;
    const int tile0 = split * per;
    const int tile1 = min(n_tiles, tile0 + per);
    int oldest = (st.head - st.count) % N;  // physical slot of the oldest live token
    if (oldest < 0) oldest += N;

    const size_t row_elems = (size_t)p.Hkv * d;
    const size_t blk = ((size_t)p.layer * p.B + b) * (size_t)(p.ring_off + N);
    const size_t s_row0 = (size_t)st.bank * p.S_max;     // first row of the static bank in use
    const T *k_blk = (const T *)p.k_slab + blk * row_elems + (size_t)kv * d;
    const T *v_blk = (const T *)p.v_slab + blk * row_elems + (size_t)kv * d;
    const T *k_dyn = (const T *)p.k_dyn + (size_t)b * p.T * row_elems + (size_t)kv * d;
    const T *v_dyn = (const T *)p.v_dyn + (size_t)b * p.T * row_elems + (size_t)kv * d;

    const T *q_row = (const T *)p.q + (((size_t)b * p.T + t) * p.Hq + h) * d;
    {
        float f[DPL];
        RowIO<T, DPL>::load(q_row + lane * DPL, f);
#pragma unroll
        for (int i = 0; i < DPL; ++i) q_s[warp][lane * DPL + i] = f[i];
    }
    __syncwarp();

    float m = -INFINITY, l = 0.f;
    float acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = 0.f;

    for (int tile = tile0; tile < tile1; ++tile) {
        const int idx = tile * 32 + lane;
        const T *kp = nullptr, *vp = nullptr;
        if (idx < S) {
            kp = k_blk + (s_row0 + idx) * row_elems; vp = v_blk + (s_row0 + idx) * row_elems;
        } else if (idx < S + N) {
            const int slot = idx - S;
            int age = slot - oldest;
            if (age < 0) age += N;
            if (age < st.count) {
                kp = k_blk + (size_t)(p.ring_off + slot) * row_elems; vp = v_blk + (size_t)(p.ring_off + slot) * row_elems;
            }
        } else if (idx < n_keys) {
            const int j = idx - S - N;
            if (!(p.dyn_mask && j > t)) { kp = k_dyn + (size_t)j * row_elems; vp = v_dyn + (size_t)j * row_elems; }
        }
        float s = -INFINITY;
        if (kp) s = dot_row<T>(kp, q_s[warp], d) * p.scale;
        float tmax = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
        const float m_new = fmaxf(m, tmax);
        if (m_new == -INFINITY) continue;  // nothing live so far (warp-uniform)
        const float alpha = (m == -INFINITY) ? 0.f : expf(m - m_new);
        const float pj = kp ? expf(s - m_new) : 0.f;
        float psum = pj;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
        l = l * alpha + psum;
        m = m_new;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] *= alpha;
        const unsigned long long vaddr = (unsigned long long)vp;
        for (int j = 0; j < 32; ++j) {
            const float w = __shfl_sync(0xffffffffu, pj, j);
            const unsigned long long va = __shfl_sync(0xffffffffu, vaddr, j);
            if (va == 0ull) continue;  // dead key: its V row is never read (may hold stale or poisoned bytes)
            float f[DPL];
            RowIO<T, DPL>::load((const T *)va + lane * DPL, f);
#pragma unroll
            for (int i = 0; i < DPL; ++i) acc[i] = fmaf(w, f[i], acc[i]);
        }
    }

    if (p.nsplit == 1) {
        const float inv = 1.f / l;  // l > 0: a dynamic query always sees itself
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] *= inv;
        T *o = (T *)p.out + (((size_t)b * p.T + t) * p.Hq + h) * d;
        RowIO<T, DPL>::store(o + lane * DPL, acc);
    } else {
        const size_t slot = partial_slot(b, rows, r, p.nsplit, split);
        float *po = partial_o(p.partials, slot, d), *pml = partial_ml(p.partials, (size_t)p.B * rows * p.nsplit, slot, d);
        if (lane == 0) { pml[0] = m; pml[1] = l; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) po[lane * DPL + i] = acc[i];
    }
}

// Merge of split partials: m* = max m_s, l = sum l_s e^{m_s-m*}, o = sum acc_s e^{m_s-m*} / l. One warp per query row
// (lane s fetches slice s's (m, l); every lane owns d/32 output columns), 8 rows per block, all loads independent.
template <typename T, int DPL>
__global__ void __launch_bounds__(256)
attn_merge_kernel(AttnParams p)
{
    constexpr int d = DPL * 32;
    // launched with programmatic stream serialisation: wait for the attention kernel ahead of it before reading its partials
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rows = p.T * p.Hq;
    const int gr = blockIdx.x * 8 + warp;      // row over all streams
    if (gr >= p.B * rows) return;
    const int b = gr / rows, r = gr % rows;
    const size_t n_slots = (size_t)p.B * rows * p.nsplit;
    const size_t slot0 = partial_slot(b, rows, r, p.nsplit, 0);
    float ms = -INFINITY, ls = 0.f;
    if (lane < p.nsplit) {
        const float2 ml = *reinterpret_cast<const float2 *>(partial_ml(p.partials, n_slots, slot0 + lane, d));
        ms = ml.x; ls = ml.y;
    }
    float mstar = ms;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, o));
    const float w = (ms == -INFINITY) ? 0.f : expf(ms - mstar);
    float l = ls * w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    float acc[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
    // Slices in batches of eight: all of a batch's loads are issued before the first is used (guarded one by one, every slice
    // was an L2 round trip of its own in front of the next). An empty slice never wrote its O row: whatever is read there
    // is dropped by the weight test, not multiplied by zero.
    for (int s0 = 0; s0 < p.nsplit; s0 += 8) {
        float f[8][DPL], ws[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int s = min(s0 + j, p.nsplit - 1);
            ws[j] = s0 + j < p.nsplit ? __shfl_sync(0xffffffffu, w, s) : 0.f;
            const float *po = partial_o(p.partials, slot0 + s, d) + lane * DPL;
            if constexpr (DPL % 4 == 0) {
#pragma unroll
                for (int i = 0; i < DPL; i += 4) {
                    const float4 v = *reinterpret_cast<const float4 *>(po + i);
                    f[j][i] = v.x; f[j][i + 1] = v.y; f[j][i + 2] = v.z; f[j][i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < DPL; ++i) f[j][i] = po[i];
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (ws[j] != 0.f) {
#pragma unroll
                for (int i = 0; i < DPL; ++i) acc[i] = fmaf(f[j][i], ws[j], acc[i]);
            }
        }
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= inv;
    const int t = r / p.Hq, h = r % p.Hq;
    T *out = (T *)p.out + (((size_t)b * p.T + t) * p.Hq + h) * d;
    RowIO<T, DPL>::store(out + lane * DPL, acc);
}

int simt_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count)
{
    const int rows = p.T * p.Hq;
    const int blocks = ((rows + kSimtWarps - 1) / kSimtWarps) * p.B;
    const int n_tiles = (p.S_max + p.N + p.T + 31) / 32;
    int want = (4 * sm_count + blocks - 1) / blocks;  // aim at ~4 blocks per SM
    if (want > n_tiles / 2) want = n_tiles / 2;       // at least two key tiles per split
    if (want > kMaxSplits) want = kMaxSplits;
    const size_t per_split = (size_t)p.B * rows * (p.d + 2) * sizeof(float);
    if (per_split > 0 && (size_t)want * per_split > partial_bytes) want = (int)(partial_bytes / per_split);
    if (want < 1) want = 1;
    return want;
}

template <typename T>
static cudaError_t launch_simt_t(const AttnParams &p, cudaStream_t st)
{
    const int rows = p.T * p.Hq;
    dim3 grid((rows + kSimtWarps - 1) / kSimtWarps, p.B, p.nsplit);
    switch (p.d / 32) {
        case 1: attn_simt_kernel<T, 1><<<grid, kSimtWarps * 32, 0, st>>>(p); break;
        case 2: attn_simt_kernel<T, 2><<<grid, kSimtWarps * 32, 0, st>>>(p); break;
        case 4: attn_simt_kernel<T, 4><<<grid, kSimtWarps * 32, 0, st>>>(p); break;
        case 8: attn_simt_kernel<T, 8><<<grid, kSimtWarps * 32, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || p.nsplit == 1) return e;
    return launch_attention_merge(p, st);
}

template <typename T>
static cudaError_t launch_merge_t(const AttnParams &p, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.B * p.T * p.Hq + 7) / 8);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    switch (p.d / 32) {
        case 1: e = cudaLaunchKernelEx(&cfg, attn_merge_kernel<T, 1>, p); break;
        case 2: e = cudaLaunchKernelEx(&cfg, attn_merge_kernel<T, 2>, p); break;
        case 4: e = cudaLaunchKernelEx(&cfg, attn_merge_kernel<T, 4>, p); break;
        case 8: e = cudaLaunchKernelEx(&cfg, attn_merge_kernel<T, 8>, p); break;
        default: return cudaErrorInvalidValue;
    }
    count_launch();
    return e;
}

cudaError_t launch_attention_merge(const AttnParams &p, cudaStream_t st)
{
    if (p.dtype == REFLEX_DTYPE_BF16) return launch_merge_t<__nv_bfloat16>(p, st);
    return launch_merge_t<float>(p, st);
}

cudaError_t launch_attention_simt(const AttnParams &p, cudaStream_t st)
{
    if (p.dtype == REFLEX_DTYPE_BF16) return launch_simt_t<__nv_bfloat16>(p, st);
    return launch_simt_t<float>(p, st);
}

}  // namespace reflex
