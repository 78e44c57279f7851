// AdaRMSNorm (Eq. 2, App. B.3): y = x * rsqrt(mean x^2 + eps) * (1 + W2 SiLU(W1 c + b1) + b2).
// Row statistics, the gate MLP accumulation and the product are fp32; the result is rounded once on store.
#include "reflex_internal.cuh"

namespace reflex {

template <typename T> struct Vec8;
template <> struct Vec8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[8]) {
        uint4 u = *reinterpret_cast<const uint4 *>(p);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&f)[8]) {
        uint4 u;
        __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        *reinterpret_cast<uint4 *>(p) = u;
    }
};
template <> struct Vec8<float> {
    static __device__ __forceinline__ void load(const float *p, float (&f)[8]) {
        float4 a = reinterpret_cast<const float4 *>(p)[0], b = reinterpret_cast<const float4 *>(p)[1];
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&f)[8]) {
        reinterpret_cast<float4 *>(p)[0] = make_float4(f[0], f[1], f[2], f[3]);
        reinterpret_cast<float4 *>(p)[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// hidden = SiLU(W1 c + b1) for one stream into shared memory; c_s is scratch of Cd floats.
template <typename T>
__device__ void gate_hidden(const T *__restrict__ cond_b, const T *__restrict__ W1, const T *__restrict__ b1, int Cd, int Hd,
                            float *c_s, float *hid_s)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    for (int e = threadIdx.x; e < Cd; e += blockDim.x) c_s[e] = to_f<T>(cond_b[e]);
    __syncthreads();
    for (int j = warp; j < Hd; j += nwarp) {
        const T *w = W1 + (size_t)j * Cd;
        float acc = 0.f;
        for (int e = lane * 8; e < Cd; e += 256) {
            float f[8];
            Vec8<T>::load(w + e, f);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc = fmaf(f[i], c_s[e + i], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            const float z = acc + to_f<T>(b1[j]);
            hid_s[j] = z / (1.f + expf(-z));
        }
    }
    __syncthreads();
}

// gate[i] = 1 + b2[i] + W2[i] . hidden for columns [i0, i1): one warp per column.
template <typename T>
__device__ void gate_columns(const T *__restrict__ W2, const T *__restrict__ b2, int Hd, int i0, int i1, const float *hid_s,
                             float *gate_out /* indexed by i - i0 */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    for (int i = i0 + warp; i < i1; i += nwarp) {
        const T *w = W2 + (size_t)i * Hd;
        float acc = 0.f;
        for (int e = lane * 8; e < Hd; e += 256) {
            float f[8];
            Vec8<T>::load(w + e, f);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc = fmaf(f[k], hid_s[e + k], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) gate_out[i - i0] = 1.f + (acc + to_f<T>(b2[i]));
    }
}

// grid = (column chunks, B): writes gate_buf[b][i].
template <typename T>
__global__ void __launch_bounds__(256)
gate_kernel(const T *__restrict__ cond, const T *__restrict__ W1, const T *__restrict__ b1, const T *__restrict__ W2,
            const T *__restrict__ b2, float *__restrict__ gate_buf, int D, int Cd, int Hd, int cols_per_block)
{
    extern __shared__ float smem[];
    float *c_s = smem, *hid_s = smem + Cd;
    const int b = blockIdx.y;
    gate_hidden<T>(cond + (size_t)b * Cd, W1, b1, Cd, Hd, c_s, hid_s);
    const int i0 = blockIdx.x * cols_per_block;
    const int i1 = min(D, i0 + cols_per_block);
    gate_columns<T>(W2, b2, Hd, i0, i1, hid_s, gate_buf + (size_t)b * D + i0);
}

// grid = (row chunks, B); one warp per row. FUSED: the block computes its stream's gate itself.
template <typename T, bool FUSED>
__global__ void __launch_bounds__(256)
adarmsnorm_kernel(const T *x, T *y, const T *__restrict__ cond, const T *__restrict__ W1,
                  const T *__restrict__ b1, const T *__restrict__ W2, const T *__restrict__ b2,
                  const float *__restrict__ gate_buf, int R, int D, int Cd, int Hd, float eps, int rows_per_block)
{
    extern __shared__ float smem[];
    float *gate_s = smem;  // D floats
    const int b = blockIdx.y;
    if (FUSED) {
        float *c_s = smem + D, *hid_s = c_s + Cd;
        gate_hidden<T>(cond + (size_t)b * Cd, W1, b1, Cd, Hd, c_s, hid_s);
        gate_columns<T>(W2, b2, Hd, 0, D, hid_s, gate_s);
    } else {
        for (int i = threadIdx.x; i < D; i += blockDim.x) gate_s[i] = gate_buf[(size_t)b * D + i];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    const int r0 = blockIdx.x * rows_per_block;
    const int r1 = min(R, r0 + rows_per_block);
    const float inv_D = 1.f / (float)D;
    for (int r = r0 + warp; r < r1; r += nwarp) {
        const T *xr = x + ((size_t)b * R + r) * D;
        T *yr = y + ((size_t)b * R + r) * D;
        float ss = 0.f;
        for (int e = lane * 8; e < D; e += 256) {
            float f[8];
            Vec8<T>::load(xr + e, f);
#pragma unroll
            for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
        }
        ss = warp_sum(ss);
        const float rinv = 1.f / sqrtf(ss * inv_D + eps);
        for (int e = lane * 8; e < D; e += 256) {
            float f[8];
            Vec8<T>::load(xr + e, f);  // second read hits L1/L2; x and y may alias, each lane rewrites only what it read
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = f[i] * rinv * gate_s[e + i];
            Vec8<T>::store(yr + e, f);
        }
    }
}


// ---- gate MLP with scratch (gate_buf given): two small launches, hidden then gate, each ONE round of memory
// ---- latency: a block stages 8 weight rows and the vectors of up to 32 streams in shared memory, then every thread
// ---- owns one (weight row, stream) dot product -- no shuffles, no dependent loads.
constexpr int kGateStreams = 32;   // streams per block
constexpr int kGateUnits = 8;      // weight rows (hidden units or gate columns) per block

// out[s][u0+u] = act(bias[u0+u] + W[u0+u][:] . vec[b0+s][:]);  SILU: hidden layer, else 1 + (.) for the gate.
// vec is T (conditioning) or float (hidden activations). grid = (ceil(units/8), ceil(B/32)), 256 threads.
template <typename T, typename VT, bool SILU>
__global__ void __launch_bounds__(256)
gate_layer_kernel(const VT *vec, const T *__restrict__ W, const T *__restrict__ bias, float *out, int B, int len, int units,
                  int wait_prior, size_t vec_lstride, size_t out_lstride, int upb)
{
    // upb = weight rows per block (a multiple of 8): the staged stream vectors are reused by upb/8 passes of 8 rows
    // blockIdx.z = layer: weights and biases of the layers are stacked ([L][units][len], [L][units]); the input vectors
    // are shared by the layers (conditioning, stride 0) or per layer (hidden activations)
    vec += (size_t)blockIdx.z * vec_lstride;
    W += (size_t)blockIdx.z * units * len;
    bias += (size_t)blockIdx.z * units;
    out += (size_t)blockIdx.z * out_lstride;
    extern __shared__ __align__(16) float sm_gl[];
    const int pitch = len + 4;                   // +4 floats: the 32 stream rows start in different banks
    float *w_s = sm_gl;                          // [upb][len]
    float *v_s = sm_gl + upb * len;              // [32][pitch]
    const int b0 = blockIdx.y * kGateStreams;
    const int nb = min(kGateStreams, B - b0);
    const int u0 = blockIdx.x * upb;
    const int nu = min(upb, units - u0);
    // weight rows do not depend on the preceding launch: fetch them first, then wait for it (programmatic dependent launch)
    for (int i = threadIdx.x * 8; i < nu * len; i += blockDim.x * 8) {
        float f[8];
        Vec8<T>::load(W + (size_t)u0 * len + i, f);
        *reinterpret_cast<float4 *>(w_s + i) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4 *>(w_s + i + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    if (wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int chunks = len / 8;
    for (int i = threadIdx.x; i < nb * chunks; i += blockDim.x) {
        const int s = i / chunks, e = (i % chunks) * 8;
        float f[8];
        Vec8<VT>::load(vec + (size_t)(b0 + s) * len + e, f);
        *reinterpret_cast<float4 *>(v_s + s * pitch + e) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4 *>(v_s + s * pitch + e + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    __syncthreads();
    const int sidx = threadIdx.x & 31;
    if (sidx >= nb) return;
    const float *vr = v_s + sidx * pitch;
    for (int u = threadIdx.x >> 5; u < nu; u += kGateUnits) {
        const float *wr = w_s + u * len;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        for (int e = 0; e < len; e += 4) {
            const float4 wv = *reinterpret_cast<const float4 *>(wr + e);
            const float4 vv = *reinterpret_cast<const float4 *>(vr + e);
            a0 = fmaf(wv.x, vv.x, a0); a1 = fmaf(wv.y, vv.y, a1); a2 = fmaf(wv.z, vv.z, a2); a3 = fmaf(wv.w, vv.w, a3);
        }
        const float z = ((a0 + a1) + (a2 + a3)) + to_f<T>(bias[u0 + u]);
        out[(size_t)(b0 + sidx) * units + u0 + u] = SILU ? z / (1.f + expf(-z)) : 1.f + z;
    }
}

// Register-tiled form of one gate layer, used when many layers are evaluated by one call (blockIdx.z = layer): a block
// owns 64 weight rows and up to 32 streams and each thread accumulates a 2 (rows) x 4 (streams) tile, so one 16-byte
// shared-memory load feeds up to eight FMAs instead of two. Every dot product is summed in the same order as in
// gate_layer_kernel (four interleaved partial sums), so the two kernels give identical bits.
constexpr int kTileUnits = 64;
template <typename T, typename VT, bool SILU>
__global__ void __launch_bounds__(256)
gate_layer_tiled_kernel(const VT *vec, const T *__restrict__ W, const T *__restrict__ bias, float *out, int B, int len, int units,
                        int wait_prior, size_t vec_lstride, size_t out_lstride)
{
    vec += (size_t)blockIdx.z * vec_lstride;
    W += (size_t)blockIdx.z * units * len;
    bias += (size_t)blockIdx.z * units;
    out += (size_t)blockIdx.z * out_lstride;
    extern __shared__ __align__(16) float sm_gt[];
    const int pitch = len + 4;
    float *w_s = sm_gt;                              // [64][pitch]
    float *v_s = sm_gt + kTileUnits * pitch;         // [32][pitch]
    const int b0 = blockIdx.y * kGateStreams;
    const int nb = min(kGateStreams, B - b0);
    const int u0 = blockIdx.x * kTileUnits;
    const int nu = min(kTileUnits, units - u0);
    const int chunks = len / 8;
    for (int i = threadIdx.x; i < kTileUnits * chunks; i += blockDim.x) {
        const int u = i / chunks, e = (i % chunks) * 8;
        float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (u < nu) Vec8<T>::load(W + (size_t)(u0 + u) * len + e, f);
        *reinterpret_cast<float4 *>(w_s + u * pitch + e) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4 *>(w_s + u * pitch + e + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    if (wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = threadIdx.x; i < kGateStreams * chunks; i += blockDim.x) {
        const int sx = i / chunks, e = (i % chunks) * 8;
        float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (sx < nb) Vec8<VT>::load(vec + (size_t)(b0 + sx) * len + e, f);
        *reinterpret_cast<float4 *>(v_s + sx * pitch + e) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4 *>(v_s + sx * pitch + e + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
    __syncthreads();
    const int sg = threadIdx.x & 7, up = threadIdx.x >> 3;   // streams sg, sg+8, sg+16, sg+24 (bank-conflict free), weight rows up*2, up*2+1
    const float *w0 = w_s + (up * 2) * pitch, *w1 = w0 + pitch;
    const float *v0 = v_s + sg * pitch;
    float4 acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int e = 0; e < len; e += 4) {
        const float4 a = *reinterpret_cast<const float4 *>(w0 + e), c = *reinterpret_cast<const float4 *>(w1 + e);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 v = *reinterpret_cast<const float4 *>(v0 + j * 8 * pitch + e);
            acc[0][j].x = fmaf(a.x, v.x, acc[0][j].x); acc[0][j].y = fmaf(a.y, v.y, acc[0][j].y);
            acc[0][j].z = fmaf(a.z, v.z, acc[0][j].z); acc[0][j].w = fmaf(a.w, v.w, acc[0][j].w);
            acc[1][j].x = fmaf(c.x, v.x, acc[1][j].x); acc[1][j].y = fmaf(c.y, v.y, acc[1][j].y);
            acc[1][j].z = fmaf(c.z, v.z, acc[1][j].z); acc[1][j].w = fmaf(c.w, v.w, acc[1][j].w);
        }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int u = up * 2 + i;
        if (u >= nu) continue;
        const float bi = to_f<T>(bias[u0 + u]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int sx = sg + 8 * j;
            if (sx >= nb) continue;
            const float z = ((acc[i][j].x + acc[i][j].y) + (acc[i][j].z + acc[i][j].w)) + bi;
            out[(size_t)(b0 + sx) * units + u0 + u] = SILU ? z / (1.f + expf(-z)) : 1.f + z;
        }
    }
}

// One warp per row, the row kept in registers between the statistics pass and the scaling pass
// (D <= 256 * NCH), so x is read from memory exactly once. grid = ceil(B*R / 8).
template <typename T, int NCH>
__global__ void __launch_bounds__(256)
adarmsnorm_rows_kernel(const T *x, T *y, const float *gate_buf, int rows, int R, int D, float eps, int wait_first)
{
    // Programmatic dependent launch, both ways. This grid may have been scheduled before the kernel launched ahead of it on
    // the stream has finished: unless that kernel is the library's own gate kernel (which does not write x: wait_first = 0)
    // nothing is read before it is known to be complete. And the kernel launched after this one may be scheduled as soon as
    // every block of this grid has started; it waits the same way before it touches memory.
    if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * 8 + warp;
    if (row >= rows) return;
    const int b = row / R;
    const T *xr = x + (size_t)row * D;
    T *yr = y + (size_t)row * D;
    const float *g = gate_buf + (size_t)b * D;
    float f[NCH][8];
    float4 gg[NCH][2];
    float ss = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int e = c * 256 + lane * 8;
        if (e < D) {
            Vec8<T>::load(xr + e, f[c]);
            if (wait_first) {   // the gate is final already: fetch it in the same round trip as the row
                gg[c][0] = *reinterpret_cast<const float4 *>(g + e);
                gg[c][1] = *reinterpret_cast<const float4 *>(g + e + 4);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) ss = fmaf(f[c][i], f[c][i], ss);
        }
    }
    ss = warp_sum(ss);
    const float rinv = 1.f / sqrtf(ss / (float)D + eps);
    // the gate may still be in the making by the preceding launch (programmatic dependent launch): x is already in
    // registers and the statistics are done, now wait for that grid to finish and its writes to be visible
    if (!wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int e = c * 256 + lane * 8;
        if (e < D) {
            const float4 g0 = wait_first ? gg[c][0] : *reinterpret_cast<const float4 *>(g + e);
            const float4 g1 = wait_first ? gg[c][1] : *reinterpret_cast<const float4 *>(g + e + 4);
            float o[8];
            o[0] = f[c][0] * rinv * g0.x; o[1] = f[c][1] * rinv * g0.y; o[2] = f[c][2] * rinv * g0.z; o[3] = f[c][3] * rinv * g0.w;
            o[4] = f[c][4] * rinv * g1.x; o[5] = f[c][5] * rinv * g1.y; o[6] = f[c][6] * rinv * g1.z; o[7] = f[c][7] * rinv * g1.w;
            Vec8<T>::store(yr + e, o);
        }
    }
}

template <typename T>
static cudaError_t launch_rows_t(const T *x, T *y, const float *gate_buf, int B, int R, int D, float eps, bool after_gate, cudaStream_t st)
// after_gate: the kernel launched just before on this stream is the gate kernel of the same call (it may still be running
// while the rows are read and their statistics taken); otherwise the grid waits for whatever precedes it before reading.
{
    const int rows = B * R;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((rows + 7) / 8);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int wait_first = after_gate ? 0 : 1;
    cudaError_t e;
    if (D <= 512) e = cudaLaunchKernelEx(&cfg, adarmsnorm_rows_kernel<T, 2>, x, y, gate_buf, rows, R, D, eps, wait_first);
    else if (D <= 1024) e = cudaLaunchKernelEx(&cfg, adarmsnorm_rows_kernel<T, 4>, x, y, gate_buf, rows, R, D, eps, wait_first);
    else if (D <= 2048) e = cudaLaunchKernelEx(&cfg, adarmsnorm_rows_kernel<T, 8>, x, y, gate_buf, rows, R, D, eps, wait_first);
    else return cudaErrorNotSupported;
    count_launch();
    return e;
}

static bool gate_scratch_fits(int Cd, int Hd)
{
    const size_t smem_h = (size_t)(32 * Cd + kGateStreams * (Cd + 4)) * 4;
    const size_t smem_g = (size_t)(32 * Hd + kGateStreams * (Hd + 4)) * 4;
    return smem_h <= 160 * 1024 && smem_g <= 160 * 1024;
}

// gamma_l(c) = 1 + W2_l SiLU(W1_l c + b1_l) + b2_l for L layers (stacked weights) and B streams: gates into
// gate_buf[L][B][D], hidden activations into gate_buf + L*B*D ([L][B][Hd]). Two launches whatever L is.
template <typename T>
static cudaError_t launch_gate_t(const T *cond, const T *W1, const T *b1, const T *W2, const T *b2, float *gate_buf, int L, int B,
                                 int D, int Cd, int Hd, cudaStream_t st)
{
    // one layer: 8 weight rows per block (more blocks, lower latency); many layers: 32 rows per block, so the staged
    // stream vectors are fetched four times less often
    const int upb = L > 1 ? 32 : kGateUnits;
    const size_t smem_h = (size_t)(upb * Cd + kGateStreams * (Cd + 4)) * 4;
    const size_t smem_g = (size_t)(upb * Hd + kGateStreams * (Hd + 4)) * 4;
    float *hid = gate_buf + (size_t)L * B * D;
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        cudaError_t e = cudaFuncSetAttribute(gate_layer_kernel<T, T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gate_layer_kernel<T, float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
        return e;
    });
    if (e0 != cudaSuccess) return e0;
    if constexpr (sizeof(T) == 2) {
        // bf16: both layers on the tensor cores, whatever L is (one call for L layers and L calls give the same bits); the
        // FMA kernels below remain for fp32 and for widths the tensor-core kernel does not take
        if (gate_tc_supported(B, D, Cd, Hd)) {
            cudaError_t e = launch_gate_tc(cond, W1, b1, W2, b2, gate_buf, L, B, D, Cd, Hd, st);
            if (e != cudaErrorInvalidValue) return e;   // invalid value: no tensor maps from this driver, fall through
        }
    }
    const int groups = (B + kGateStreams - 1) / kGateStreams;
    const size_t tiled_h = (size_t)(kTileUnits + kGateStreams) * (Cd + 4) * 4, tiled_g = (size_t)(kTileUnits + kGateStreams) * (Hd + 4) * 4;
    if (L > 1 && tiled_h <= 200 * 1024 && tiled_g <= 200 * 1024) {
        // many layers in one call: throughput of the whole batch matters more than the latency of one small grid
        static std::atomic<unsigned long long> tiled_attr_set{0};
        e0 = once_per_device(tiled_attr_set, [] {
            cudaError_t e = cudaFuncSetAttribute(gate_layer_tiled_kernel<T, T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(gate_layer_tiled_kernel<T, float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            return e;
        });
        if (e0 != cudaSuccess) return e0;
        gate_layer_tiled_kernel<T, T, true><<<dim3((Hd + kTileUnits - 1) / kTileUnits, groups, L), 256, tiled_h, st>>>(
            cond, W1, b1, hid, B, Cd, Hd, 0, (size_t)0, (size_t)B * Hd);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((D + kTileUnits - 1) / kTileUnits, groups, L);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = tiled_g;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, gate_layer_tiled_kernel<T, float, false>, (const float *)hid, W2, b2, gate_buf, B, Hd, D, 1,
                               (size_t)B * Hd, (size_t)B * D);
        count_launch();
        return e;
    }
    gate_layer_kernel<T, T, true><<<dim3((Hd + upb - 1) / upb, groups, L), 256, smem_h, st>>>(
        cond, W1, b1, hid, B, Cd, Hd, 0, (size_t)0, (size_t)B * Hd, upb);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((D + upb - 1) / upb, groups, L);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = smem_g;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, gate_layer_kernel<T, float, false>, (const float *)hid, W2, b2, gate_buf, B, Hd, D, 1,
                           (size_t)B * Hd, (size_t)B * D, upb);
    count_launch();
    return e;
}

template <typename T>
static cudaError_t launch_norm_t(const T *x, T *y, const T *cond, const T *W1, const T *b1, const T *W2, const T *b2,
                                 float *gate_buf, int B, int R, int D, int Cd, int Hd, float eps, cudaStream_t st)
{
    bool after_gate = false;
    if (cond && gate_buf && gate_scratch_fits(Cd, Hd)) {
        cudaError_t e = launch_gate_t<T>(cond, W1, b1, W2, b2, gate_buf, 1, B, D, Cd, Hd, st);
        if (e != cudaSuccess) return e;
        after_gate = true;
    } else if (cond && gate_buf) {
        // very wide conditioning / hidden layers: per-block gate (shared-memory staging of 16 streams would not fit)
        const int cols = 64;
        gate_kernel<T><<<dim3((D + cols - 1) / cols, B), 256, (size_t)(Cd + Hd) * 4, st>>>(cond, W1, b1, W2, b2, gate_buf, D, Cd, Hd, cols);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (gate_buf && D <= 2048) return launch_rows_t<T>(x, y, gate_buf, B, R, D, eps, after_gate, st);
    // enough blocks to cover the SMs about twice, at least one row per warp
    int chunks = (296 + B - 1) / B;
    const int max_chunks = (R + 7) / 8;
    if (chunks > max_chunks) chunks = max_chunks;
    if (chunks < 1) chunks = 1;
    const int rows_per_block = (R + chunks - 1) / chunks;
    chunks = (R + rows_per_block - 1) / rows_per_block;
    dim3 grid(chunks, B);
    if (cond && !gate_buf) {
        size_t smem = (size_t)(D + Cd + Hd) * 4;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(adarmsnorm_kernel<T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        adarmsnorm_kernel<T, true><<<grid, 256, smem, st>>>(x, y, cond, W1, b1, W2, b2, nullptr, R, D, Cd, Hd, eps, rows_per_block);
    } else {
        size_t smem = (size_t)D * 4;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(adarmsnorm_kernel<T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        adarmsnorm_kernel<T, false><<<grid, 256, smem, st>>>(x, y, nullptr, nullptr, nullptr, nullptr, nullptr, gate_buf, R, D, Cd, Hd, eps, rows_per_block);
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_adarmsnorm(const void *x, void *y, const void *cond, const void *W1, const void *b1, const void *W2,
                              const void *b2, float *gate_buf, int B, int R, int D, int Cd, int Hd, float eps, int dtype,
                              cudaStream_t st)
{
    if (dtype == REFLEX_DTYPE_BF16)
        return launch_norm_t<__nv_bfloat16>((const __nv_bfloat16 *)x, (__nv_bfloat16 *)y, (const __nv_bfloat16 *)cond,
                                            (const __nv_bfloat16 *)W1, (const __nv_bfloat16 *)b1, (const __nv_bfloat16 *)W2,
                                            (const __nv_bfloat16 *)b2, gate_buf, B, R, D, Cd, Hd, eps, st);
    return launch_norm_t<float>((const float *)x, (float *)y, (const float *)cond, (const float *)W1, (const float *)b1,
                                (const float *)W2, (const float *)b2, gate_buf, B, R, D, Cd, Hd, eps, st);
}

// Euler update (Sec. 2.1; App. C): x <- x + dt * v on the fp32 master, optional low-precision mirror.
template <typename T>
__global__ void flow_step_kernel(float *__restrict__ x, const T *__restrict__ v, T *__restrict__ x_lowp, size_t n, float dt)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float nx = fmaf(dt, to_f<T>(v[i]), x[i]);
        x[i] = nx;
        if (x_lowp) {
            if constexpr (sizeof(T) == 2) x_lowp[i] = __float2bfloat16_rn(nx);
            else x_lowp[i] = nx;
        }
    }
}

template <typename T>
static cudaError_t launch_gate_wide_t(const T *cond, const T *W1, const T *b1, const T *W2, const T *b2, float *gate_buf, int L, int B,
                                      int D, int Cd, int Hd, cudaStream_t st)
{
    const int cols = 64;
    for (int l = 0; l < L; ++l) {
        gate_kernel<T><<<dim3((D + cols - 1) / cols, B), 256, (size_t)(Cd + Hd) * 4, st>>>(
            cond, W1 + (size_t)l * Hd * Cd, b1 + (size_t)l * Hd, W2 + (size_t)l * D * Hd, b2 + (size_t)l * D, gate_buf + (size_t)l * B * D, D, Cd, Hd, cols);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_adarmsnorm_gate(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2, float *gate_buf,
                                   int L, int B, int D, int Cd, int Hd, int dtype, cudaStream_t st)
{
    if (!gate_scratch_fits(Cd, Hd)) {
        // conditioning or hidden layers too wide to stage 32 streams' vectors in shared memory: the per-stream kernel, layer by layer
        if (dtype == REFLEX_DTYPE_BF16)
            return launch_gate_wide_t<__nv_bfloat16>((const __nv_bfloat16 *)cond, (const __nv_bfloat16 *)W1, (const __nv_bfloat16 *)b1,
                                                     (const __nv_bfloat16 *)W2, (const __nv_bfloat16 *)b2, gate_buf, L, B, D, Cd, Hd, st);
        return launch_gate_wide_t<float>((const float *)cond, (const float *)W1, (const float *)b1, (const float *)W2, (const float *)b2,
                                         gate_buf, L, B, D, Cd, Hd, st);
    }
    if (dtype == REFLEX_DTYPE_BF16)
        return launch_gate_t<__nv_bfloat16>((const __nv_bfloat16 *)cond, (const __nv_bfloat16 *)W1, (const __nv_bfloat16 *)b1,
                                            (const __nv_bfloat16 *)W2, (const __nv_bfloat16 *)b2, gate_buf, L, B, D, Cd, Hd, st);
    return launch_gate_t<float>((const float *)cond, (const float *)W1, (const float *)b1, (const float *)W2, (const float *)b2,
                                gate_buf, L, B, D, Cd, Hd, st);
}

cudaError_t launch_flow_step(float *x, const void *v, void *x_lowp, size_t n, float dt, int dtype, cudaStream_t st)
{
    int blocks = (int)((n + 255) / 256);
    if (blocks > 1184) blocks = 1184;
    if (blocks < 1) blocks = 1;
    if (dtype == REFLEX_DTYPE_BF16)
        flow_step_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(x, (const __nv_bfloat16 *)v, (__nv_bfloat16 *)x_lowp, n, dt);
    else
        flow_step_kernel<float><<<blocks, 256, 0, st>>>(x, (const float *)v, (float *)x_lowp, n, dt);
    count_launch();
    return cudaGetLastError();
}

}  // namespace reflex

// ------------------------------------------------------------------------------------------------
// Entry point that needs no scratch from the caller (see reflex.h). Lives in this file because host code
// may only name the array below through cudaGetSymbolAddress, and that lookup has to sit beside the definition.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr size_t kNoAllocFloats = 96 * 1024;   // 384 KiB per GPU that loads the library, held until the process exits
static __device__ __align__(256) float g_noalloc_gate[kNoAllocFloats];

constexpr int kMaxDevices = 64;
float *g_noalloc_ptr[kMaxDevices] = {};        // device address of the array, per device, resolved on first use

}  // namespace

extern "C" int reflex_adarmsnorm_noalloc(const void *x, void *y, const void *cond, const void *W1, const void *b1,
                                         const void *W2, const void *b2, int B, int R, int D, int Cd, int Hd, float eps,
                                         int dtype, void *stream)
{
    // same argument checks as reflex_adarmsnorm with cond given, plus the size limit of the built-in scratch
    if (B < 1 || R < 1 || D < 8 || D % 8 != 0 || D > 2048 || Hd < 8 || Hd % 8 != 0 || Cd < 8 || Cd % 8 != 0 || Cd > 4096 || Hd > 4096)
        return reflex::api_fail(REFLEX_ERR_SHAPE, "reflex_adarmsnorm_noalloc: need B, R >= 1, D a multiple of 8 in [8, 2048], Cd and Hd multiples of 8 in [8, 4096]");
    if ((size_t)B * (size_t)(D + Hd) > kNoAllocFloats)
        return reflex::api_fail(REFLEX_ERR_SHAPE, "reflex_adarmsnorm_noalloc: B*(D+Hd) = %zu floats exceeds the built-in scratch of %zu floats; "
                                "use reflex_adarmsnorm with a caller-provided gate_buf", (size_t)B * (size_t)(D + Hd), kNoAllocFloats);
    if (!x || !y || !cond || !W1 || !b1 || !W2 || !b2) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "reflex_adarmsnorm_noalloc: NULL argument");
    if (dtype != REFLEX_DTYPE_BF16 && dtype != REFLEX_DTYPE_F32) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (!(eps >= 0.f)) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "eps must be >= 0");
    const void *ptrs[7] = {x, y, cond, W1, b1, W2, b2};
    for (const void *q : ptrs)
        if (reinterpret_cast<uintptr_t>(q) & 15u) return reflex::api_fail(REFLEX_ERR_ALIGN, "reflex_adarmsnorm_noalloc: pointer not 16-byte aligned");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return reflex::api_fail(REFLEX_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return reflex::api_fail(REFLEX_ERR_INVALID_ARG, "device ordinal %d not supported", dev);
    if (!g_noalloc_ptr[dev]) {
        // First call on this device: turn the symbol into a device address. In host code `g_noalloc_gate` is only a
        // stand-in for the symbol, never an address a kernel could use.
        float *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_gate);
        if (e != cudaSuccess || !ptr) return reflex::api_fail(REFLEX_ERR_CUDA, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        g_noalloc_ptr[dev] = ptr;
    }
    e = reflex::launch_adarmsnorm(x, y, cond, W1, b1, W2, b2, g_noalloc_ptr[dev], B, R, D, Cd, Hd, eps, dtype, (cudaStream_t)stream);
    if (e != cudaSuccess) return reflex::api_fail(REFLEX_ERR_CUDA, "adarmsnorm launch: %s", cudaGetErrorString(e));
    return REFLEX_OK;
}
