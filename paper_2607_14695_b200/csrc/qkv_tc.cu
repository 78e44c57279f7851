// Adaptive norm folded into the packed Q/K/V projection (Sec. 3.3 "System Optimizations": W_QKV = [W_Q; W_K; W_V] as one
// GEMM; Sec. 4 "Operator Fusion Impact": the adaptive norm combined with the linear layer after it, so that the norm output
// never reaches memory):
//     [q | k_dyn | v_dyn][r][n] = (1 / RMS(x_r)) * sum_i (x[r][i] * gamma_b[i]) * W_QKV[n][i]          (Eq. 2 + projection)
//
// bf16 path: a pair of CTAs (cta_group::2) owns a 256 x 256 output tile and walks the contraction axis in 64-column
// steps through a ring of stages. Per step and CTA, TMA brings 128 rows of x and 128 rows of W_QKV into shared memory.
// Eight warps (two threads per row) read their half row of x, multiply by the stream's gate (staged in shared memory
// once per CTA), round to bf16 and store the result into a ring of A stages in TENSOR memory (tcgen05.st; the MMA takes
// its A operand from there), accumulating the row's sum of squares on the way. One elected thread of the leader CTA
// issues the MMAs into a 256-column fp32 accumulator. The row scale 1/RMS does not depend on the contraction index, so
// it multiplies the accumulator in the epilogue: the threads that summed a row's squares read that row out of tensor
// memory, scale, round to bf16 and write it to the Q, K or V tensor its columns belong to.
// Measured on the way (3200 x 2560 x 1024): x rewritten in place in shared memory as the A operand, gate from global
// memory: 29.5 us (shared memory carried 96 KB per step and CTA against the 64 KB it moves in a 512-cycle MMA step, and
// every step waited for an L2 round trip of gate values); x loaded from global memory by the row-owning threads: 40 us
// (32 different cache lines per load instruction).
//
// Any other dtype or shape: a plain kernel (one block per row, fp32 FMAs) with the same semantics.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

using namespace ptx;

namespace {

constexpr int kQkThreads = 64 + 256;   // producer warp, MMA warp, eight transform / epilogue warps (two threads per row)
constexpr int kQkBM = 128;             // rows of x per CTA (256 per pair)
constexpr int kQkBN = 256;             // output columns per pair (each CTA loads 128 rows of W_QKV)
constexpr int kQkBK = 64;              // contraction step: one 128-byte swizzled row of W_QKV
constexpr int kQkStages = 5;
constexpr int kQkColA = kQkBN;         // tensor memory: accumulator in columns [0, 256), A stages of 32 columns behind it
constexpr int kQkTmemCols = 512;
static_assert(kQkColA + kQkStages * (kQkBK / 2) <= kQkTmemCols, "tensor memory budget");
constexpr unsigned long long kQkWaitNs = 1000000000ull;

struct QkSmem {
    static constexpr uint32_t X_STAGE = kQkBM * 128;
    static constexpr uint32_t B_STAGE = (kQkBN / 2) * 128;
    static constexpr uint32_t OFF_X = 0;
    static constexpr uint32_t OFF_B = kQkStages * X_STAGE;
    static constexpr uint32_t OFF_BAR = OFF_B + kQkStages * B_STAGE;
    static constexpr uint32_t OFF_SS = OFF_BAR + 512;         // [2][128] partial sums of squares
    static constexpr uint32_t OFF_GATE = OFF_SS + 1024;       // gates of the streams this CTA's rows belong to, [n][D] fp32
    static constexpr uint32_t GATE_MAX = 48 * 1024;
    static constexpr uint32_t TOTAL = OFF_GATE + GATE_MAX + 1024;   // + slack for the 1024-byte alignment
};
enum { Q_XFULL = 0, Q_BFULL = kQkStages, Q_AREADY = 2 * kQkStages, Q_EMPTY = 3 * kQkStages, Q_ACC = 4 * kQkStages, Q_COUNT };

struct QkParams {
    const float *gate;          // [B][D]
    __nv_bfloat16 *q, *k, *v;   // [M][nq], [M][nk], [M][nk]
    int M, R, B, D, nq, nk;     // M = B * R rows; nq = Hq * d, nk = Hkv * d
    int m_tiles;                // 256-row tiles
    float eps;
    uint32_t *status;
};

#ifdef REFLEX_QK_TRACE
__device__ long long g_qk_trace[3 * 32 * 8];
#define QK_TRACE(role, step, ev) do { if (blockIdx.x == 0 && (step) < 32) g_qk_trace[((role) * 32 + (step)) * 8 + (ev)] = clock64(); } while (0)
#else
#define QK_TRACE(role, step, ev) do { } while (0)
#endif

__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1)
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kQkThreads, 1)
norm_qkv_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, QkParams p)
{
    using S = QkSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    auto bar = [&](int i) -> uint32_t { return base + S::OFF_BAR + 8u * (uint32_t)i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + S::OFF_BAR + 8 * Q_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int m0 = (pair % p.m_tiles) * (2 * kQkBM) + (int)rank * kQkBM;   // this CTA's first row
    const int n0 = (pair / p.m_tiles) * kQkBN;                              // the pair's first output column
    const int nk_steps = p.D / kQkBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQkStages; ++s) {
            mbar_init(bar(Q_XFULL + s), 1);
            mbar_init(bar(Q_BFULL + s), 1);
            mbar_init(bar(Q_AREADY + s), 16);   // one arrival per transform warp of either CTA
            mbar_init(bar(Q_EMPTY + s), 1);
        }
        mbar_init(bar(Q_ACC), 1);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_w);
    }
    if (warp == 1) tmem_alloc2(smem_u32((const void *)tmem_slot), kQkTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // both CTAs' barriers exist before anything crosses the pair
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (threadIdx.x == 64) QK_TRACE(2, 30, 0);
    // programmatic dependent launch: whatever produced x and the gate is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    auto wait = [&](int i, uint32_t parity, uint32_t code) -> bool {
        if (mbar_try_wait(bar(i), parity)) return true;
        const unsigned long long t_start = globaltimer_ns();
        for (uint32_t n = 1;; ++n) {
            if (mbar_try_wait(bar(i), parity)) return true;
            if ((n & 255u) == 0u) {
                if (*abort_flag) return false;
                if (globaltimer_ns() - t_start > kQkWaitNs) break;
            }
        }
        *abort_flag = 1u;
        if (p.status) atomicCAS(p.status, 0u, 0x80000000u | ((code + 96u) << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            bool ok = true;
            for (int ks = 0; ks < nk_steps && ok; ++ks) {
                const int s = ks % kQkStages;
                if (ks >= kQkStages) ok = wait(Q_EMPTY + s, (uint32_t)(ks / kQkStages - 1) & 1u, 1);
                if (!ok) break;
                QK_TRACE(0, ks, 0);
                mbar_expect_tx(bar(Q_XFULL + s), S::X_STAGE);
                tma_load_2d(base + S::OFF_X + s * S::X_STAGE, &tm_x, bar(Q_XFULL + s), ks * kQkBK, m0);
                if (rank == 0) mbar_expect_tx(bar(Q_BFULL + s), 2 * S::B_STAGE);
                tma2_load_2d(base + S::OFF_B + s * S::B_STAGE, &tm_w, bar(Q_BFULL + s) & kPeerBitMask, ks * kQkBK, n0 + (int)rank * (kQkBN / 2));
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA; the warp stays converged, one elected lane issues) ----------------
        if (rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * kQkBM, kQkBN, false);
            bool ok = true;
            for (int ks = 0; ks < nk_steps && ok; ++ks) {
                const int s = ks % kQkStages;
                const uint32_t ph = (uint32_t)(ks / kQkStages) & 1u;
                if (lane == 0) QK_TRACE(1, ks, 0);
                ok = wait(Q_BFULL + s, ph, 2);
                if (lane == 0) QK_TRACE(1, ks, 1);
                ok = ok && wait(Q_AREADY + s, ph, 3);
                if (lane == 0) QK_TRACE(1, ks, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_tmem = tmem + kQkColA + s * (kQkBK / 2);
                uint64_t bd = umma_desc_sw128(base + S::OFF_B + s * S::B_STAGE, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < kQkBK / 16; ++kk) {
                    umma2_ts_elect(tmem, a_tmem + kk * 8, bd, idesc, (ks > 0 || kk > 0) ? 1u : 0u);   // 16 bf16 of K = 8 columns of A
                    umma_desc_advance(bd, 32);
                }
                umma2_commit_mc_elect(bar(Q_EMPTY + s), (uint16_t)3);
                if (lane == 0) QK_TRACE(1, ks, 3);
            }
            umma2_commit_mc_elect(bar(Q_ACC), (uint16_t)3);   // also after a wait that ran out: the epilogue warps must not wait for nothing
        }
    } else {
        // ---------------- gate multiply (A operand) and epilogue: two threads per row ----------------
        // Thread (row, half) owns columns [32 half, 32 half + 32) of the row's 64 in every step, and columns
        // [128 half, 128 half + 128) of the row's accumulator in the epilogue. Two warps per scheduler hide each other's
        // load latencies; the arithmetic is packed (two fp32 per instruction).
        const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const int r_glob = m0 + row;
        const int b = min(r_glob / p.R, p.B - 1);     // (rows past the end contribute zeros and are never stored)
        // the gates of the streams under this CTA's 128 rows go to shared memory once: every step needs 128 fresh bytes of
        // them per thread, and as global loads those were an L2 round trip per step on the critical path
        const int b_first = min(m0 / p.R, p.B - 1), b_last = min((m0 + kQkBM - 1) / p.R, p.B - 1);
        float *gsm = reinterpret_cast<float *>(smem + S::OFF_GATE);
        {
            const int n4 = (b_last - b_first + 1) * p.D / 4;
            const float4 *src = reinterpret_cast<const float4 *>(p.gate + (size_t)b_first * p.D);
            for (int i = threadIdx.x - 64; i < n4; i += 256) reinterpret_cast<float4 *>(gsm)[i] = __ldg(src + i);
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        const float *grow = gsm + (size_t)(b - b_first) * p.D + half * 32;
        const uint32_t leader_aready0 = mapa(bar(Q_AREADY), 0);
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        uint64_t ss2 = 0ull;
        bool ok = true;
        // operands of one step in registers: this thread's half row of x (four 16-byte chunks) and the 32 gate values for it
        struct Ops { uint4 x[4]; ulonglong2 g[8]; };
        auto load = [&](int ks, Ops &o) {
            const int s = ks % kQkStages;
            ok = ok && wait(Q_XFULL + s, (uint32_t)(ks / kQkStages) & 1u, 6);
            const uint8_t *rowp = smem + S::OFF_X + s * S::X_STAGE + row * 128;
#pragma unroll
            for (int c = 0; c < 4; ++c)   // 128-byte swizzle: chunk j of row r sits at j ^ (r % 8)
                o.x[c] = *reinterpret_cast<const uint4 *>(rowp + (((4 * half + c) ^ (row & 7)) << 4));
            const ulonglong2 *g2 = reinterpret_cast<const ulonglong2 *>(grow + ks * kQkBK);
#pragma unroll
            for (int i = 0; i < 8; ++i) o.g[i] = g2[i];
        };
        auto step = [&](int ks, const Ops &o) {
            if (threadIdx.x == 64) QK_TRACE(2, ks, 0);
            const int s = ks % kQkStages;
            uint32_t packed[16];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint64_t gg[4] = {o.g[2 * c].x, o.g[2 * c].y, o.g[2 * c + 1].x, o.g[2 * c + 1].y};
                const uint32_t vv[4] = {o.x[c].x, o.x[c].y, o.x[c].z, o.x[c].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint64_t x2 = pack_f32x2(__uint_as_float(vv[k] << 16), __uint_as_float(vv[k] & 0xFFFF0000u));
                    ss2 = fma_f32x2(x2, x2, ss2);
                    float y0, y1;
                    unpack_f32x2(mul_f32x2(x2, gg[k]), y0, y1);
                    __nv_bfloat162 y2 = __floats2bfloat162_rn(y0, y1);
                    packed[4 * c + k] = *reinterpret_cast<uint32_t *>(&y2);
                }
            }
            if (threadIdx.x == 64) QK_TRACE(2, ks, 1);
            // the A stage is free once the MMAs that read it (kQkStages steps ago) are complete
            if (ks >= kQkStages) {
                ok = ok && wait(Q_EMPTY + s, (uint32_t)(ks / kQkStages - 1) & 1u, 4);
                tc_fence_after();
            }
            if (threadIdx.x == 64) QK_TRACE(2, ks, 2);
            tmem_st16(tmem + lane_addr + kQkColA + s * (kQkBK / 2) + half * 16, packed);
            tmem_wait_st();
            if (threadIdx.x == 64) QK_TRACE(2, ks, 3);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_aready0 + 8u * (uint32_t)s);
            if (threadIdx.x == 64) QK_TRACE(2, ks, 4);
        };
        {
            // the next step's operands are read from shared memory before this step's result is handed over, so their
            // latency runs under the store to tensor memory and the barrier traffic
            Ops oa, ob;
            load(0, oa);
            for (int ks = 0; ks < nk_steps; ks += 2) {       // (the conditions are uniform over the CTA)
                if (ks + 1 < nk_steps) load(ks + 1, ob);
                step(ks, oa);
                if (ks + 2 < nk_steps) load(ks + 2, oa);
                if (ks + 1 < nk_steps) step(ks + 1, ob);
            }
        }
        // the row's sum of squares: both halves meet through shared memory
        float *ssm = reinterpret_cast<float *>(smem + S::OFF_SS);
        {
            float s0, s1;
            unpack_f32x2(ss2, s0, s1);
            ssm[half * 128 + row] = s0 + s1;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const float ss = ssm[row] + ssm[128 + row];
        if (threadIdx.x == 64) QK_TRACE(2, 31, 0);
        ok = wait(Q_ACC, 0u, 5) && ok;
        if (threadIdx.x == 64) QK_TRACE(2, 31, 1);
        tc_fence_after();
        const float rs = rsqrtf(ss / (float)p.D + p.eps);
        const int n_out = p.nq + 2 * p.nk;
        // The tile goes out through shared memory (the stage ring is idle now: every load has been consumed and every MMA
        // has completed): each thread drops its half row, scaled and rounded, as 16-byte pieces at [row][piece ^ (row % 32)]
        // (conflict-free for 32 rows at a time), then every warp writes whole 512-byte rows, 16 bytes per lane. (Straight
        // from registers every store instruction touched 32 rows 4 KB apart: 6.3 k cycles per tile.)
        uint4 *stg = reinterpret_cast<uint4 *>(smem + S::OFF_X);      // [128 rows][32 pieces of 8 columns]
        static_assert(kQkBM * kQkBN * 2 <= (int)(S::OFF_BAR - S::OFF_X), "staging area of the epilogue");
#pragma unroll 1
        for (int c = 0; c < kQkBN / 64; ++c) {
            uint32_t acc[32];
            tmem_ld32(tmem + lane_addr + half * (kQkBN / 2) + c * 32, acc);      // warp-wide: every lane takes part, whatever its row
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 o;
                uint32_t *oo = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[8 * i + 2 * k]) * rs, __uint_as_float(acc[8 * i + 2 * k + 1]) * rs);
                    oo[k] = *reinterpret_cast<uint32_t *>(&h);
                }
                const int piece = half * 16 + c * 4 + i;
                stg[row * 32 + (piece ^ (row & 31))] = o;
            }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        {
            const int n = n0 + lane * 8;            // this lane's 8 columns: they never straddle Q, K and V (head_dim % 8 == 0)
            __nv_bfloat16 *dst0 = nullptr;          // column n of row 0 of the tensor it belongs to
            size_t pitch = 0;
            if (n < p.nq) { dst0 = p.q + n; pitch = (size_t)p.nq; }
            else if (n < p.nq + p.nk) { dst0 = p.k + (n - p.nq); pitch = (size_t)p.nk; }
            else if (n < n_out) { dst0 = p.v + (n - p.nq - p.nk); pitch = (size_t)p.nk; }
            const int w8 = warp - 2;                // 0..7: rows w8, w8 + 8, ...
            if (ok && dst0) {
#pragma unroll 4
                for (int r = w8; r < kQkBM; r += 8) {
                    if (m0 + r >= p.M) break;
                    *reinterpret_cast<uint4 *>(dst0 + (size_t)(m0 + r) * pitch) = stg[r * 32 + (lane ^ (r & 31))];
                }
            }
        }
    }

    if (threadIdx.x == 64) QK_TRACE(2, 31, 2);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // neither CTA retires while its partner can still touch its shared memory or barriers
    if (warp == 1) tmem_dealloc2(tmem, kQkTmemCols);
}

// Any dtype, any shape: one block per row. y = x * gamma / RMS(x) in shared memory (fp32), then every thread takes output
// features n = tid, tid + 256, ... as plain dot products.
template <typename T>
__device__ __forceinline__ float qk_to_f(T v);
template <> __device__ __forceinline__ float qk_to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float qk_to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T qk_from_f(float v);
template <> __device__ __forceinline__ float qk_from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 qk_from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256)
norm_qkv_simt_kernel(const T *__restrict__ x, const float *__restrict__ gate, const T *__restrict__ W, T *q, T *k, T *v,
                     int R, int D, int nq, int nk, float eps)
{
    extern __shared__ float ysm[];    // [D] + 8 partial sums
    float *part = ysm + D;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t r = blockIdx.x;
    const int b = (int)(r / (size_t)R);
    const T *xr = x + r * D;
    float ss = 0.f;
    for (int i = threadIdx.x; i < D; i += blockDim.x) {
        const float xv = qk_to_f<T>(xr[i]);
        ysm[i] = xv * gate[(size_t)b * D + i];
        ss = fmaf(xv, xv, ss);
    }
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += part[w];
    const float rs = rsqrtf(tot / (float)D + eps);
    const int n_out = nq + 2 * nk;
    for (int n = threadIdx.x; n < n_out; n += blockDim.x) {
        const T *wr = W + (size_t)n * D;
        float acc = 0.f;
        for (int i = 0; i < D; ++i) acc = fmaf(ysm[i], qk_to_f<T>(wr[i]), acc);
        acc *= rs;
        if (n < nq) q[r * nq + n] = qk_from_f<T>(acc);
        else if (n < nq + nk) k[r * nk + (n - nq)] = qk_from_f<T>(acc);
        else v[r * nk + (n - nq - nk)] = qk_from_f<T>(acc);
    }
}

template <typename T>
cudaError_t launch_simt(const void *x, const float *gate, const void *W, void *q, void *k, void *v, int M, int R, int D, int nq, int nk, float eps,
                        cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = (size_t)(D + 8) * sizeof(float);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, norm_qkv_simt_kernel<T>, (const T *)x, gate, (const T *)W, (T *)q, (T *)k, (T *)v, R, D, nq, nk, eps);
    count_launch();
    return e;
}

}  // namespace

bool norm_qkv_tc_supported(int dtype, int B, int R, int D, int nq, int nk)
{
    if (dtype != REFLEX_DTYPE_BF16 || B < 1 || R < 1) return false;
    if (D < kQkBK || D % kQkBK != 0) return false;
    if (nq % 8 != 0 || nk % 8 != 0) return false;
    if ((size_t)((kQkBM - 1) / R + 2) * D * sizeof(float) > QkSmem::GATE_MAX) return false;   // gates of a CTA's streams in shared memory
    const long long pairs = ((long long)B * R + 2 * kQkBM - 1) / (2 * kQkBM) * ((nq + 2 * nk + kQkBN - 1) / kQkBN);
    return pairs <= 0x3FFFFFFF;
}

cudaError_t launch_adarmsnorm_qkv(const void *x, const float *gate, const void *Wqkv, void *q, void *k, void *v, int B, int R, int D, int nq, int nk,
                                  float eps, int dtype, int impl, uint32_t *status, cudaStream_t st)
{
    const int M = B * R;
    const bool tc = impl != 1 && norm_qkv_tc_supported(dtype, B, R, D, nq, nk);
    if (!tc) {
        if ((size_t)(D + 8) * sizeof(float) > 48 * 1024) return cudaErrorInvalidValue;
        return dtype == REFLEX_DTYPE_BF16 ? launch_simt<__nv_bfloat16>(x, gate, Wqkv, q, k, v, M, R, D, nq, nk, eps, st)
                                          : launch_simt<float>(x, gate, Wqkv, q, k, v, M, R, D, nq, nk, eps, st);
    }
    CUtensorMap mx, mw;
    if (!tensor_map_2d_bf16(&mx, x, D, M, kQkBM) || !tensor_map_2d_bf16(&mw, Wqkv, D, nq + 2 * nk, kQkBN / 2)) return cudaErrorInvalidValue;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(norm_qkv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QkSmem::TOTAL);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    QkParams p;
    p.gate = gate; p.q = (__nv_bfloat16 *)q; p.k = (__nv_bfloat16 *)k; p.v = (__nv_bfloat16 *)v;
    p.M = M; p.R = R; p.B = B; p.D = D; p.nq = nq; p.nk = nk;
    p.m_tiles = (M + 2 * kQkBM - 1) / (2 * kQkBM);
    p.eps = eps; p.status = status;
    const int n_tiles = (nq + 2 * nk + kQkBN - 1) / kQkBN;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * (unsigned)p.m_tiles * (unsigned)n_tiles);
    cfg.blockDim = dim3(kQkThreads);
    cfg.dynamicSmemBytes = QkSmem::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, norm_qkv_tc_kernel, mx, mw, p);
    count_launch();
    return e;
}

}  // namespace reflex

#ifdef REFLEX_QK_TRACE
extern "C" int reflex_debug_qk_trace(long long *out)
{
    return (int)cudaMemcpyFromSymbol(out, reflex::g_qk_trace, sizeof(long long) * 3 * 32 * 8);
}
#endif
