// Gate MLP of AdaRMSNorm (Eq. 2) on the tensor cores: gamma_l(c) = 1 + W2_l SiLU(W1_l c + b1_l) + b2_l for L layers
// (stacked weights) and B streams, bf16 weights and conditioning vectors.
//
// Both layers of the MLP are the same small GEMM, out[b][u] = act(bias[u] + sum_k W[u][k] vec[b][k]): one CTA takes 128
// weight rows (the M of a tcgen05.mma, K-major A operand) and up to 64 streams (N, K-major B operand), loads both
// operands whole with TMA (80 KB + 40 KB at the paper's widths), issues len/16 MMAs into a 64-column accumulator in
// tensor memory and finishes with one thread per weight row. bf16 x bf16 products are exact in the fp32 accumulator. The
// hidden activations go to the second layer as two bf16 arrays, hi = bf16(h) and lo = bf16(h - hi) (two passes of MMAs,
// about 17 bits of h), in the space the fp32 hidden activations of the FMA kernels take.
//
// Why not CUDA cores: the whole MLP is 0.8 GFLOP per denoising step at 64 streams, but as fp32 FMAs fed from shared
// memory it took 45 us per step (27 us for a single stream); mma.sync runs at a small fraction of tcgen05's rate on
// this part (82 us). Here the cost is the 12 MB of weights and the latency of one load-compute-store round.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

using namespace ptx;

namespace {

constexpr int kGtUnits = 128;     // weight rows per CTA
constexpr int kGtStreams = 64;    // streams per CTA
constexpr int kGtMaxChunks = 5;   // 64-column chunks of the contraction axis held in shared memory (len <= 320)
constexpr uint32_t kGtWaitNs = 1000000000u;

struct GateTcSmem {
    static constexpr uint32_t A_CHUNK = kGtUnits * 128;      // 128 rows x 64 bf16
    static constexpr uint32_t B_CHUNK = kGtStreams * 128;    // 64 rows x 64 bf16
    static constexpr uint32_t OFF_A = 0;
    static constexpr uint32_t OFF_B = kGtMaxChunks * A_CHUNK;                  // two passes (hi, lo) of B chunks
    static constexpr uint32_t OFF_BAR = OFF_B + 2 * kGtMaxChunks * B_CHUNK;
    static constexpr uint32_t TOTAL = OFF_BAR + 64 + 1024;                     // + slack for the 1024-byte alignment
};

// SILU: first layer (writes hi/lo bf16 hidden activations); else second layer (writes fp32 gates 1 + z). PASSES: 1 = one
// bf16 vector per stream (tm_v0), 2 = hi and lo halves (tm_v0, tm_v1).
template <bool SILU, int PASSES>
__global__ void __launch_bounds__(128, 1)
gate_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_v0, const __grid_constant__ CUtensorMap tm_v1,
               const __nv_bfloat16 *__restrict__ bias, float *out_f32, __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int B, int len, int units,
               int vec_rows_per_layer, uint32_t *status)
{
    using S = GateTcSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar_load = base + S::OFF_BAR, bar_mma = bar_load + 8;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + S::OFF_BAR + 16);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int layer = blockIdx.z, u0 = blockIdx.x * kGtUnits;
    const int chunks = (len + 63) / 64, ksteps = len / 16;
    // A CTA keeps its 128 weight rows in shared memory and walks the groups of 64 streams that fall to it (blockIdx.y takes
    // a contiguous share of the groups): with many streams -- the conditioning vectors of all steps of a control tick
    // stacked -- the weights are fetched once per CTA instead of once per group, and the next group's vectors come in
    // while this group's results are stored.
    const int n_groups = (B + kGtStreams - 1) / kGtStreams;
    const int gpc = (n_groups + (int)gridDim.y - 1) / (int)gridDim.y;
    const int g_first = (int)blockIdx.y * gpc;
    const int ng = max(0, min(n_groups, g_first + gpc) - g_first);

    if (threadIdx.x == 0) {
        mbar_init(bar_load, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        prefetch_tmap(&tm_w); prefetch_tmap(&tm_v0);
        if (PASSES == 2) prefetch_tmap(&tm_v1);
    }
    if (warp == 0) tmem_alloc(smem_u32((const void *)tmem_slot), 64);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // programmatic dependent launch: the first layer's output (second kernel) or whatever precedes the call is complete
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    auto wait = [&](uint32_t bar, uint32_t parity, uint32_t code) -> bool {
        if (mbar_try_wait(bar, parity)) return true;
        const unsigned long long t_start = globaltimer_ns();
        for (uint32_t n = 1;; ++n) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((n & 255u) == 0u && globaltimer_ns() - t_start > kGtWaitNs) break;
        }
        if (status) atomicCAS(status, 0u, 0x80000000u | ((code + 64u) << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };
    auto load_vectors = [&](int g) {   // the (up to) 64 vectors of group g, one or two bf16 arrays
        for (int c = 0; c < chunks; ++c) {
            tma_load_2d(base + S::OFF_B + c * S::B_CHUNK, &tm_v0, bar_load, c * 64, layer * vec_rows_per_layer + g * kGtStreams);
            if (PASSES == 2)
                tma_load_2d(base + S::OFF_B + (kGtMaxChunks + c) * S::B_CHUNK, &tm_v1, bar_load, c * 64, layer * vec_rows_per_layer + g * kGtStreams);
        }
    };

    bool ok = true;
    if (warp == 0 && lane == 0 && ng > 0) {
        mbar_expect_tx(bar_load, (uint32_t)chunks * (S::A_CHUNK + PASSES * S::B_CHUNK));
        for (int c = 0; c < chunks; ++c) tma_load_2d(base + S::OFF_A + c * S::A_CHUNK, &tm_w, bar_load, c * 64, layer * units + u0);
        load_vectors(g_first);
    }
    const int u = u0 + warp * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    const float bi = u < units ? __bfloat162float(bias[(size_t)layer * units + u]) : 0.f;
#pragma unroll 1
    for (int i = 0; i < ng; ++i) {
        const int b0 = (g_first + i) * kGtStreams;
        const uint32_t ph = (uint32_t)i & 1u;
        if (warp == 0) {
            // the whole warp stays converged; one elected lane issues
            ok = ok && wait(bar_load, ph, 1);
            tc_fence_after();
            if (ok) {
                constexpr uint32_t idesc = umma_idesc_bf16(kGtUnits, kGtStreams, false);
#pragma unroll 1
                for (int pass = 0; pass < PASSES; ++pass) {
#pragma unroll 1
                    for (int kk = 0; kk < ksteps; ++kk) {
                        const uint32_t a = base + S::OFF_A + (kk >> 2) * S::A_CHUNK + (kk & 3) * 32;
                        const uint32_t b = base + S::OFF_B + (pass * kGtMaxChunks + (kk >> 2)) * S::B_CHUNK + (kk & 3) * 32;
                        umma_ss_elect(tmem, umma_desc_sw128(a, 16, 1024), umma_desc_sw128(b, 16, 1024), idesc, (pass > 0 || kk > 0) ? 1u : 0u);
                    }
                }
            }
            umma_commit_elect(bar_mma);   // also when the load never came: the other warps must not wait for nothing
        }
        ok = wait(bar_mma, ph, 2) && ok;
        tc_fence_after();
        // the MMAs that read this group's vectors are complete: the next group's may land on them
        if (warp == 0 && lane == 0 && i + 1 < ng) {
            mbar_expect_tx(bar_load, (uint32_t)chunks * (PASSES * S::B_CHUNK));
            load_vectors(g_first + i + 1);
        }
        // epilogue: thread = weight row (TMEM lane), 64 columns = streams
        uint32_t acc[64];
        tmem_ld32(tmem + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(acc));
        tmem_ld32(tmem + lane_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(acc + 32));
        tmem_wait_ld();
        tc_fence_before();
        __syncthreads();      // every warp holds its accumulators in registers: the next group's MMAs may overwrite them
        const int nb = min(kGtStreams, B - b0);
        if (!ok && u < units) {
            // a bounded wait ran out: this CTA's slice of the output is marked invalid (quiet NaN) instead of keeping the
            // previous call's values, so whatever consumes the gates shows it
            for (int n = 0; n < nb; ++n) {
                const size_t o = ((size_t)layer * B + b0 + n) * units + u;
                if (SILU) { out_hi[o] = __float2bfloat16_rn(__int_as_float(0x7fc00000)); out_lo[o] = __float2bfloat16_rn(0.f); }
                else out_f32[o] = __int_as_float(0x7fc00000);
            }
        }
        if (ok && u < units) {
#pragma unroll
            for (int n = 0; n < kGtStreams; ++n) {
                if (n >= nb) continue;   // (fully unrolled: the accumulator stays in registers)
                const float z = __uint_as_float(acc[n]) + bi;
                const size_t o = ((size_t)layer * B + b0 + n) * units + u;
                if (SILU) {
                    const float h = z / (1.f + expf(-z));
                    const __nv_bfloat16 hi = __float2bfloat16_rn(h);
                    out_hi[o] = hi;
                    out_lo[o] = __float2bfloat16_rn(h - __bfloat162float(hi));
                } else {
                    out_f32[o] = 1.f + z;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 64);
}

template <bool SILU, int PASSES>
cudaError_t launch_one(const CUtensorMap &mw, const CUtensorMap &mv0, const CUtensorMap &mv1, const __nv_bfloat16 *bias, float *out_f32,
                       __nv_bfloat16 *out_hi, __nv_bfloat16 *out_lo, int L, int B, int len, int units, int vec_rows_per_layer, cudaStream_t st)
{
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        return cudaFuncSetAttribute(gate_tc_kernel<SILU, PASSES>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GateTcSmem::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    cudaLaunchConfig_t cfg = {};
    // groups of 64 streams are spread over blockIdx.y only as far as that adds CTAs the SMs can hold at once; beyond, a CTA
    // walks several groups with its weights resident
    const int ux = (units + kGtUnits - 1) / kGtUnits, n_groups = (B + kGtStreams - 1) / kGtStreams;
    int gy = 148 / (ux * L);
    gy = gy < 1 ? 1 : (gy > n_groups ? n_groups : gy);
    cfg.gridDim = dim3(ux, gy, L);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = GateTcSmem::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gate_tc_kernel<SILU, PASSES>, mw, mv0, mv1, bias, out_f32, out_hi, out_lo, B, len, units,
                                       vec_rows_per_layer, (uint32_t *)nullptr);
    count_launch();
    return e;
}

}  // namespace

bool gate_tc_supported(int B, int D, int Cd, int Hd)
{
    if (B < 1 || Cd % 16 != 0 || Hd % 16 != 0 || Cd > 64 * kGtMaxChunks || Hd > 64 * kGtMaxChunks) return false;
    return D % 8 == 0;
}

cudaError_t launch_gate_tc(const void *cond, const void *W1, const void *b1, const void *W2, const void *b2, float *gate_buf, int L, int B,
                           int D, int Cd, int Hd, cudaStream_t st)
{
    // scratch behind the gates: hi and lo halves of the hidden activations, [L][B][Hd] bf16 each (the space of [L][B][Hd] floats)
    __nv_bfloat16 *hid_hi = reinterpret_cast<__nv_bfloat16 *>(gate_buf + (size_t)L * B * D);
    __nv_bfloat16 *hid_lo = hid_hi + (size_t)L * B * Hd;
    CUtensorMap mw1, mw2, mc, mhi, mlo;
    if (!tensor_map_2d_bf16(&mw1, W1, Cd, L * Hd, kGtUnits) || !tensor_map_2d_bf16(&mw2, W2, Hd, L * D, kGtUnits) ||
        !tensor_map_2d_bf16(&mc, cond, Cd, B, kGtStreams) || !tensor_map_2d_bf16(&mhi, hid_hi, Hd, L * B, kGtStreams) ||
        !tensor_map_2d_bf16(&mlo, hid_lo, Hd, L * B, kGtStreams))
        return cudaErrorInvalidValue;
    cudaError_t e = launch_one<true, 1>(mw1, mc, mc, (const __nv_bfloat16 *)b1, nullptr, hid_hi, hid_lo, L, B, Cd, Hd, 0, st);
    if (e != cudaSuccess) return e;
    return launch_one<false, 2>(mw2, mhi, mlo, (const __nv_bfloat16 *)b2, gate_buf, nullptr, nullptr, L, B, Hd, D, B, st);
}

}  // namespace reflex
