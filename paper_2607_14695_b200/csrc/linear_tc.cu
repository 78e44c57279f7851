// A plain projection of the action expert with its residual connection (Sec. 3.3 names the expert's linear layers; the
// attention output projection and the down projection of the SwiGLU block each add their result to the residual stream):
//     out[r][n] = res[r][n] + sum_i a[r][i] * W[n][i]
//
// bf16 path: one pair of CTAs (tcgen05.mma.cta_group::2, M = 256) per 256 x 256 output tile. Each CTA stages its own 128
// rows of a and its 128 rows of W (its half of the B operand) per 64-column contraction step through a ring of five
// 32 KB stages filled by TMA; one elected thread of the leader CTA issues the MMAs into a 256-column fp32 accumulator in
// tensor memory. The residual tile (128 rows x 256 columns, 64 KB) comes in by TMA behind the last operand tiles into a
// buffer of its own; the epilogue threads (two per row) take it into registers while the last stages are multiplied, add
// the accumulator (fp32 add, one rounding to bf16) and write the result back into the same buffer, which leaves through
// TMA stores (they clip rows and columns past the end). out may alias res: a tile is read and written by one CTA only.
// What bounds the kernel: without multicast every CTA fetches its own operand tiles, 32 KB per contraction step against
// 512 cycles of MMAs = 64 B/clk, and an SM takes in 50 to 58 B/clk from the L2: 10.75 us for the main loop of the
// 3200 x 1024 x 2048 problem against 8.3 us of tensor-pipe time.
// The contraction is long (2048 or 4096) and the output small (3200 x 1024 at 64 streams): 52 tiles on 74 SM pairs in
// one wave, so the kernel is not persistent.
//
// Few rows (at most 128 in all): the weights-as-A-operand kernel of the fused projections with the gate stage switched off
// (qkv_tc.cu). Any other dtype or shape: a plain kernel, one block per row, fp32 FMAs.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

using namespace ptx;

namespace {

constexpr int kLinThreads = 64 + 256;   // producer warp, MMA warp, eight epilogue warps (two threads per row)
constexpr int kLinBM = 128;             // rows per CTA (256 per pair)
constexpr int kLinBK = 64;              // contraction step: one 128-byte swizzled row
constexpr unsigned long long kLinWaitNs = 1000000000ull;

template <int BN>
struct LinSmem {
    static constexpr int NST = 5;
    static constexpr uint32_t A_STAGE = kLinBM * 128;
    static constexpr uint32_t B_STAGE = (BN / 2) * 128;            // this CTA's half of the B operand: BN / 2 rows of W
    static constexpr uint32_t CHUNK = kLinBM * 128;                // 128 rows x 64 columns of the residual / output tile
    static constexpr uint32_t OFF_A = 0;
    static constexpr uint32_t OFF_B = NST * A_STAGE;
    static constexpr uint32_t OFF_RES = OFF_B + NST * B_STAGE;
    static constexpr uint32_t RES_BYTES = (BN / 64) * CHUNK;
    static constexpr uint32_t OFF_BAR = OFF_RES + RES_BYTES;
    static constexpr uint32_t TOTAL = OFF_BAR + 256 + 1024;        // + slack for the 1024-byte alignment
    static constexpr int C_FULL = 0, C_EMPTY = NST, C_ACC = 2 * NST, C_RES = 2 * NST + 1, C_COUNT = 2 * NST + 2;
    static_assert(TOTAL <= 227u * 1024u && 8 * C_COUNT + 8 <= 256, "shared memory budget");
};

struct LinParams {
    int M, K, N;
    int m_tiles;          // 256-row tiles
    int has_res;
    uint32_t *status;     // status word of a cache, or NULL
};

// Optional timeline (debug builds only: -DREFLEX_LIN_TRACE): %globaltimer stamps of every CTA's milestones.
#ifdef REFLEX_LIN_TRACE
__device__ unsigned long long g_lin_trace[512 * 8];
#define LIN_TRACE(ev) do { if (blockIdx.x < 512) g_lin_trace[blockIdx.x * 8 + (ev)] = globaltimer_ns(); } while (0)
#else
#define LIN_TRACE(ev) do { } while (0)
#endif

__device__ __forceinline__ void lin_tma2_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void lin_tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}

// KS = 2 (128-column tiles only): the cluster holds the two pairs that share an output tile, each taking half of the contraction;
// at the end every CTA stages the 64 columns its counterpart in the other pair finishes as fp32 in the idle stage ring, and takes
// the counterpart's share of its own 64 columns from there through distributed shared memory. Launched with the cluster shape as
// a launch attribute (2 KS CTAs).
template <int BN, int KS>
__global__ void __launch_bounds__(kLinThreads, 1)
linear_res_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                     const __grid_constant__ CUtensorMap tm_res, const __grid_constant__ CUtensorMap tm_out, LinParams p)
{
    static_assert(KS == 1 || (KS == 2 && BN == 128), "contraction split");
    using S = LinSmem<BN>;
    constexpr int NST = S::NST;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    auto bar = [&](int i) -> uint32_t { return base + S::OFF_BAR + 8u * (uint32_t)i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + S::OFF_BAR + 8 * S::C_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = cluster_ctarank();
    const uint32_t rank = crank & 1u;                                        // rank inside the pair
    const int kq = KS > 1 ? (int)(crank >> 1) : 0;                           // which part of the contraction this pair takes
    const uint16_t pair_mask = (uint16_t)(3u << (crank & ~1u));              // both CTAs of this pair, for multicast commits
    const int pair = blockIdx.x / (2 * KS);                                  // output tile
    const int m0 = (pair % p.m_tiles) * (2 * kLinBM) + (int)rank * kLinBM;   // this CTA's first row
    const int n0 = (pair / p.m_tiles) * BN;                                  // the tile's first output column
    const int nk_steps = ((p.K + kLinBK - 1) / kLinBK) / KS;                 // (columns past K come in as TMA's zeros; KS = 2: an even count)
    const int k_first = kq * nk_steps;
    if (threadIdx.x == 64) LIN_TRACE(0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < S::C_COUNT; ++i) mbar_init(bar(i), 1);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_a); prefetch_tmap(&tm_w); prefetch_tmap(&tm_out);
        if (p.has_res) prefetch_tmap(&tm_res);
    }
    if (warp == 1) tmem_alloc2(smem_u32((const void *)tmem_slot), BN);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // both CTAs' barriers exist before anything crosses the pair
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (threadIdx.x == 64) LIN_TRACE(1);
    // programmatic dependent launch: whatever produced a and res is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 64) LIN_TRACE(2);

    auto wait = [&](int i, uint32_t parity, uint32_t code) -> bool {
        if (mbar_try_wait(bar(i), parity)) return true;
        const unsigned long long t_start = globaltimer_ns();
        for (uint32_t n = 1;; ++n) {
            if (mbar_try_wait(bar(i), parity)) return true;
            if ((n & 255u) == 0u) {
                if (*abort_flag) return false;
                if (globaltimer_ns() - t_start > kLinWaitNs) break;
            }
        }
        *abort_flag = 1u;
        if (p.status) atomicCAS(p.status, 0u, 0x80000000u | ((code + 80u) << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };

    [[maybe_unused]] bool split_ok = true;     // (KS = 2) this thread's waits all came through

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            bool ok = true;
            for (int ks = 0; ks < nk_steps && ok; ++ks) {
                const int s = ks % NST;
                if (ks >= NST) ok = wait(S::C_EMPTY + s, (uint32_t)(ks / NST - 1) & 1u, 1);
                if (!ok) break;
                // both CTAs' loads complete on the leader's barrier: the issuing thread there waits for all four at once
                if (rank == 0) mbar_expect_tx(bar(S::C_FULL + s), 2 * (S::A_STAGE + S::B_STAGE));
                lin_tma2_load_2d(base + S::OFF_A + s * S::A_STAGE, &tm_a, bar(S::C_FULL + s) & kPeerBitMask, (k_first + ks) * kLinBK, m0);
                lin_tma2_load_2d(base + S::OFF_B + s * S::B_STAGE, &tm_w, bar(S::C_FULL + s) & kPeerBitMask, (k_first + ks) * kLinBK, n0 + (int)rank * (BN / 2));
            }
            if (ok) {
                // the residual tile goes last: it is not needed before the epilogue, and ahead of the main loop's operands it
                // would hold them up for the time 64 KB take to come in (measured: 0.7 us per launch)
                if (p.has_res && KS > 1) {       // (only the 64 columns this CTA finishes)
                    mbar_expect_tx(bar(S::C_RES), S::CHUNK);
                    tma_load_2d(base + S::OFF_RES + kq * S::CHUNK, &tm_res, bar(S::C_RES), n0 + kq * 64, m0);
                } else if (p.has_res) {
                    mbar_expect_tx(bar(S::C_RES), S::RES_BYTES);
#pragma unroll
                    for (int ch = 0; ch < BN / 64; ++ch) tma_load_2d(base + S::OFF_RES + ch * S::CHUNK, &tm_res, bar(S::C_RES), n0 + ch * 64, m0);
                } else {
                    mbar_arrive(bar(S::C_RES));
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA; the warp stays converged, one elected lane issues) ----------------
        if (rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * kLinBM, BN, false);
            bool ok = true;
            for (int ks = 0; ks < nk_steps && ok; ++ks) {
                const int s = ks % NST;
                ok = wait(S::C_FULL + s, (uint32_t)(ks / NST) & 1u, 2);
                if (!ok) break;
                if (ks == 0 && lane == 0) LIN_TRACE(3);
                tc_fence_after();
                uint64_t ad = umma_desc_sw128(base + S::OFF_A + s * S::A_STAGE, 16, 1024);
                uint64_t bd = umma_desc_sw128(base + S::OFF_B + s * S::B_STAGE, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < kLinBK / 16; ++kk) {
                    umma2_ss_elect(tmem, ad, bd, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                    umma_desc_advance(ad, 32);
                    umma_desc_advance(bd, 32);
                }
                umma2_commit_mc_elect(bar(S::C_EMPTY + s), pair_mask);
            }
            umma2_commit_mc_elect(bar(S::C_ACC), pair_mask);   // also after a wait that ran out: the epilogue warps must not wait for nothing
        }
    } else {
        // ---------------- epilogue: two threads per row, each owns BN / 2 columns ----------------
        const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        // The residual tile comes in by TMA behind the last operand tiles; every thread takes its BN / 2 columns of its row
        // out of shared memory into registers while the last stages are multiplied, so that after the accumulator is final
        // only tensor-memory loads, adds and the stores into the same staging buffer remain. (As global loads by these
        // threads, 16 bytes per row and instruction, the residual cost the main loop 2.5 us: what an SM takes in from
        // the L2 is what limits this kernel, and half-used sectors waste it.)
        bool ok = wait(S::C_RES, 0u, 3);
        if constexpr (KS > 1) {
            // Contraction split: thread (row, half) holds this pair's share of columns [64 half, 64 half + 64) of its row. The
            // half that the counterpart CTA (same rank, other pair) finishes goes to shared memory as fp32, 16-byte pieces at
            // [row][piece ^ (row % 16)]; the other half stays in tensor memory until the cluster has met.
            ok = wait(S::C_ACC, 0u, 4) && ok;
            if (threadIdx.x == 64) LIN_TRACE(4);
            tc_fence_after();
            split_ok = ok;
            if (half != kq) {
                uint4 *stage = reinterpret_cast<uint4 *>(smem + S::OFF_A);     // [128 rows][16 pieces]; the stage ring is idle
                static_assert(S::NST * S::A_STAGE >= 128u * 64u * 4u, "staging area of the split");
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t acc[32];
                    tmem_ld32(tmem + lane_addr + half * 64 + g * 32, acc);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        stage[row * 16 + ((g * 8 + i) ^ (row & 15))] = ok ? make_uint4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3])
                                                                           : make_uint4(0x7fc00000u, 0x7fc00000u, 0x7fc00000u, 0x7fc00000u);
                }
            }
        } else {
        constexpr int CPT = BN / 2 / 64;              // 64-column chunks per thread
        uint4 rr[CPT * 8];
#pragma unroll
        for (int j = 0; j < CPT * 8; ++j) {
            // 128-byte swizzle of the TMA box: 16-byte piece j of row r sits at j ^ (r % 8)
            rr[j] = make_uint4(0u, 0u, 0u, 0u);
            if (p.has_res) rr[j] = *reinterpret_cast<const uint4 *>(smem + S::OFF_RES + (half * CPT + j / 8) * S::CHUNK + row * 128 + (((j & 7) ^ (row & 7)) << 4));
        }
        ok = wait(S::C_ACC, 0u, 4) && ok;
        if (threadIdx.x == 64) LIN_TRACE(4);
        tc_fence_after();
#pragma unroll
        for (int cc = 0; cc < CPT; ++cc) {
            const int ch = half * CPT + cc;
            uint8_t *rowp = smem + S::OFF_RES + ch * S::CHUNK + row * 128;
#pragma unroll
            for (int g = 0; g < 2; ++g) {             // 32 columns at a time
                uint32_t acc[32];
                tmem_ld32(tmem + lane_addr + ch * 64 + g * 32, acc);   // warp-wide: every lane takes part, whatever its row
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 t = rr[cc * 8 + g * 4 + i];
                    const uint32_t rv[4] = {t.x, t.y, t.z, t.w};
                    uint32_t ov[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float v0 = __uint_as_float(acc[8 * i + 2 * k]) + __uint_as_float(rv[k] << 16);
                        float v1 = __uint_as_float(acc[8 * i + 2 * k + 1]) + __uint_as_float(rv[k] & 0xFFFF0000u);
                        if (!ok) v0 = v1 = __int_as_float(0x7fc00000);   // a wait ran out: the tile is marked invalid, not left stale
                        __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                        ov[k] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    // 128-byte swizzle of the TMA box: 16-byte piece j of row r sits at j ^ (r % 8)
                    *reinterpret_cast<uint4 *>(rowp + (((g * 4 + i) ^ (row & 7)) << 4)) = make_uint4(ov[0], ov[1], ov[2], ov[3]);
                }
            }
            // this half's chunk is complete once its 128 threads are through: one of them hands it to the TMA engine
            fence_proxy_async_smem();
            asm volatile("bar.sync %0, 128;" ::"r"(1 + half) : "memory");
            if (quarter == 0 && lane == 0 && m0 < p.M && n0 + ch * 64 < p.N) {
                lin_tma_store_2d(&tm_out, base + S::OFF_RES + ch * S::CHUNK, n0 + ch * 64, m0);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        }
        if (threadIdx.x == 64) LIN_TRACE(5);
        // (the staging buffer has been read; the writes themselves are complete when the grid is)
        if (quarter == 0 && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        if (warp == 4 && lane == 0) LIN_TRACE(6);
        }
    }

    if constexpr (KS > 1) {
        // (cluster barriers are warp-aligned: the lanes of the producer warp that idled while lane 0 ran the loads must not
        // reach them before lane 0 does, so the CTA meets first)
        __syncthreads();
        cluster_arrive();
        cluster_wait();       // every CTA's staged half is in place
        if (warp >= 2) {
            // both threads of a row finish 32 of the 64 columns each
            const int half = (warp - 2) >> 2;
            const int quarter = warp & 3, row = quarter * 32 + lane;
            const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
            // the counterpart's share of this thread's 32 columns: 8 loads through distributed shared memory, all in flight
            const uint32_t peer = crank ^ 2u;
            const uint32_t st0 = base + S::OFF_A + (uint32_t)row * 256u;
            float4 pv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t a = mapa(st0 + (uint32_t)(((half * 8 + j) ^ (row & 15)) << 4), peer);
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(pv[j].x), "=f"(pv[j].y), "=f"(pv[j].z), "=f"(pv[j].w) : "r"(a) : "memory");
            }
            uint8_t *rowp = smem + S::OFF_RES + kq * S::CHUNK + row * 128;     // residual in, output out: one chunk of 64 columns
            uint4 rr[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                rr[j] = make_uint4(0u, 0u, 0u, 0u);
                if (p.has_res) rr[j] = *reinterpret_cast<const uint4 *>(rowp + (((half * 4 + j) ^ (row & 7)) << 4));
            }
            tc_fence_after();
            uint32_t acc[32];
            tmem_ld32(tmem + lane_addr + kq * 64 + half * 32, acc);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 t = rr[i];
                const uint32_t rv[4] = {t.x, t.y, t.z, t.w};
                const float4 q0 = pv[2 * i], q1 = pv[2 * i + 1];
                const float pp[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
                uint32_t ov[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float v0 = __uint_as_float(acc[8 * i + 2 * k]) + pp[2 * k] + __uint_as_float(rv[k] << 16);
                    float v1 = __uint_as_float(acc[8 * i + 2 * k + 1]) + pp[2 * k + 1] + __uint_as_float(rv[k] & 0xFFFF0000u);
                    if (!split_ok) v0 = v1 = __int_as_float(0x7fc00000);
                    __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                    ov[k] = *reinterpret_cast<uint32_t *>(&h);
                }
                *reinterpret_cast<uint4 *>(rowp + (((half * 4 + i) ^ (row & 7)) << 4)) = make_uint4(ov[0], ov[1], ov[2], ov[3]);
            }
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 256;" ::: "memory");     // the chunk's 256 threads
            if (warp == 2 && lane == 0) {
                if (m0 < p.M && n0 + kq * 64 < p.N) {
                    lin_tma_store_2d(&tm_out, base + S::OFF_RES + kq * S::CHUNK, n0 + kq * 64, m0);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // no CTA retires while another can still touch its shared memory or barriers
    if (warp == 1) tmem_dealloc2(tmem, BN);
    if (threadIdx.x == 64) LIN_TRACE(7);
}

// Any dtype, any shape: one block per row; the row of a in shared memory (fp32), every thread takes output features
// n = tid, tid + 256, ... as plain dot products.
template <typename T> __device__ __forceinline__ float lin_to_f(T v);
template <> __device__ __forceinline__ float lin_to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float lin_to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T lin_from_f(float v);
template <> __device__ __forceinline__ float lin_from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 lin_from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256)
linear_res_simt_kernel(const T *__restrict__ a, const T *__restrict__ W, const T *res, T *out, int K, int N)
{
    extern __shared__ float asm_row[];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const size_t r = blockIdx.x;
    for (int i = threadIdx.x; i < K; i += blockDim.x) asm_row[i] = lin_to_f<T>(a[r * K + i]);
    __syncthreads();
    for (int n = threadIdx.x; n < N; n += blockDim.x) {
        const T *wr = W + (size_t)n * K;
        float acc = 0.f;
        for (int i = 0; i < K; ++i) acc = fmaf(asm_row[i], lin_to_f<T>(wr[i]), acc);
        if (res) acc += lin_to_f<T>(res[r * N + n]);
        out[r * N + n] = lin_from_f<T>(acc);
    }
}

template <typename T>
cudaError_t launch_lin_simt(const void *a, const void *W, const void *res, void *out, int M, int K, int N, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = (size_t)K * sizeof(float);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, linear_res_simt_kernel<T>, (const T *)a, (const T *)W, (const T *)res, (T *)out, K, N);
    count_launch();
    return e;
}

template <int BN, int KS>
cudaError_t launch_lin_tc(const CUtensorMap &ma, const CUtensorMap &mw, const CUtensorMap &mr, const CUtensorMap &mo, const LinParams &p, int n_tiles,
                          cudaStream_t st)
{
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        return cudaFuncSetAttribute(linear_res_tc_kernel<BN, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LinSmem<BN>::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2u * KS * (unsigned)p.m_tiles * (unsigned)n_tiles);
    cfg.blockDim = dim3(kLinThreads);
    cfg.dynamicSmemBytes = LinSmem<BN>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // a pair of CTAs, or the two pairs that split a tile's contraction
    attr[1].val.clusterDim.x = 2u * KS; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, linear_res_tc_kernel<BN, KS>, ma, mw, mr, mo, p);
    count_launch();
    return e;
}

}  // namespace

bool linear_tc_supported(int dtype, int M, int K, int N)
{
    return dtype == REFLEX_DTYPE_BF16 && M >= 1 && K >= 8 && K % 8 == 0 && N >= 8 && N % 8 == 0 && (long long)M * N <= 0x3FFFFFFF;
}

// impl: 0 = tensor cores where supported, 1 = plain kernel, 2 = tensor cores, the 256-row tiles whatever M is
cudaError_t launch_linear_residual(const void *a, const void *W, const void *res, void *out, int M, int K, int N, int dtype, int impl,
                                   uint32_t *status, cudaStream_t st)
{
    const bool tc = impl != 1 && linear_tc_supported(dtype, M, K, N);
    if (!tc) {
        if ((size_t)K * sizeof(float) > 48 * 1024) return cudaErrorInvalidValue;
        return dtype == REFLEX_DTYPE_BF16 ? launch_lin_simt<__nv_bfloat16>(a, W, res, out, M, K, N, st) : launch_lin_simt<float>(a, W, res, out, M, K, N, st);
    }
    if (impl == 0 && linear_small_takes(M, K, N)) return launch_linear_small(a, W, res, out, M, K, N, status, st);
    LinParams p;
    p.M = M; p.K = K; p.N = N; p.m_tiles = (M + 2 * kLinBM - 1) / (2 * kLinBM); p.has_res = res ? 1 : 0; p.status = status;
    // 256-column tiles unless they would leave more than half of the SM pairs without one: then 128-column tiles, twice as
    // many pairs at work on a contraction that is as long (every CTA then fetches 24 KB per step for half the MMA work)
    const bool narrow = p.m_tiles * ((N + 255) / 256) * 2 <= 74;
    CUtensorMap ma, mw, mr, mo;
    if (!tensor_map_2d_bf16(&ma, a, K, M, kLinBM) || !tensor_map_2d_bf16(&mw, W, K, N, narrow ? 64 : 128) || !tensor_map_2d_bf16(&mo, out, N, M, kLinBM))
        return cudaErrorInvalidValue;
    if (res) { if (!tensor_map_2d_bf16(&mr, res, N, M, kLinBM)) return cudaErrorInvalidValue; }
    else mr = mo;
    if (narrow) {
        // ... and the contraction in two halves on two pairs of a 4-CTA cluster while that still leaves every pair an SM pair of
        // its own and the halves are long enough to pay for the exchange, which costs about 4 us (two cluster barriers, 32 KB
        // per CTA through distributed shared memory, the slower pair's lag): 300-1000 rows x 4096 -> 1024 15.5-17.0 -> 12.9-15.0 us;
        // x 2048 9.3-9.4 -> 9.8-11.0, so only contractions of 4096 and more are split
        const int n_tiles = (N + 127) / 128, nk_all = (K + kLinBK - 1) / kLinBK;
        if (p.m_tiles * n_tiles * 2 <= 74 && nk_all % 2 == 0 && nk_all >= 64) return launch_lin_tc<128, 2>(ma, mw, mr, mo, p, n_tiles, st);
        return launch_lin_tc<128, 1>(ma, mw, mr, mo, p, n_tiles, st);
    }
    return launch_lin_tc<256, 1>(ma, mw, mr, mo, p, (N + 255) / 256, st);
}

}  // namespace reflex

#ifdef REFLEX_LIN_TRACE
extern "C" int reflex_debug_lin_trace(unsigned long long *out)
{
    return (int)cudaMemcpyFromSymbol(out, reflex::g_lin_trace, sizeof(unsigned long long) * 512 * 8);
}
#endif
