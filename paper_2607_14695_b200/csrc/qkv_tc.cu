// Adaptive norm folded into the packed Q/K/V projection (Sec. 3.3 "System Optimizations": W_QKV = [W_Q; W_K; W_V] as one
// GEMM; Sec. 4 "Operator Fusion Impact": the adaptive norm combined with the linear layer after it, so that the norm output
// never reaches memory):
//     [q | k_dyn | v_dyn][r][n] = (1 / RMS(x_r)) * sum_i (x[r][i] * gamma_b[i]) * W_QKV[n][i]          (Eq. 2 + projection)
//
// bf16 path: a pair of CTAs (cta_group::2) owns 256 rows and NACC x 256 output columns (NACC fp32 accumulators of 256
// columns in tensor memory) and walks the contraction axis in 64-column steps through a ring of shared-memory stages.
// Per step and CTA, TMA brings 128 rows of x and NACC x 128 rows of W_QKV. Eight warps (two threads per row) multiply
// the x tile by the stream's gate in place (bf16(x * gamma), the A operand; the gates of the CTA's streams are staged
// in shared memory once), accumulating the row's sum of squares on the way; one elected thread of the leader CTA
// issues the tcgen05 MMAs. The row scale 1/RMS does not depend on the contraction index, so it multiplies the
// accumulator in the epilogue: the threads that summed a row's squares read that row out of tensor memory, scale and
// round to bf16; the tile is staged in shared memory and written as whole 512-byte rows to the Q, K or V tensor.
// NACC = 2 where 256-column tiles would not fit the SM pairs in one wave: the gate multiply (ALU work that every column
// tile of the same rows repeats) is then spread over twice the MMA work, and 3200 x 2560 becomes 65 tiles on 74 pairs.
// Measured on the way (3200 x 2560 x 1024, NACC = 1, 130 tiles in two waves): in-place rewrite with the gate read from
// global memory 29.5 us (an L2 round trip of gate values per step on the critical path); x loaded from global memory by
// the row-owning threads 40 us (32 cache lines per load instruction); A operand stored to tensor memory instead of back
// to shared memory 23.2 us (the gate multiply, about 700 cycles per step, stayed above the 512 cycles of the MMAs).
//
// The same kernel serves the fused gate / up projections of a SwiGLU block (Sec. 3.3: "combine the Gate and Up projections"):
// accumulator 0 takes 256 rows of W_gate, accumulator 1 the same rows of W_up, and the epilogue writes
// SiLU(gate) * up for those 256 hidden columns (swiglu_F > 0 in the parameters). With more tiles than SM pairs (3200 rows x
// 4096 hidden columns: 208) the grid is one CTA pair per SM pair and every pair walks its tiles (WALK): 48.8 -> 44.7 us,
// the loads of a tile's first steps and the set-up of a wave no longer waiting behind the last tile's epilogue.
//
// Any other dtype or shape: a plain kernel (one block per row, fp32 FMAs) with the same semantics.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

using namespace ptx;

namespace {

constexpr int kQkThreads = 64 + 256;   // producer warp, MMA warp, eight transform / epilogue warps (two threads per row)
constexpr int kQkBM = 128;             // rows of x per CTA (256 per pair)
constexpr int kQkBN = 256;             // output columns per accumulator (each CTA loads 128 rows of W_QKV for it)
constexpr int kQkBK = 64;              // contraction step: one 128-byte swizzled row
constexpr int kQkStages = 4;
constexpr unsigned long long kQkWaitNs = 1000000000ull;

template <int NACC>
struct QkSmem {
    static constexpr uint32_t X_STAGE = kQkBM * 128;
    static constexpr uint32_t B_HALF = (kQkBN / 2) * 128;     // 128 rows of W_QKV: this CTA's half of one accumulator's B operand
    static constexpr uint32_t B_STAGE = NACC * B_HALF;
    static constexpr uint32_t OFF_X = 0;
    static constexpr uint32_t OFF_B = kQkStages * X_STAGE;
    static constexpr uint32_t OFF_BAR = OFF_B + kQkStages * B_STAGE;
    static constexpr uint32_t OFF_SS = OFF_BAR + 512;         // [2][128] partial sums of squares
    static constexpr uint32_t OFF_GATE = OFF_SS + 1024;       // gates of the streams this CTA's rows belong to, [n][D] fp32
    static constexpr uint32_t GATE_MAX = (NACC == 1 ? 64u : 28u) * 1024u;
    static constexpr uint32_t TOTAL = OFF_GATE + GATE_MAX + 1024;   // + slack for the 1024-byte alignment
    static_assert(TOTAL <= 227u * 1024u, "shared memory budget");
};
enum { Q_XFULL = 0, Q_BFULL = kQkStages, Q_AREADY = 2 * kQkStages, Q_EMPTY = 3 * kQkStages, Q_ACC = 4 * kQkStages, Q_ACCFREE, Q_STAGEFREE, Q_COUNT };

struct QkParams {
    const float *gate;          // [B][D]
    __nv_bfloat16 *q, *k, *v;   // [M][nq], [M][nk], [M][nk]
    int M, R, B, D, nq, nk;     // M = B * R rows; nq = Hq * d, nk = Hkv * d
    int m_tiles;                // 256-row tiles
    int n_tiles;                // column tiles (256-row kernel: a CTA pair walks tiles pair, pair + pairs, ... of m_tiles x n_tiles)
    int swiglu_F;               // 0: columns go to Q, K, V. F > 0: W holds [W_gate; W_up] ([2F][D]), out (= q, pitch nq = F) gets SiLU(g) * u
    float eps;
    uint32_t *status;
    const __nv_bfloat16 *res;   // plain projection only (few-rows kernel with PLAIN): residual [M][nq] added to the output, or NULL
    int ksplit;                 // few-rows kernel: CTAs of a cluster that share one feature tile, each taking a slice of the contraction
    int tma_out;                // 256-row kernel: the output tile leaves through TMA stores (tensor maps over q / k / v given)
};

#ifdef REFLEX_QK_TRACE
__device__ long long g_qk_trace[3 * 32 * 8];
#define QK_TRACE(role, step, ev) do { if (blockIdx.x == 0 && (step) < 32) g_qk_trace[((role) * 32 + (step)) * 8 + (ev)] = clock64(); } while (0)
#else
#define QK_TRACE(role, step, ev) do { } while (0)
#endif

// SiLU(g) * u with one special-function operation per element: g / (1 + e^-g) = g (1 + tanh(g / 2)) / 2. The epilogue of the
// gate/up kernel is bound by the special-function unit (16 results per clock and SM; 32 K elements per tile): with an
// exponential and a reciprocal per element it took 7.7 k cycles of a 26 k-cycle tile. tanh.approx is accurate to about 2^-11,
// a quarter of the spacing of the bf16 the result is rounded to.
__device__ __forceinline__ float silu_mul(float g, float u)
{
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
    return fmaf(t, 0.5f * g, 0.5f * g) * u;
}

__device__ __forceinline__ void qk_tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ void tma2_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1)
                 : "memory");
}

template <int NACC, bool WALK>      // WALK: more tiles than CTA pairs (otherwise one tile per pair, and the tile loops fold away)
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kQkThreads, 1)
norm_qkv_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_q,
                   const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, QkParams p)
{
    using S = QkSmem<NACC>;
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
    const bool swiglu = NACC == 2 && p.swiglu_F > 0;
    const int nk_steps = p.D / kQkBK;
    // A pair takes tiles pair, pair + pairs, ... (row tiles fastest, so that the pairs working at the same time share weight
    // rows in L2). With more tiles than pairs the grid is one pair per SM pair and the roles below run ahead of each other
    // across tile boundaries: the producer refills the weight stages and the tensor pipe starts the next tile's first
    // steps while the eight warps still convert and store the last tile. The stage ring, its barrier phases and the
    // accumulator hand-over all count steps and tiles from the start of the kernel.
    const int n_pairs = (int)(gridDim.x >> 1);
    const int total_tiles = p.m_tiles * p.n_tiles;
    const int my_tiles = !WALK ? 1 : pair < total_tiles ? (total_tiles - pair + n_pairs - 1) / n_pairs : 0;
    auto tile_m0 = [&](int it) -> int { return ((pair + it * n_pairs) % p.m_tiles) * (2 * kQkBM) + (int)rank * kQkBM; };    // this CTA's first row
    auto tile_n0 = [&](int it) -> int { return ((pair + it * n_pairs) / p.m_tiles) * (swiglu ? kQkBN : NACC * kQkBN); };   // the pair's first output column

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQkStages; ++s) {
            mbar_init(bar(Q_XFULL + s), 1);
            mbar_init(bar(Q_BFULL + s), 1);
            mbar_init(bar(Q_AREADY + s), 16);   // one arrival per transform warp of either CTA
            mbar_init(bar(Q_EMPTY + s), 1);
        }
        mbar_init(bar(Q_ACC), 1);
        mbar_init(bar(Q_ACCFREE), 16);      // one arrival per epilogue warp of either CTA: the accumulators have been read
        mbar_init(bar(Q_STAGEFREE), 2);     // the two threads that hand this CTA's staged chunks to the TMA engine: all of them read
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_w);
    }
    if (warp == 1) tmem_alloc2(smem_u32((const void *)tmem_slot), NACC * kQkBN);
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
            // the epilogue stages accumulator 0 in the x stages and (packed projection, two accumulators) accumulator 1 in the
            // weight stages: loads into either wait until the last tile's stores have read them
            const bool w_staged = !swiglu && NACC == 2;
            for (int it = 0; it < my_tiles && ok; ++it) {
                const int m0 = tile_m0(it), n0 = tile_n0(it);
                const int g0 = it * nk_steps;
                auto stage_free = [&](int ks) -> bool {     // the MMAs that read the stage of step ks four steps ago are complete
                    const int g = g0 + ks;
                    return g < kQkStages || wait(Q_EMPTY + g % kQkStages, (uint32_t)(g / kQkStages - 1) & 1u, 1);
                };
                auto load_x = [&](int ks) {
                    const int s = (g0 + ks) % kQkStages;
                    mbar_expect_tx(bar(Q_XFULL + s), S::X_STAGE);
                    tma_load_2d(base + S::OFF_X + s * S::X_STAGE, &tm_x, bar(Q_XFULL + s), ks * kQkBK, m0);
                };
                auto load_w = [&](int ks) {
                    const int s = (g0 + ks) % kQkStages;
                    if (rank == 0) mbar_expect_tx(bar(Q_BFULL + s), 2 * S::B_STAGE);
#pragma unroll
                    for (int j = 0; j < NACC; ++j)
                        tma2_load_2d(base + S::OFF_B + s * S::B_STAGE + j * S::B_HALF, &tm_w, bar(Q_BFULL + s) & kPeerBitMask, ks * kQkBK,
                                     (swiglu ? j * p.swiglu_F + n0 : n0 + j * kQkBN) + (int)rank * (kQkBN / 2));
                };
                int ks = 0;
                if (it > 0) {
                    // head of a later tile: the weights of its first steps go out while the last tile's epilogue still owns the
                    // x stages, the x tiles follow once its stores have read them
                    const int nh = nk_steps < kQkStages ? nk_steps : kQkStages;
                    const uint32_t ph = (uint32_t)(it - 1) & 1u;
                    if (w_staged) ok = wait(Q_STAGEFREE, ph, 7);
                    for (int h = 0; h < nh && ok; ++h) {
                        ok = stage_free(h);
                        if (ok) load_w(h);
                    }
                    if (ok && !w_staged) ok = wait(Q_STAGEFREE, ph, 7);
                    for (int h = 0; h < nh && ok; ++h) load_x(h);
                    ks = nh;
                }
                for (; ks < nk_steps && ok; ++ks) {
                    ok = stage_free(ks);
                    if (!ok) break;
                    QK_TRACE(0, ks, 0);
                    load_x(ks);
                    load_w(ks);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA; the warp stays converged, one elected lane issues) ----------------
        if (rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * kQkBM, kQkBN, false);
            bool ok = true;
            for (int it = 0; it < my_tiles && ok; ++it) {
                // the epilogue warps of both CTAs have read the last tile's accumulators
                if (it > 0) ok = wait(Q_ACCFREE, (uint32_t)(it - 1) & 1u, 6);
                for (int ks = 0; ks < nk_steps && ok; ++ks) {
                    const int g = it * nk_steps + ks;
                    const int s = g % kQkStages;
                    const uint32_t ph = (uint32_t)(g / kQkStages) & 1u;
                    if (lane == 0) QK_TRACE(1, ks, 0);
                    ok = wait(Q_BFULL + s, ph, 2);
                    if (lane == 0) QK_TRACE(1, ks, 1);
                    ok = ok && wait(Q_AREADY + s, ph, 3);
                    if (lane == 0) QK_TRACE(1, ks, 2);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int j = 0; j < NACC; ++j) {
                        uint64_t ad = umma_desc_sw128(base + S::OFF_X + s * S::X_STAGE, 16, 1024);
                        uint64_t bd = umma_desc_sw128(base + S::OFF_B + s * S::B_STAGE + j * S::B_HALF, 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < kQkBK / 16; ++kk) {
                            umma2_ss_elect(tmem + j * kQkBN, ad, bd, idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                            umma_desc_advance(ad, 32);
                            umma_desc_advance(bd, 32);
                        }
                    }
                    umma2_commit_mc_elect(bar(Q_EMPTY + s), (uint16_t)3);
                    if (lane == 0) QK_TRACE(1, ks, 3);
                }
                umma2_commit_mc_elect(bar(Q_ACC), (uint16_t)3);   // also after a wait that ran out: the epilogue warps must not wait for nothing
            }
        }
    } else {
        // ---------------- gate multiply (A operand) and epilogue: two threads per row ----------------
        // Thread (row, half) owns columns [32 half, 32 half + 32) of the row's 64 in every step, and columns
        // [128 half, 128 half + 128) of the row's accumulator in the epilogue. Two warps per scheduler hide each other's
        // load latencies; the arithmetic is packed (two fp32 per instruction).
        const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        float *gsm = reinterpret_cast<float *>(smem + S::OFF_GATE);
        float *ssm = reinterpret_cast<float *>(smem + S::OFF_SS);
        const uint32_t leader_aready0 = mapa(bar(Q_AREADY), 0);
        const uint32_t leader_accfree = mapa(bar(Q_ACCFREE), 0);
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int n_out = p.nq + 2 * p.nk;
        bool ok = true;
#pragma unroll 1
        for (int it = 0; it < my_tiles; ++it) {
        const int m0 = tile_m0(it), n0 = tile_n0(it);
        const int g0 = it * nk_steps;
        const int r_glob = m0 + row;
        const int b = min(r_glob / p.R, p.B - 1);     // (rows past the end contribute zeros and are never stored)
        // the gates of the streams under this CTA's 128 rows go to shared memory once per tile: every step needs 128 fresh bytes
        // of them per thread, and as global loads those were an L2 round trip per step on the critical path. (Every warp is
        // through with the last tile's gates: they are read in the step loop only, and all eight warps have met since.)
        const int b_first = min(m0 / p.R, p.B - 1), b_last = min((m0 + kQkBM - 1) / p.R, p.B - 1);
        {
            const int n4 = (b_last - b_first + 1) * p.D / 4;
            const float4 *src = reinterpret_cast<const float4 *>(p.gate + (size_t)b_first * p.D);
            for (int i = threadIdx.x - 64; i < n4; i += 256) reinterpret_cast<float4 *>(gsm)[i] = __ldg(src + i);
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        const float *grow = gsm + (size_t)(b - b_first) * p.D + half * 32;
        uint64_t ss2 = 0ull;
        for (int ks = 0; ks < nk_steps; ++ks) {
            if (threadIdx.x == 64) QK_TRACE(2, ks, 0);
            const int s = (g0 + ks) % kQkStages;
            const ulonglong2 *g2 = reinterpret_cast<const ulonglong2 *>(grow + ks * kQkBK);
            ulonglong2 gq[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) gq[i] = g2[i];      // 32 gate values, read before the wait for the tile
            ok = ok && wait(Q_XFULL + s, (uint32_t)((g0 + ks) / kQkStages) & 1u, 4);
            if (threadIdx.x == 64) QK_TRACE(2, ks, 1);
            uint8_t *rowp = smem + S::OFF_X + s * S::X_STAGE + row * 128;
            uint4 xr[4];
#pragma unroll
            for (int c = 0; c < 4; ++c)   // 128-byte swizzle: chunk j of row r sits at j ^ (r % 8)
                xr[c] = *reinterpret_cast<const uint4 *>(rowp + (((4 * half + c) ^ (row & 7)) << 4));
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint64_t gg[4] = {gq[2 * c].x, gq[2 * c].y, gq[2 * c + 1].x, gq[2 * c + 1].y};
                uint32_t vv[4] = {xr[c].x, xr[c].y, xr[c].z, xr[c].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint64_t x2 = pack_f32x2(__uint_as_float(vv[k] << 16), __uint_as_float(vv[k] & 0xFFFF0000u));
                    ss2 = fma_f32x2(x2, x2, ss2);
                    float y0, y1;
                    unpack_f32x2(mul_f32x2(x2, gg[k]), y0, y1);
                    __nv_bfloat162 y2 = __floats2bfloat162_rn(y0, y1);
                    vv[k] = *reinterpret_cast<uint32_t *>(&y2);
                }
                *reinterpret_cast<uint4 *>(rowp + (((4 * half + c) ^ (row & 7)) << 4)) = make_uint4(vv[0], vv[1], vv[2], vv[3]);
            }
            if (threadIdx.x == 64) QK_TRACE(2, ks, 2);
            fence_proxy_async_smem();   // the tensor pipe reads what these threads wrote
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_aready0 + 8u * (uint32_t)s);
            if (threadIdx.x == 64) QK_TRACE(2, ks, 4);
        }
        // the row's sum of squares: both halves meet through shared memory
        {
            float s0, s1;
            unpack_f32x2(ss2, s0, s1);
            ssm[half * 128 + row] = s0 + s1;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        const float ss = ssm[row] + ssm[128 + row];
        if (threadIdx.x == 64) QK_TRACE(2, 31, 0);
        ok = wait(Q_ACC, (uint32_t)it & 1u, 5) && ok;
        if (threadIdx.x == 64) QK_TRACE(2, 31, 1);
        tc_fence_after();
        const float rs = rsqrtf(ss / (float)p.D + p.eps);
        if (p.tma_out) {
            // The tile goes out through shared memory and TMA stores. The stage ring is idle now (every load has been consumed and
            // every MMA has completed): accumulator j is staged in the x stages (j = 0) or the weight stages (j = 1) as four
            // chunks of 128 rows x 64 columns in the layout of a 128-byte-swizzled TMA box, each thread dropping its half row,
            // scaled and rounded, as 16-byte pieces; a chunk is handed to the TMA engine as soon as the 128 threads that fill it
            // are through, and the stores drain while the next chunk is converted. (With every warp copying whole rows from
            // the staging area to global memory the epilogue took 6.4 k cycles of a 25 k-cycle tile.)
            static_assert(S::OFF_B - S::OFF_X >= 4u * 128u * 128u && S::OFF_BAR - S::OFF_B >= 4u * 128u * 128u, "staging areas of the epilogue");
#pragma unroll 1
            for (int j = 0; j < (swiglu ? 1 : NACC); ++j) {
                const uint32_t stage_off = j == 0 ? S::OFF_X : S::OFF_B;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    const int ch = half * 2 + cc;                 // 64-column chunk of the accumulator
                    uint8_t *rowp = smem + stage_off + ch * (128 * 128) + row * 128;
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        uint32_t acc[32];
                        tmem_ld32(tmem + lane_addr + j * kQkBN + ch * 64 + g * 32, acc);   // warp-wide: every lane takes part, whatever its row
                        if (swiglu) {     // (uniform) the up projection of the same columns; acc <- SiLU(g) * u, both scaled by 1/RMS first
                            uint32_t up[32];
                            tmem_ld32(tmem + lane_addr + kQkBN + ch * 64 + g * 32, up);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(silu_mul(__uint_as_float(acc[i]) * rs, __uint_as_float(up[i]) * rs));
                        } else {
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * rs);
                        }
                        if (WALK && cc == 1 && g == 1 && j == (swiglu ? 0 : NACC - 1)) {
                            // this warp's last read of the accumulators: the tensor pipe may start the next tile over them
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(leader_accfree);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 o;
                            uint32_t *oo = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[8 * i + 2 * k]), __uint_as_float(acc[8 * i + 2 * k + 1]));
                                oo[k] = *reinterpret_cast<uint32_t *>(&h);
                            }
                            // 128-byte swizzle of the TMA box: 16-byte piece p of row r sits at p ^ (r % 8)
                            *reinterpret_cast<uint4 *>(rowp + (((g * 4 + i) ^ (row & 7)) << 4)) = o;
                        }
                    }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync %0, 128;" ::"r"(2 + half) : "memory");   // the chunk's 128 threads
                    if (quarter == 0 && lane == 0 && ok && m0 < p.M) {
                        const int n = n0 + j * kQkBN + ch * 64;     // first output column of the chunk (chunks never straddle Q, K and V:
                                                                    // the launcher takes this path only when their widths are multiples of 64)
                        const uint32_t src = base + stage_off + ch * (128 * 128);
                        if (swiglu) { if (n < p.swiglu_F) qk_tma_store_2d(&tm_q, src, n, m0); }
                        else if (n < p.nq) qk_tma_store_2d(&tm_q, src, n, m0);
                        else if (n < p.nq + p.nk) qk_tma_store_2d(&tm_k, src, n - p.nq, m0);
                        else if (n < n_out) qk_tma_store_2d(&tm_v, src, n - p.nq - p.nk, m0);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
            // (the staging areas have been read -- the producer may load the next tile over them; the writes themselves are
            // complete when the grid is)
            if (quarter == 0 && lane == 0) {
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                if (WALK) mbar_arrive(bar(Q_STAGEFREE));
            }
        } else {
        // The tile goes out through shared memory (the stage ring is idle now: every load has been consumed and every MMA
        // has completed): each thread drops its half row, scaled and rounded, as 16-byte pieces at [row][piece ^ (row % 32)]
        // (conflict-free for 32 rows at a time), then every warp writes whole 512-byte rows, 16 bytes per lane. (Straight
        // from registers every store instruction touched 32 rows 4 KB apart: 6.3 k cycles per tile.)
        uint4 *stg = reinterpret_cast<uint4 *>(smem + S::OFF_X);      // [128 rows][32 pieces of 8 columns]
        static_assert(kQkBM * kQkBN * 2 <= (int)(S::OFF_BAR - S::OFF_X), "staging area of the epilogue");
#pragma unroll 1
        for (int j = 0; j < (swiglu ? 1 : NACC); ++j) {
#pragma unroll 1
            for (int c = 0; c < kQkBN / 64; ++c) {
                uint32_t acc[32];
                tmem_ld32(tmem + lane_addr + j * kQkBN + half * (kQkBN / 2) + c * 32, acc);   // warp-wide: every lane takes part, whatever its row
                if (swiglu) {     // (uniform) the up projection of the same columns; acc <- SiLU(g) * u, both scaled by 1/RMS first
                    uint32_t up[32];
                    tmem_ld32(tmem + lane_addr + kQkBN + half * (kQkBN / 2) + c * 32, up);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float g = __uint_as_float(acc[i]) * rs, u = __uint_as_float(up[i]) * rs;
                        acc[i] = __float_as_uint(silu_mul(g, u));
                    }
                } else {
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] = __float_as_uint(__uint_as_float(acc[i]) * rs);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 o;
                    uint32_t *oo = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[8 * i + 2 * k]), __uint_as_float(acc[8 * i + 2 * k + 1]));
                        oo[k] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    const int piece = half * 16 + c * 4 + i;
                    stg[row * 32 + (piece ^ (row & 31))] = o;
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            {
                const int n = n0 + j * kQkBN + lane * 8;   // this lane's 8 columns: they never straddle Q, K and V (head_dim % 8 == 0)
                __nv_bfloat16 *dst0 = nullptr;              // column n of row 0 of the tensor it belongs to
                size_t pitch = 0;
                if (n < p.nq) { dst0 = p.q + n; pitch = (size_t)p.nq; }
                else if (n < p.nq + p.nk) { dst0 = p.k + (n - p.nq); pitch = (size_t)p.nk; }
                else if (n < n_out) { dst0 = p.v + (n - p.nq - p.nk); pitch = (size_t)p.nk; }
                const int w8 = warp - 2;                    // 0..7: rows w8, w8 + 8, ...
                if (ok && dst0) {
#pragma unroll 4
                    for (int r = w8; r < kQkBM; r += 8) {
                        if (m0 + r >= p.M) break;
                        *reinterpret_cast<uint4 *>(dst0 + (size_t)(m0 + r) * pitch) = stg[r * 32 + (lane ^ (r & 31))];
                    }
                }
            }
            if (j + 1 < (swiglu ? 1 : NACC)) asm volatile("bar.sync 1, 256;" ::: "memory");   // the staging area is rewritten by the next round
        }
        }
        }   // tiles of this pair
    }

    if (threadIdx.x == 64) QK_TRACE(2, 31, 2);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // neither CTA retires while its partner can still touch its shared memory or barriers
    if (warp == 1) tmem_dealloc2(tmem, NACC * kQkBN);
}

// ---- few rows (a handful of streams): weights as the A operand ------------------------------------------------------------
// With a few hundred rows at most, tiles of 256 rows would be mostly padding and the launch a chain of sixteen dependent steps
// on a handful of CTAs. Here the roles are swapped: out^T [features][rows] = W [features][D] . y'^T [D][rows]. A CTA owns 128
// output features (the M of a cta_group::1 MMA; for SwiGLU 128 hidden features with a gate and an up accumulator) and a
// group of rows, which are the N (64 or 128): the grid is features / 128 x row groups CTAs that each stream their slice of
// the weights once (the whole cost of the call) while eight warps rewrite the small x tile of every step as the gated B
// operand. Groups of 64 rows are taken while every (feature tile, group) still has an SM of its own (grid y).
constexpr int kSmThreads = 64 + 256;   // producer warp, MMA warp, eight warps that rewrite x and run the epilogue

template <int NT, int NACC>      // NT: rows (tokens) padded to 64 or 128; NACC: 1, or 2 for SwiGLU (gate and up rows)
struct SmSmem {
    static constexpr int CPS = NACC == 2 ? 1 : 2;                 // 64-column chunks of the contraction axis per step: fewer, longer
                                                                  // steps where the stages allow (every step costs ~560 cycles of hand-overs)
    static constexpr int STAGES = NACC == 2 ? 4 : (NT == 64 ? 4 : 3);
    static constexpr uint32_t W_TILE = 128 * 128;                 // 128 feature rows x 64 k
    static constexpr uint32_t W_STAGE = NACC * CPS * W_TILE;
    static constexpr uint32_t X_TILE = NT * 128;                  // NT rows x 64 k
    static constexpr uint32_t X_STAGE = CPS * X_TILE;
    static constexpr uint32_t OFF_W = 0;
    static constexpr uint32_t OFF_X = STAGES * W_STAGE;
    static constexpr uint32_t OFF_BAR = OFF_X + STAGES * X_STAGE;
    static constexpr uint32_t OFF_SS = OFF_BAR + 512;             // [4][128] partial sums of squares per row, then [128] 1/RMS
    static constexpr uint32_t OFF_GATE = OFF_SS + 2560;
    static constexpr uint32_t GATE_MAX = 16 * 1024;               // gates of the (at most 4) streams the rows belong to
    static constexpr uint32_t TOTAL = OFF_GATE + GATE_MAX + 1024;
    static_assert(TOTAL <= 227u * 1024u, "shared memory budget");
    // mbarrier indices
    static constexpr int S_XFULL = 0, S_BREADY = STAGES, S_EMPTY = 2 * STAGES, S_ACC = 3 * STAGES, S_COUNT = S_ACC + 1;
};

// PLAIN: no norm at all (out = res + x W^T, the expert's output / down projections for one or two streams): the eight warps
// only pass each landed step on to the MMA warp, and the epilogue adds the residual instead of scaling by 1/RMS.
template <int NT, int NACC, bool PLAIN = false>
__global__ void __launch_bounds__(kSmThreads, 1)
norm_linear_small_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, QkParams p)
{
    using S = SmSmem<NT, NACC>;
    constexpr int kSmStages = S::STAGES;
    constexpr int S_XFULL = S::S_XFULL, S_BREADY = S::S_BREADY, S_EMPTY = S::S_EMPTY, S_ACC = S::S_ACC, S_COUNT = S::S_COUNT;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    auto bar = [&](int i) -> uint32_t { return base + S::OFF_BAR + 8u * (uint32_t)i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + S::OFF_BAR + 8 * S_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool swiglu = NACC == 2;
    // ksplit > 1: the ksplit CTAs of a cluster own the same 128 features and a slice of the contraction axis each (whole
    // steps only: the launcher picks ksplit so that the chunks divide), and add up their accumulators -- and, with the
    // norm, their shares of every row's sum of squares -- through distributed shared memory at the end. With a handful of
    // CTAs streaming the weights the launch is a chain of dependent steps; split, 80 to 128 CTAs share it.
    const int ksplit = p.ksplit;
    const int krank = ksplit > 1 ? (int)cluster_ctarank() : 0;
    const int f0 = (blockIdx.x / ksplit) * 128;       // first output feature (hidden feature for SwiGLU) of this CTA
    const int row0 = blockIdx.y * NT;                 // first row of this CTA's group of NT rows (grid y: row groups)
    constexpr int CPS = S::CPS;
    const int all_chunks = p.D / kQkBK;
    const int chunk0 = krank * (all_chunks / ksplit);      // this CTA's first 64-column chunk of the contraction axis
    const int n_chunks = ksplit > 1 ? all_chunks / ksplit : all_chunks;
    const int nk_steps = (n_chunks + CPS - 1) / CPS;       // (a last step may hold one chunk only: TMA zero-fills the other)
    constexpr int TP = 256 / NT;                      // transform threads per row: 4 (64 rows) or 2 (128 rows)
    constexpr uint32_t kCols = NACC * NT < 32 ? 32 : NACC * NT;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSmStages; ++s) {
            mbar_init(bar(S_XFULL + s), 1);
            mbar_init(bar(S_BREADY + s), 8);          // one arrival per transform warp
            mbar_init(bar(S_EMPTY + s), 1);
        }
        mbar_init(bar(S_ACC), 1);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_w);
    }
    if (warp == 1) tmem_alloc(smem_u32((const void *)tmem_slot), kCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (threadIdx.x == 64) QK_TRACE(2, 30, 0);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 64) QK_TRACE(2, 30, 1);
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
        if (p.status) atomicCAS(p.status, 0u, 0x80000000u | ((code + 112u) << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            bool ok = true;
            for (int ks = 0; ks < nk_steps && ok; ++ks) {
                const int s = ks % kSmStages;
                if (ks >= kSmStages) ok = wait(S_EMPTY + s, (uint32_t)(ks / kSmStages - 1) & 1u, 1);
                if (!ok) break;
                // one barrier for both operands of the step: the threads that rewrite x wait for it, so their hand-over to the
                // MMA warp also says that the weights are in place (one wait less per step in the issuing loop)
                mbar_expect_tx(bar(S_XFULL + s), S::X_STAGE + S::W_STAGE);
#pragma unroll
                for (int cc = 0; cc < CPS; ++cc) {
                    const int col = (chunk0 + ks * CPS + cc) * kQkBK;
                    tma_load_2d(base + S::OFF_X + s * S::X_STAGE + cc * S::X_TILE, &tm_x, bar(S_XFULL + s), col, row0);
#pragma unroll
                    for (int j = 0; j < NACC; ++j)
                        tma_load_2d(base + S::OFF_W + s * S::W_STAGE + (j * CPS + cc) * S::W_TILE, &tm_w, bar(S_XFULL + s), col, j * p.swiglu_F + f0);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (the warp stays converged, one elected lane issues) ----------------
        constexpr uint32_t idesc = umma_idesc_bf16(128, NT, false);
        bool ok = true;
        for (int ks = 0; ks < nk_steps && ok; ++ks) {
            const int s = ks % kSmStages;
            const uint32_t ph = (uint32_t)(ks / kSmStages) & 1u;
            if (lane == 0) QK_TRACE(1, ks, 0);
            ok = wait(S_BREADY + s, ph, 3);
            if (lane == 0) QK_TRACE(1, ks, 2);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < NACC; ++j) {
#pragma unroll
                for (int cc = 0; cc < CPS; ++cc) {
                    uint64_t ad = umma_desc_sw128(base + S::OFF_W + s * S::W_STAGE + (j * CPS + cc) * S::W_TILE, 16, 1024);
                    uint64_t bd = umma_desc_sw128(base + S::OFF_X + s * S::X_STAGE + cc * S::X_TILE, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < kQkBK / 16; ++kk) {
                        umma_ss_elect(tmem + j * NT, ad, bd, idesc, (ks > 0 || cc > 0 || kk > 0) ? 1u : 0u);
                        umma_desc_advance(ad, 32);
                        umma_desc_advance(bd, 32);
                    }
                }
            }
            umma_commit_elect(bar(S_EMPTY + s));
        }
        umma_commit_elect(bar(S_ACC));    // also after a wait that ran out: the epilogue warps must not wait for nothing
    } else {
        // ---------------- gate multiply (B operand) and epilogue ----------------
        const int tid = threadIdx.x - 64;              // 0..255
        const int row = tid % NT;                      // row (token) this thread rewrites
        const int kpart = tid / NT;                    // which 64 / TP columns of every step
        constexpr int KW = kQkBK / TP;                 // columns per thread and step: 16 or 32
        const int b = min((row0 + row) / p.R, p.B - 1);
        const int b_first = min(row0 / p.R, p.B - 1), b_last = min((row0 + NT - 1) / p.R, p.B - 1);   // streams under this group's rows
        float *gsm = reinterpret_cast<float *>(smem + S::OFF_GATE);
        if constexpr (!PLAIN) {
            const int n4 = (b_last - b_first + 1) * p.D / 4;     // (they fit: checked by the launcher)
            const float4 *src = reinterpret_cast<const float4 *>(p.gate + (size_t)b_first * p.D);
            for (int i = tid; i < n4; i += 256) reinterpret_cast<float4 *>(gsm)[i] = __ldg(src + i);
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        if (threadIdx.x == 64) QK_TRACE(2, 30, 2);
        const float *grow = gsm + (size_t)(b - b_first) * p.D + kpart * KW;
        uint64_t ss2 = 0ull;
        bool ok = true;
        for (int ks = 0; ks < nk_steps; ++ks) {
            const int s = ks % kSmStages;
            if (threadIdx.x == 64) QK_TRACE(2, ks, 0);
            ok = ok && wait(S_XFULL + s, (uint32_t)(ks / kSmStages) & 1u, 4);
            if (threadIdx.x == 64) QK_TRACE(2, ks, 1);
            if constexpr (PLAIN) {
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(S_BREADY + s));
                continue;
            }
            // all loads of the step first (x pieces and gate values of every chunk), then the arithmetic and the stores: the
            // stores could alias the later loads for all the compiler knows, and with a few independent loads per thread the
            // shared-memory latency was most of a step
            constexpr int NPC = KW / 8;                 // 16-byte pieces per thread and chunk
            uint4 xv[CPS * NPC];
            ulonglong2 gv[CPS * NPC * 2];
#pragma unroll
            for (int cc = 0; cc < CPS; ++cc) {
                const int chunk = chunk0 + min(ks * CPS + cc, n_chunks - 1);      // (a chunk past the end: loaded but never used)
                const ulonglong2 *g2 = reinterpret_cast<const ulonglong2 *>(grow + chunk * kQkBK);
                const uint8_t *rowp = smem + S::OFF_X + s * S::X_STAGE + cc * S::X_TILE + row * 128;
#pragma unroll
                for (int c = 0; c < NPC; ++c) {
                    xv[cc * NPC + c] = *reinterpret_cast<const uint4 *>(rowp + (((kpart * NPC + c) ^ (row & 7)) << 4));   // 128-byte swizzle
                    gv[(cc * NPC + c) * 2] = g2[2 * c];
                    gv[(cc * NPC + c) * 2 + 1] = g2[2 * c + 1];
                }
            }
#pragma unroll
            for (int cc = 0; cc < CPS; ++cc) {
                if (ks * CPS + cc < n_chunks) {         // (uniform; a chunk past the end holds TMA's zeros and stays as it is)
                    uint8_t *rowp = smem + S::OFF_X + s * S::X_STAGE + cc * S::X_TILE + row * 128;
#pragma unroll
                    for (int c = 0; c < NPC; ++c) {
                        const uint64_t gg[4] = {gv[(cc * NPC + c) * 2].x, gv[(cc * NPC + c) * 2].y, gv[(cc * NPC + c) * 2 + 1].x, gv[(cc * NPC + c) * 2 + 1].y};
                        uint32_t vv[4] = {xv[cc * NPC + c].x, xv[cc * NPC + c].y, xv[cc * NPC + c].z, xv[cc * NPC + c].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint64_t x2 = pack_f32x2(__uint_as_float(vv[k] << 16), __uint_as_float(vv[k] & 0xFFFF0000u));
                            ss2 = fma_f32x2(x2, x2, ss2);
                            float y0, y1;
                            unpack_f32x2(mul_f32x2(x2, gg[k]), y0, y1);
                            __nv_bfloat162 y2 = __floats2bfloat162_rn(y0, y1);
                            vv[k] = *reinterpret_cast<uint32_t *>(&y2);
                        }
                        *reinterpret_cast<uint4 *>(rowp + (((kpart * NPC + c) ^ (row & 7)) << 4)) = make_uint4(vv[0], vv[1], vv[2], vv[3]);
                    }
                }
            }
            fence_proxy_async_smem();   // the tensor pipe reads what these threads wrote
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(S_BREADY + s));
            if (threadIdx.x == 64) QK_TRACE(2, ks, 4);
        }
        // 1 / RMS of every row (a column of the accumulator), shared by all threads
        float *ssm = reinterpret_cast<float *>(smem + S::OFF_SS);
        {
            float s0, s1;
            unpack_f32x2(ss2, s0, s1);
            ssm[kpart * 128 + row] = s0 + s1;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // ... as a table, one entry per row, behind the partial sums
        float *rsm = ssm + 512;
        if (tid < NT) {
            float ssr = 0.f;
#pragma unroll
            for (int t = 0; t < TP; ++t) ssr += ssm[t * 128 + tid];
            // (contraction split over a cluster: this CTA has seen its slice of the row only; the shares meet in the reduction)
            rsm[tid] = PLAIN ? 1.f : (ksplit > 1 ? ssr : rsqrtf(ssr * (1.f / (float)p.D) + p.eps));
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (threadIdx.x == 64) QK_TRACE(2, 31, 0);
        ok = wait(S_ACC, 0u, 5) && ok;
        if (threadIdx.x == 64) QK_TRACE(2, 31, 1);
        tc_fence_after();
        // epilogue: thread = output feature (TMEM lane), columns = rows of x; the two warps of a lane quarter take alternate
        // blocks of 32 rows
        const int quarter = warp & 3;
        const int egroup = (warp - 2) >> 2;
        const int f = f0 + quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int n_feat = swiglu ? p.swiglu_F : p.nq + 2 * p.nk;
        __nv_bfloat16 *dst0 = nullptr;            // row 0 of this feature's column in the tensor it belongs to
        size_t pitch = 0;
        if (swiglu || f < p.nq) { dst0 = p.q + f; pitch = (size_t)p.nq; }
        else if (f < p.nq + p.nk) { dst0 = p.k + (f - p.nq); pitch = (size_t)p.nk; }
        else { dst0 = p.v + (f - p.nq - p.nk); pitch = (size_t)p.nk; }
#pragma unroll 1
        for (int c = egroup; c < NT / 32; c += 2) {
            uint32_t acc[32], up[32];
            tmem_ld32(tmem + lane_addr + c * 32, acc);          // warp-wide: every lane takes part
            if (swiglu) tmem_ld32(tmem + lane_addr + NT + c * 32, up);
            tmem_wait_ld();
            if (ksplit > 1) {
                // this CTA's share of the sums goes to shared memory (the stage ring is idle: every load has been consumed
                // and every MMA has completed), [row][feature] so that a warp writes 128 contiguous bytes; the up projection's
                // share behind it
                float *part = reinterpret_cast<float *>(smem + S::OFF_W);
                static_assert(S::STAGES * S::W_STAGE >= (uint32_t)NACC * NT * 128 * 4, "partial sums fit in the stage ring");
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    part[(c * 32 + i) * 128 + quarter * 32 + lane] = ok ? __uint_as_float(acc[i]) : __int_as_float(0x7fc00000);
                    if (swiglu) part[(NT + c * 32 + i) * 128 + quarter * 32 + lane] = __uint_as_float(up[i]);
                }
                continue;
            }
            if (!ok || f >= n_feat) continue;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int r = c * 32 + i, rg = row0 + r;
                if (rg < p.M) {                     // (no early exit: the accumulator stays in registers)
                    const float rs = rsm[r];
                    float val = __uint_as_float(acc[i]) * rs;
                    if (swiglu) { const float u = __uint_as_float(up[i]) * rs; val = silu_mul(val, u); }
                    if constexpr (PLAIN) { if (p.res) val += __bfloat162float(p.res[(size_t)rg * pitch + f]); }
                    dst0[(size_t)rg * pitch] = __float2bfloat16_rn(val);    // a warp writes 64 contiguous bytes per row
                }
            }
        }
    }

    if (ksplit > 1) {
        // (cluster barriers are warp-aligned: the lanes of the producer warp that idled while lane 0 ran the loads must
        // not reach them before lane 0 does, so the CTA meets first)
        __syncthreads();
        cluster_arrive();
        cluster_wait();
        // CTA krank adds up rows [krank, krank + 1) * NT / ksplit of all slices and finishes them
        const int rows_mine = NT / ksplit, r0 = krank * rows_mine;
        float *ssm = reinterpret_cast<float *>(smem + S::OFF_SS);
        float *rsm = ssm + 512;                  // [NT] this CTA's share of every row's sum of squares (1 for the plain projection)
        float *rs_mine = ssm;                    // [rows_mine] 1 / RMS of this CTA's rows (the partial sums there have been consumed)
        if (warp >= 2) {
            if constexpr (!PLAIN) {
                const int t = threadIdx.x - 64;
                if (t < rows_mine) {
                    float ss = 0.f, sv[8];
                    const uint32_t a0 = smem_u32(rsm + r0 + t);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {      // (all slices' loads in flight together)
                        sv[q] = 0.f;
                        if (q < ksplit) asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(sv[q]) : "r"(mapa(a0, (uint32_t)q)) : "memory");
                    }
#pragma unroll
                    for (int q = 0; q < 8; ++q) ss += sv[q];
                    rs_mine[t] = rsqrtf(ss * (1.f / (float)p.D) + p.eps);
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            const float *part = reinterpret_cast<const float *>(smem + S::OFF_W);
            const int n_feat = swiglu ? p.swiglu_F : p.nq + 2 * p.nk;
            // four consecutive features of one row per thread and round: one 16-byte load from every slice's partial sums, all of
            // them issued before the first is used. (One feature per thread, its slices read one after the other: 32 dependent
            // round trips through distributed shared memory per thread, 7.7 k of the kernel's 10 k cycles for one stream.)
            for (int e = threadIdx.x - 64; e < rows_mine * 32; e += 256) {
                const int r = r0 + e / 32, fl = (e % 32) * 4, f = f0 + fl;
                const int rg = row0 + r;
                const uint32_t a0 = smem_u32(part + r * 128 + fl);
                float4 v[8], u[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    v[q] = make_float4(0.f, 0.f, 0.f, 0.f); u[q] = v[q];
                    if (q < ksplit) {
                        const uint32_t aq = mapa(a0, (uint32_t)q);
                        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[q].x), "=f"(v[q].y), "=f"(v[q].z), "=f"(v[q].w) : "r"(aq) : "memory");
                        if (swiglu)
                            asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(u[q].x), "=f"(u[q].y), "=f"(u[q].z), "=f"(u[q].w)
                                         : "r"(aq + (uint32_t)NT * 128 * 4) : "memory");
                    }
                }
                float sum[4] = {0.f, 0.f, 0.f, 0.f}, sum_up[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    sum[0] += v[q].x; sum[1] += v[q].y; sum[2] += v[q].z; sum[3] += v[q].w;
                    sum_up[0] += u[q].x; sum_up[1] += u[q].y; sum_up[2] += u[q].z; sum_up[3] += u[q].w;
                }
                if (rg >= p.M || f >= n_feat) continue;      // (feature counts are multiples of 8: the four stand or fall together, in one tensor)
                __nv_bfloat16 *dst;
                if (swiglu || f < p.nq) dst = p.q + (size_t)rg * p.nq + f;
                else if (f < p.nq + p.nk) dst = p.k + (size_t)rg * p.nk + (f - p.nq);
                else dst = p.v + (size_t)rg * p.nk + (f - p.nq - p.nk);
                if constexpr (PLAIN) {
                    if (p.res) {
                        const uint2 rr = *reinterpret_cast<const uint2 *>(p.res + (size_t)rg * p.nq + f);
                        sum[0] += __uint_as_float(rr.x << 16); sum[1] += __uint_as_float(rr.x & 0xFFFF0000u);
                        sum[2] += __uint_as_float(rr.y << 16); sum[3] += __uint_as_float(rr.y & 0xFFFF0000u);
                    }
                } else {
                    const float rs = rs_mine[r - r0];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        sum[i] *= rs;
                        if (swiglu) sum[i] = silu_mul(sum[i], sum_up[i] * rs);
                    }
                }
                __nv_bfloat162 h0 = __floats2bfloat162_rn(sum[0], sum[1]), h1 = __floats2bfloat162_rn(sum[2], sum[3]);
                uint2 o;
                o.x = *reinterpret_cast<uint32_t *>(&h0); o.y = *reinterpret_cast<uint32_t *>(&h1);
                *reinterpret_cast<uint2 *>(dst) = o;
            }
        }
        cluster_arrive();
        cluster_wait();   // no CTA retires while a peer may still read its partial sums
    }
    if (threadIdx.x == 64) QK_TRACE(2, 31, 2);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kCols);
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
                     int R, int D, int nq, int nk, int swiglu_F, float eps)
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
    if (swiglu_F > 0) {     // W = [W_gate; W_up], q = out [M][F]
        for (int f = threadIdx.x; f < swiglu_F; f += blockDim.x) {
            const T *wg = W + (size_t)f * D, *wu = W + (size_t)(swiglu_F + f) * D;
            float g = 0.f, u = 0.f;
            for (int i = 0; i < D; ++i) { g = fmaf(ysm[i], qk_to_f<T>(wg[i]), g); u = fmaf(ysm[i], qk_to_f<T>(wu[i]), u); }
            g *= rs; u *= rs;
            q[r * swiglu_F + f] = qk_from_f<T>(g / (1.f + expf(-g)) * u);
        }
        return;
    }
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
cudaError_t launch_simt(const void *x, const float *gate, const void *W, void *q, void *k, void *v, int M, int R, int D, int nq, int nk, int swiglu_F,
                        float eps, cudaStream_t st)
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, norm_qkv_simt_kernel<T>, (const T *)x, gate, (const T *)W, (T *)q, (T *)k, (T *)v, R, D, nq, nk, swiglu_F, eps);
    count_launch();
    return e;
}

}  // namespace

// 256-column tiles unless they would need more than one wave of SM pairs and the gates of a CTA's streams still fit
// beside the larger stages
static int qk_choose_nacc(int M, int R, int D, int n_out, int sm_count)
{
    const size_t gate_bytes = (size_t)((kQkBM - 1) / R + 2) * D * sizeof(float);
    const long long m_tiles = (M + 2 * kQkBM - 1) / (2 * kQkBM);
    const long long tiles1 = m_tiles * ((n_out + kQkBN - 1) / kQkBN);
    if (tiles1 > sm_count / 2 && gate_bytes <= QkSmem<2>::GATE_MAX) return 2;
    return gate_bytes <= QkSmem<1>::GATE_MAX ? 1 : 0;
}

bool norm_qkv_tc_supported(int dtype, int B, int R, int D, int nq, int nk)
{
    if (dtype != REFLEX_DTYPE_BF16 || B < 1 || R < 1) return false;
    if (D < kQkBK || D % kQkBK != 0) return false;
    if (nq % 8 != 0 || nk % 8 != 0) return false;
    if ((long long)B * R > 0x3FFFFFFF) return false;
    return qk_choose_nacc(B * R, R, D, nq + 2 * nk, 148) != 0;   // gates of a CTA's streams must fit in shared memory
}

template <int NACC>
static cudaError_t launch_tc(const CUtensorMap &mx, const CUtensorMap &mw, QkParams p, int n_tiles, int sm_count, cudaStream_t st)
{
    // tensor maps over the outputs when every tensor's width is a multiple of the 64-column chunks the epilogue stores
    CUtensorMap mq = mx, mk = mx, mv = mx;
    p.tma_out = 0;
    if (p.swiglu_F > 0) {
        p.tma_out = tensor_map_2d_bf16(&mq, p.q, p.swiglu_F, p.M, kQkBM) ? 1 : 0;
    } else if (p.nq % 64 == 0 && p.nk % 64 == 0) {
        p.tma_out = (tensor_map_2d_bf16(&mq, p.q, p.nq, p.M, kQkBM) && tensor_map_2d_bf16(&mk, p.k, p.nk, p.M, kQkBM) &&
                     tensor_map_2d_bf16(&mv, p.v, p.nk, p.M, kQkBM)) ? 1 : 0;
    }
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        cudaError_t e = cudaFuncSetAttribute(norm_qkv_tc_kernel<NACC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QkSmem<NACC>::TOTAL);
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(norm_qkv_tc_kernel<NACC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QkSmem<NACC>::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    cudaLaunchConfig_t cfg = {};
    // one CTA pair per tile, or per SM pair when there are more tiles than that (the pairs then walk the tiles; the
    // hand-overs between tiles go with the TMA-store epilogue)
    p.n_tiles = n_tiles;
    const unsigned tiles = (unsigned)p.m_tiles * (unsigned)n_tiles;
    const unsigned pairs_max = (unsigned)((sm_count > 0 ? sm_count : 148) / 2);
    const bool walk = p.tma_out && tiles > pairs_max && pairs_max > 0;
    cfg.gridDim = dim3(2u * (walk ? pairs_max : tiles));
    cfg.blockDim = dim3(kQkThreads);
    cfg.dynamicSmemBytes = QkSmem<NACC>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = walk ? cudaLaunchKernelEx(&cfg, norm_qkv_tc_kernel<NACC, true>, mx, mw, mq, mk, mv, p)
                         : cudaLaunchKernelEx(&cfg, norm_qkv_tc_kernel<NACC, false>, mx, mw, mq, mk, mv, p);
    count_launch();
    return e;
}

template <int NT, int NACC, bool PLAIN = false>
static cudaError_t launch_small(const CUtensorMap &mx, const CUtensorMap &mw, QkParams p, unsigned grid, unsigned groups, cudaStream_t st)
{
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        return cudaFuncSetAttribute(norm_linear_small_kernel<NT, NACC, PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SmSmem<NT, NACC>::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, groups);
    cfg.blockDim = dim3(kSmThreads);
    cfg.dynamicSmemBytes = SmSmem<NT, NACC>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // plain projection: the CTAs that split one feature tile's contraction
    attr[1].val.clusterDim.x = (unsigned)p.ksplit; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.ksplit > 1 ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, norm_linear_small_kernel<NT, NACC, PLAIN>, mx, mw, p);
    count_launch();
    return e;
}

// swiglu_F = 0: W = W_QKV, outputs q / k / v with nq and nk columns. swiglu_F = F > 0: W = [W_gate; W_up] ([2F][D]),
// q = the [M][F] output SiLU(gate) * up; nq, nk, k, v unused.
cudaError_t launch_adarmsnorm_qkv(const void *x, const float *gate, const void *W, void *q, void *k, void *v, int B, int R, int D, int nq, int nk,
                                  int swiglu_F, float eps, int dtype, int impl, int sm_count, uint32_t *status, cudaStream_t st)
{
    const int M = B * R;
    if (swiglu_F > 0) { nq = swiglu_F; nk = 0; }
    const size_t gate_bytes = (size_t)((kQkBM - 1) / R + 2) * D * sizeof(float);
    const bool tc = impl != 1 && norm_qkv_tc_supported(dtype, B, R, D, nq, nk) && (swiglu_F == 0 || gate_bytes <= QkSmem<2>::GATE_MAX);
    if (!tc) {
        if ((size_t)(D + 8) * sizeof(float) > 48 * 1024) return cudaErrorInvalidValue;
        return dtype == REFLEX_DTYPE_BF16 ? launch_simt<__nv_bfloat16>(x, gate, W, q, k, v, M, R, D, nq, nk, swiglu_F, eps, st)
                                          : launch_simt<float>(x, gate, W, q, k, v, M, R, D, nq, nk, swiglu_F, eps, st);
    }
    const int w_rows = swiglu_F > 0 ? 2 * swiglu_F : nq + 2 * nk;
    // Few rows: weights as the A operand, one CTA per 128 output features and group of rows. One group of 64 or 128 rows, or,
    // while every (feature tile, group) still has an SM of its own, several groups of 64: the chain of a CTA stays as short as for
    // one stream (100 rows as two groups of 64: 6.6 us against 10.0 as one group of 128; 200 rows: 6.8 against 11.6 with the
    // 256-row tiles). Beyond that, groups of 128 rows under the same condition (450-800 rows: 10.4 us against 11.7-12.2).
    const int sms = sm_count > 0 ? sm_count : 148;
    const int n_feat = swiglu_F > 0 ? swiglu_F : nq + 2 * nk;
    const int ftiles = (n_feat + 127) / 128;
    auto gates_fit = [&](int nt) { return (size_t)std::min(B, (nt - 1) / R + 2) * D * sizeof(float) <= SmSmem<64, 1>::GATE_MAX; };
    int NT = 0, groups = 1;
    if (impl == 0) {
        if (M <= 64 && gates_fit(64)) NT = 64;
        else if (gates_fit(64) && ((M + 63) / 64) * ftiles <= sms) { NT = 64; groups = (M + 63) / 64; }
        else if (gates_fit(128) && ((M + 127) / 128) * ftiles <= sms) { NT = 128; groups = (M + 127) / 128; }
    }
    if (NT != 0) {
        CUtensorMap sx, sw;
        if (!tensor_map_2d_bf16(&sx, x, D, M, NT) || !tensor_map_2d_bf16(&sw, W, D, w_rows, 128)) return cudaErrorInvalidValue;
        QkParams sp;
        sp.gate = gate; sp.q = (__nv_bfloat16 *)q; sp.k = (__nv_bfloat16 *)k; sp.v = (__nv_bfloat16 *)v;
        sp.M = M; sp.R = R; sp.B = B; sp.D = D; sp.nq = nq; sp.nk = nk; sp.m_tiles = 1; sp.n_tiles = 1; sp.swiglu_F = swiglu_F;
        sp.eps = eps; sp.status = status; sp.res = nullptr; sp.tma_out = 0;
        // The contraction split over 4 CTAs per (feature tile, row group) where the chain has 8 steps or more and the grid stays
        // within the SMs, every slice keeping whole steps: the slices' sums meet through distributed shared memory, four
        // features per thread and all slices' loads in flight together (one stream: Q/K/V 6.4 -> 5.9 us, gate/up 11.1 -> 8.6;
        // with one feature per thread and its slices read one after the other the reduction alone took 7.7 k cycles and
        // the split made the Q/K/V projection slower). A split in two only pays for chains of 16 steps (gate/up, 100 rows:
        // 10.3 -> 9.5 us; Q/K/V: 6.6 -> 6.8).
        const int chunks = D / kQkBK, cps = swiglu_F > 0 ? 1 : 2;
        int ks = 1;
        if (chunks / cps >= 8 && chunks % (4 * cps) == 0 && ftiles * groups * 4 <= sms) ks = 4;
        else if (chunks / cps >= 16 && chunks % (2 * cps) == 0 && ftiles * groups * 2 <= sms) ks = 2;
        sp.ksplit = ks;
        const unsigned grid = (unsigned)(ftiles * ks);
        if (swiglu_F > 0) return NT == 64 ? launch_small<64, 2>(sx, sw, sp, grid, (unsigned)groups, st) : launch_small<128, 2>(sx, sw, sp, grid, (unsigned)groups, st);
        return NT == 64 ? launch_small<64, 1>(sx, sw, sp, grid, (unsigned)groups, st) : launch_small<128, 1>(sx, sw, sp, grid, (unsigned)groups, st);
    }
    CUtensorMap mx, mw;
    if (!tensor_map_2d_bf16(&mx, x, D, M, kQkBM) || !tensor_map_2d_bf16(&mw, W, D, w_rows, kQkBN / 2)) return cudaErrorInvalidValue;
    QkParams p;
    p.gate = gate; p.q = (__nv_bfloat16 *)q; p.k = (__nv_bfloat16 *)k; p.v = (__nv_bfloat16 *)v;
    p.M = M; p.R = R; p.B = B; p.D = D; p.nq = nq; p.nk = nk;
    p.m_tiles = (M + 2 * kQkBM - 1) / (2 * kQkBM);
    p.swiglu_F = swiglu_F;
    p.eps = eps; p.status = status; p.res = nullptr; p.ksplit = 1; p.tma_out = 0;
    if (swiglu_F > 0) return launch_tc<2>(mx, mw, p, (swiglu_F + kQkBN - 1) / kQkBN, sm_count, st);
    int nacc = qk_choose_nacc(M, R, D, nq + 2 * nk, sm_count > 0 ? sm_count : 148);
    if (impl == 2 && nacc == 2) nacc = 1;     // (forced 256-column tiles, for tests and timing)
    const int n_out = nq + 2 * nk;
    return nacc == 2 ? launch_tc<2>(mx, mw, p, (n_out + 2 * kQkBN - 1) / (2 * kQkBN), sm_count, st)
                     : launch_tc<1>(mx, mw, p, (n_out + kQkBN - 1) / kQkBN, sm_count, st);
}

// out [M][N] = res + a [M][K] W [N][K]^T for few rows (K a multiple of 64): the few-rows kernel without its norm stage
// Row groups of the plain projection: groups of 64 rows pay while the contraction (2048 or more) can still be split over 4 CTAs
// per (feature tile, group) inside the SMs: 200 rows x 4096 -> 1024 7.8 us against 15.4 with the 256-row tiles, x 2048 6.4
// against 9.2 (before the slices' sums were added four features per thread with all loads in flight: 10.9 and 9.6); 300 rows
// and more: the tiles.
static int linear_small_groups(int M, int K, int N)
{
    const int chunks = K / kQkBK, ftiles = (N + 127) / 128, groups = (M + 63) / 64;
    if (M <= 64) return 1;
    if (chunks % 8 == 0 && chunks >= 32 && ftiles * groups * 4 <= 148) return groups;
    return M <= 128 ? 1 : 0;       // one group of 128 rows, or not this kernel's shape
}

bool linear_small_takes(int M, int K, int N)
{
    return K % kQkBK == 0 && linear_small_groups(M, K, N) > 0;
}

cudaError_t launch_linear_small(const void *a, const void *W, const void *res, void *out, int M, int K, int N, uint32_t *status, cudaStream_t st)
{
    const int ftiles = (N + 127) / 128;
    const int groups = linear_small_groups(M, K, N);
    const int NT = (groups > 1 || M <= 64) ? 64 : 128;
    CUtensorMap sx, sw;
    if (!tensor_map_2d_bf16(&sx, a, K, M, NT) || !tensor_map_2d_bf16(&sw, W, K, N, 128)) return cudaErrorInvalidValue;
    QkParams sp;
    sp.gate = nullptr; sp.q = (__nv_bfloat16 *)out; sp.k = nullptr; sp.v = nullptr;
    sp.M = M; sp.R = M; sp.B = 1; sp.D = K; sp.nq = N; sp.nk = 0; sp.m_tiles = 1; sp.n_tiles = 1; sp.swiglu_F = 0;
    sp.eps = 0.f; sp.status = status; sp.res = (const __nv_bfloat16 *)res; sp.tma_out = 0;
    // split the contraction over up to 8 CTAs per (feature tile, row group) while every slice keeps whole steps of two 64-column
    // chunks and the grid stays within the SMs
    const int chunks = K / kQkBK;
    int ks = 1;
    if (groups > 1) ks = 4;       // (clusters of 8 CTAs: the device holds 16 of them at once)
    else while (ks < 8 && chunks % (4 * ks) == 0 && chunks / (2 * ks) >= 2 && ftiles * 2 * ks <= 148) ks *= 2;
    sp.ksplit = ks;
    const unsigned grid = (unsigned)(ftiles * ks);
    return NT == 64 ? launch_small<64, 1, true>(sx, sw, sp, grid, (unsigned)groups, st) : launch_small<128, 1, true>(sx, sw, sp, grid, 1u, st);
}

}  // namespace reflex

#ifdef REFLEX_QK_TRACE
extern "C" int reflex_debug_qk_trace(long long *out)
{
    return (int)cudaMemcpyFromSymbol(out, reflex::g_qk_trace, sizeof(long long) * 3 * 32 * 8);
}
#endif
