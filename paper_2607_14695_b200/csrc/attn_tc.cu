// Partitioned attention (Eq. 1) on the 5th-generation tensor cores: tcgen05.mma with TMEM accumulators,
// K/V tiles of the three regions staged by TMA straight from where they live (static rows and ring slots
// of the slab, dynamic tokens from the caller's tensors) -- no gather, no copy.
//
// One CTA owns one 128-row query tile of one (stream, KV head): rows are (token, head-in-group) pairs, so
// all G query heads that share a KV head ride in the same MMA. It walks 64-key tiles with an online
// softmax:
//   warp 0        TMA producer (Q once, then K and V tiles through a 2-stage ring each)
//   warp 1        MMA issuer: S = Q K^T (M128 N64, K-major operands), O += P V (M128 N=d, V is MN-major)
//   warps 2..5    softmax: S from TMEM, mask, running max / sum, P (bf16) into swizzled shared memory,
//                 lazy rescale of O in TMEM, final normalisation and store
// S is double buffered in TMEM and P in shared memory, so Q K^T of tile j+1 overlaps the softmax of tile j.
// With nsplit > 1 a CTA covers a slice of the key tiles and writes an (m, l, O) partial that the merge
// kernel of the SIMT path combines.
//
// Every wait on an mbarrier is bounded; when one runs out the CTA raises a status word, stops waiting and
// drains, so a mistake cannot hang the device.
#include <cuda.h>

#include <map>
#include <mutex>
#include <tuple>

#include "reflex_internal.cuh"
#include "sm100_ptx.cuh"

namespace reflex {

using namespace ptx;

constexpr int kBM = 128;        // query rows per CTA
constexpr int kBN = 64;         // keys per tile
constexpr int kStages = 2;      // K and V ring depth
constexpr int kTcThreads = 192;
constexpr unsigned long long kWaitNs = 1000000000ull;  // every mbarrier wait gives up after ~1 s
constexpr float kRescaleThreshold = 8.0f;  // in log2 units: O is rescaled only when the max grows by > 2^8

struct TcParams {
    const StreamState *state;
    void *out;
    float *partials;
    uint32_t *status;
    int B, L, Hq, Hkv, G, S_max, N, T, layer;
    int ring_off;      // first ring row of a (layer, stream) block: S_max times the number of static banks
    int dyn_mask;
    float scale, scale_log2;
    int nsplit;
    int tile_tokens;  // 128 / G (two-CTA kernel with live_rows = 64: half of that)
    int live_rows;    // rows of a CTA's 128-row tile that belong to its tokens: 128, or 64 (two-CTA kernel, key-split units of few streams)
    int n_qtiles;
    int cluster_merge;  // one-CTA kernel: the nsplit key slices of a query tile form a cluster and merge through shared memory
};

template <int HD> struct TcSmem {
    static constexpr int CH = HD / 64;                  // 64-element (128-byte) chunks along head_dim
    static constexpr uint32_t Q_BYTES = CH * kBM * 128;
    static constexpr uint32_t KV_STAGE = CH * kBN * 128;
    static constexpr uint32_t P_BYTES = kBM * 128;
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = OFF_Q + Q_BYTES;
    static constexpr uint32_t OFF_V = OFF_K + kStages * KV_STAGE;
    static constexpr uint32_t OFF_P = OFF_V + kStages * KV_STAGE;
    static constexpr uint32_t OFF_BAR = OFF_P + 2 * P_BYTES;
    static constexpr uint32_t TOTAL = OFF_BAR + 256 + 1024;  // barriers + slack to align the base to 1024 B
};

// barrier slots (8 bytes each) from OFF_BAR
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_SEMPTY = 11, B_PFULL = 13, B_PVDONE = 15, B_COUNT = 17 };

struct TileRef {
    int dyn;            // 0: slab map, 1: dynamic-token map
    int row0;           // first row of the tile in that map's row axis
    int kind;           // 0 static, 1 ring, 2 dynamic
    int idx;            // tile index inside its region
};

struct TileGeom {
    int S, N, T, count, oldest, ns, nr, nd, row_base, s_off, ring_off, b;   // s_off: first row of the static bank in use
    __device__ __forceinline__ TileRef decode(int it) const
    {
        TileRef t;
        if (it < ns) { t.dyn = 0; t.kind = 0; t.idx = it; t.row0 = row_base + s_off + it * kBN; }
        else if (it < ns + nr) { t.dyn = 0; t.kind = 1; t.idx = it - ns; t.row0 = row_base + ring_off + t.idx * kBN; }
        else { t.dyn = 1; t.kind = 2; t.idx = it - ns - nr; t.row0 = b * T + t.idx * kBN; }
        return t;
    }
    // bits [lo, hi) of a 64-bit word (0 <= lo, hi <= 64)
    static __device__ __forceinline__ uint64_t bit_range(int lo, int hi)
    {
        lo = max(lo, 0); hi = min(hi, 64);
        if (hi <= lo) return 0ull;
        const uint64_t upto_hi = (hi >= 64) ? ~0ull : ((1ull << hi) - 1ull);
        return upto_hi & ~((1ull << lo) - 1ull);
    }
    // which of the 64 keys of a tile are live (independent of the query row)
    __device__ __forceinline__ uint64_t tile_mask(const TileRef &t) const
    {
        const int base = t.idx * kBN;
        if (t.kind == 1) {
            // live ring slots are the circular run of `count` slots that starts at `oldest`
            const int c = min(count, N);
            const int end = oldest + c;                       // may pass N: the run wraps
            uint64_t m = bit_range(oldest - base, min(end, N) - base);
            if (end > N) m |= bit_range(0 - base, end - N - base);
            return m;
        }
        const int len = (t.kind == 0) ? S : T;
        return bit_range(0, len - base);
    }
};

// s[c] = -inf for every key c of a 64-key half that `mask` marks dead (constant bit tests, two selects per word)
__device__ __forceinline__ void apply_key_mask(float (&s)[64], uint64_t mask)
{
    const uint32_t lo = (uint32_t)mask, hi = (uint32_t)(mask >> 32);
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        if (!(lo & (1u << c))) s[c] = -INFINITY;
        if (!(hi & (1u << c))) s[32 + c] = -INFINITY;
    }
}

template <int HD>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kd,
               const __grid_constant__ CUtensorMap tm_vd, const TcParams p)
{
    using L = TcSmem<HD>;
    constexpr int CH = L::CH;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColO = 0, kColS = HD;  // O: HD fp32 columns; S: 2 x 64 columns
    static_assert(HD + 2 * kBN <= 512, "TMEM budget");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar0 = base + L::OFF_BAR;
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * (uint32_t)i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L::OFF_BAR + 8 * B_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    // programmatic dependent launch: scheduled, perhaps, before the kernel ahead on the stream has finished; nothing is read
    // before it has. The kernel after this one may be scheduled once every CTA here has started (it waits the same way).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = blockIdx.x % p.n_qtiles;
    const int kvh = blockIdx.x / p.n_qtiles;
    const int b = blockIdx.y;
    const int split = blockIdx.z;
    const int t0 = qt * p.tile_tokens;

    TileGeom g;
    {
        const StreamState st = p.state[b];
        g.S = st.static_len > 0 ? st.static_len : 0;
        g.N = p.N; g.T = p.T; g.count = st.count;
        g.oldest = (st.head - st.count) % p.N;
        if (g.oldest < 0) g.oldest += p.N;
        g.ns = (g.S + kBN - 1) / kBN;
        g.nr = g.count > 0 ? (p.N + kBN - 1) / kBN : 0;
        g.nd = (p.T + kBN - 1) / kBN;
        g.row_base = (p.layer * p.B + b) * (p.ring_off + p.N);
        g.s_off = st.bank * p.S_max; g.ring_off = p.ring_off; g.b = b;
    }
    const int n_tiles = g.ns + g.nr + g.nd;
    const int per = (n_tiles + p.nsplit - 1) / p.nsplit;
    const int it0 = split * per;
    const int it1 = min(n_tiles, it0 + per);
    const int n_local = max(0, it1 - it0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            const bool many = (i == B_SEMPTY || i == B_SEMPTY + 1 || i == B_PFULL || i == B_PFULL + 1);
            mbar_init(bar(i), many ? 128u : 1u);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v); prefetch_tmap(&tm_kd); prefetch_tmap(&tm_vd);
    }
    if (warp == 1) tmem_alloc(smem_u32((const void *)tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // bounded wait (about one second of wall time): false, and the abort flag raised, when the barrier never flips
    auto wait = [&](int i, uint32_t parity, uint32_t code) -> bool {
        if (mbar_try_wait(bar(i), parity)) return true;
        const unsigned long long t_start = globaltimer_ns();
        for (uint32_t n = 1;; ++n) {
            if (mbar_try_wait(bar(i), parity)) return true;
            if ((n & 255u) == 0u) {
                if (*abort_flag) return false;
                if (globaltimer_ns() - t_start > kWaitNs) break;
            }
        }
        *abort_flag = 1u;
        atomicCAS(p.status, 0u, 0x80000000u | (code << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };

    // what a softmax thread carries into the in-cluster merge (cluster_merge): its row's maximum (log2 units) and sum
    float fin_m = -INFINITY, fin_l = 0.f;
    bool fin_ok = true;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && n_local > 0) {
            mbar_expect_tx(bar(B_QFULL), L::Q_BYTES);
            for (int c = 0; c < CH; ++c)
                tma_load_4d(base + L::OFF_Q + c * (kBM * 128), &tm_q, bar(B_QFULL), c * 64, kvh * p.G, t0, b);
            bool ok = true;
            for (int jj = 0; jj < n_local && ok; ++jj) {
                const int st = jj % kStages;
                const uint32_t ph = (uint32_t)((jj / kStages) - 1) & 1u;
                const TileRef tr = g.decode(it0 + jj);
                if (jj >= kStages) ok = wait(B_KEMPTY + st, ph, 1);
                if (!ok) break;
                mbar_expect_tx(bar(B_KFULL + st), L::KV_STAGE);
                for (int c = 0; c < CH; ++c)
                    tma_load_3d(base + L::OFF_K + st * L::KV_STAGE + c * (kBN * 128), tr.dyn ? &tm_kd : &tm_k, bar(B_KFULL + st),
                                c * 64, kvh, tr.row0);
                if (jj >= kStages) ok = wait(B_VEMPTY + st, ph, 2);
                if (!ok) break;
                mbar_expect_tx(bar(B_VFULL + st), L::KV_STAGE);
                for (int c = 0; c < CH; ++c)
                    tma_load_3d(base + L::OFF_V + st * L::KV_STAGE + c * (kBN * 128), tr.dyn ? &tm_vd : &tm_v, bar(B_VFULL + st),
                                c * 64, kvh, tr.row0);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // (the whole warp runs the loop converged, one elected lane issues: see umma_ss_elect)
        if (n_local > 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(kBM, kBN, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(kBM, HD, true);
            auto issue_qk = [&](int jj) {
                const int st = jj % kStages, buf = jj & 1;
                const uint32_t d_tmem = tmem_base + kColS + buf * kBN;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t a = base + L::OFF_Q + (kk >> 2) * (kBM * 128) + (kk & 3) * 32;
                    const uint32_t bb = base + L::OFF_K + st * L::KV_STAGE + (kk >> 2) * (kBN * 128) + (kk & 3) * 32;
                    umma_ss_elect(d_tmem, umma_desc_sw128(a, 16, 1024), umma_desc_sw128(bb, 16, 1024), idesc_qk, kk > 0 ? 1u : 0u);
                }
                umma_commit_elect(bar(B_KEMPTY + st));
                umma_commit_elect(bar(B_SFULL + buf));
            };
            bool ok = wait(B_QFULL, 0, 3) && wait(B_KFULL + 0, 0, 4);
            if (ok) { tc_fence_after(); issue_qk(0); }
            for (int jj = 0; jj < n_local && ok; ++jj) {
                if (jj + 1 < n_local) {
                    const int nj = jj + 1;
                    ok = wait(B_KFULL + (nj % kStages), (uint32_t)(nj / kStages) & 1u, 5);
                    if (ok && nj >= 2) ok = wait(B_SEMPTY + (nj & 1), (uint32_t)((nj >> 1) - 1) & 1u, 6);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(nj);
                }
                const int st = jj % kStages, buf = jj & 1;
                ok = wait(B_VFULL + st, (uint32_t)(jj / kStages) & 1u, 7) && wait(B_PFULL + buf, (uint32_t)(jj >> 1) & 1u, 8);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk) {
                    const uint32_t a = base + L::OFF_P + buf * L::P_BYTES + kk * 32;
                    const uint32_t bb = base + L::OFF_V + st * L::KV_STAGE + kk * (16 * 128);
                    umma_ss_elect(tmem_base + kColO, umma_desc_sw128(a, 16, 1024), umma_desc_sw128(bb, kBN * 128, 1024), idesc_pv,
                            (jj > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit_elect(bar(B_VEMPTY + st));
                umma_commit_elect(bar(B_PVDONE + buf));
            }
        }
    } else {
        // ---------------- softmax / correction / epilogue: one query row per thread ----------------
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int t_row = t0 + row / p.G;
        const int hq = kvh * p.G + row % p.G;
        const bool row_live = t_row < p.T && row < p.tile_tokens * p.G;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int jj = 0; jj < n_local && ok; ++jj) {
            const int buf = jj & 1;
            const uint32_t ph = (uint32_t)(jj >> 1) & 1u;
            const TileRef tr = g.decode(it0 + jj);
            const uint64_t tmask = g.tile_mask(tr);
            uint64_t rmask = tmask;
            if (tr.kind == 2 && p.dyn_mask) {
                const int lim = t_row - tr.idx * kBN;
                rmask &= (lim < 0) ? 0ull : (lim >= 63 ? ~0ull : ((2ull << lim) - 1ull));
            }
            ok = wait(B_SFULL + buf, ph, 9);
            if (!ok) break;
            tc_fence_after();
            uint32_t r0[32], r1[32];
            const uint32_t s_addr = tmem_base + lane_addr + kColS + buf * kBN;
            tmem_ld32(s_addr, r0);
            tmem_ld32(s_addr + 32, r1);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(B_SEMPTY + buf));
            float s[64];
#pragma unroll
            for (int c = 0; c < 32; ++c) { s[c] = __uint_as_float(r0[c]); s[32 + c] = __uint_as_float(r1[c]); }
            if (rmask != ~0ull) apply_key_mask(s, rmask);
            float mx = s[0];
#pragma unroll
            for (int c = 1; c < 64; ++c) mx = fmaxf(mx, s[c]);
            if (jj == 0) {
                m_ref = mx;
            } else {
                const bool grow = (mx - m_ref) * p.scale_log2 > kRescaleThreshold;
                if (__any_sync(0xffffffffu, grow)) {
                    // O (and l) were accumulated against m_ref: bring them to the new reference before this tile's P V
                    const float alpha = grow ? ex2((m_ref - mx) * p.scale_log2) : 1.f;
                    if (grow) m_ref = mx;
                    l *= alpha;
                    ok = wait(B_PVDONE + ((jj - 1) & 1), (uint32_t)((jj - 1) >> 1) & 1u, 10);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < HD / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tmem_base + lane_addr + kColO + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tmem_base + lane_addr + kColO + c * 32, o);
                    }
                    tmem_wait_st();
                }
            }
            const float mr = (m_ref == -INFINITY) ? 0.f : m_ref * p.scale_log2;
            float sum = 0.f;
            uint32_t packed[32];
#pragma unroll
            for (int c = 0; c < 64; c += 2) {
                const float p0 = ex2(fmaf(s[c], p.scale_log2, -mr));
                const float p1 = ex2(fmaf(s[c + 1], p.scale_log2, -mr));
                sum += p0 + p1;
                __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                packed[c >> 1] = *reinterpret_cast<uint32_t *>(&h);
            }
            l += sum;
            if (jj >= 2) {
                ok = wait(B_PVDONE + buf, (uint32_t)((jj >> 1) - 1) & 1u, 11);  // P[buf] was read by the P V of tile jj-2
                if (!ok) break;
            }
            uint8_t *p_row = smem + L::OFF_P + buf * L::P_BYTES + row * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 v = make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                *reinterpret_cast<uint4 *>(p_row + ((c ^ (row & 7)) << 4)) = v;
            }
            if (tmask != ~0ull) {
                // dead keys get weight 0, but 0 x (stale NaN/Inf bytes) would still poison O: clear their V rows
                const int st = jj % kStages;
                ok = wait(B_VFULL + st, (uint32_t)(jj / kStages) & 1u, 12);
                if (!ok) break;
                if (row < kBN && !((tmask >> row) & 1ull)) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        uint4 *vr = reinterpret_cast<uint4 *>(smem + L::OFF_V + st * L::KV_STAGE + c * (kBN * 128) + row * 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i) vr[i] = make_uint4(0, 0, 0, 0);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL + buf));
        }
        // ---- epilogue ----
        if (n_local > 0 && ok) {
            const int last = n_local - 1;
            ok = wait(B_PVDONE + (last & 1), (uint32_t)(last >> 1) & 1u, 13);
        }
        const int rows_total = p.T * p.Hq;
        if (p.nsplit == 1) {
            if (n_local > 0 && ok) {
                tc_fence_after();
                const float inv = 1.f / l;
                __nv_bfloat16 *orow = (__nv_bfloat16 *)p.out + (((size_t)b * p.T + t_row) * p.Hq + hq) * HD;
#pragma unroll 1
                for (int c = 0; c < HD / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + c * 32, o);
                    tmem_wait_ld();
                    if (row_live) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 v;
                            uint32_t *vv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 2 * k]) * inv,
                                                                         __uint_as_float(o[8 * i + 2 * k + 1]) * inv);
                                vv[k] = *reinterpret_cast<uint32_t *>(&h);
                            }
                            *reinterpret_cast<uint4 *>(orow + c * 32 + i * 8) = v;
                        }
                    }
                }
            }
        } else if (p.cluster_merge) {
            fin_ok = ok;
            if (n_local > 0 && ok) { fin_m = (m_ref == -INFINITY) ? -INFINITY : m_ref * p.scale_log2; fin_l = l; }
        } else {
            const size_t slot = partial_slot(b, rows_total, t_row * p.Hq + hq, p.nsplit, split);
            float *po = partial_o(p.partials, slot, HD);
            float *pml = partial_ml(p.partials, (size_t)p.B * rows_total * p.nsplit, slot, HD);
            if (n_local > 0 && ok) {
                tc_fence_after();
                if (row_live) { pml[0] = (m_ref == -INFINITY) ? -INFINITY : m_ref * p.scale; pml[1] = l; }
#pragma unroll 1
                for (int c = 0; c < HD / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + c * 32, o);
                    tmem_wait_ld();
                    if (row_live) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            *reinterpret_cast<float4 *>(po + c * 32 + 4 * i) = make_float4(__uint_as_float(o[4 * i]), __uint_as_float(o[4 * i + 1]),
                                                                                           __uint_as_float(o[4 * i + 2]), __uint_as_float(o[4 * i + 3]));
                    }
                }
            } else if (row_live) {
                pml[0] = -INFINITY; pml[1] = 0.f;
            }
        }
    }

    if (p.nsplit > 1 && p.cluster_merge) {
        // ---- merge of the key slices inside the cluster (one CTA per slice, all of the same query tile) ----
        // 1. every softmax thread publishes its row's (m, l); 2. with everybody's (m, l) it scales its own O row to the
        // common maximum and stages it in shared memory (the Q / K / V buffers are idle now), column-major in 16-byte
        // units so that rows (lanes) are contiguous; 3. CTA s adds up columns [s, s+1) * head_dim / nsplit of all slices
        // through distributed shared memory, divides by the common sum and writes them. Three cluster barriers: after
        // 1, after 2, and before anybody leaves (a peer may still be reading this CTA's staging area).
        const int ns = p.nsplit;
        const uint32_t my_rank = cluster_ctarank();
        float2 *ml_own = reinterpret_cast<float2 *>(smem + L::OFF_P);                  // [128 rows]
        float4 *stage = reinterpret_cast<float4 *>(smem + L::OFF_Q);                   // [HD / 4][128 rows]
        const int row_m = (warp & 3) * 32 + lane;
        // (the cluster barriers are warp-aligned instructions: the lanes of the producer warp that idled while lane 0 ran the
        // loads must not reach them before lane 0 does, so the CTA meets here first)
        __syncthreads();
        if (warp >= 2) ml_own[row_m] = make_float2(fin_m, fin_l);
        cluster_arrive();
        cluster_wait();
        float w_own = 0.f, l_all = 0.f;
        uint32_t live_peers = 0u;
        if (warp >= 2) {
            float mstar = -INFINITY;
            float pm[8], pl[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                pm[q] = -INFINITY; pl[q] = 0.f;
                if (q < ns) {
                    const uint32_t a = mapa(smem_u32(ml_own + row_m), (uint32_t)q);
                    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(pm[q]), "=f"(pl[q]) : "r"(a) : "memory");
                }
                mstar = fmaxf(mstar, pm[q]);
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float wq = (pm[q] == -INFINITY) ? 0.f : ex2(pm[q] - mstar);
                l_all = fmaf(pl[q], wq, l_all);
                if (pl[q] * wq > 0.f) live_peers |= 1u << q;
                if (q == (int)my_rank) w_own = wq;
            }
            {
                // (the tensor-memory loads are warp-wide: every lane takes part, whatever its own row's weight; a row without
                // weight in this slice, or a slice without tiles whose accumulator was never written, stages nothing)
                tc_fence_after();
                const uint32_t lane_addr_m = (uint32_t)((warp & 3) * 32) << 16;
                const bool mine = fin_l > 0.f && w_own > 0.f && fin_ok;
#pragma unroll 1
                for (int c = 0; c < HD / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr_m + kColO + c * 32, o);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            stage[(c * 8 + i) * 128 + row_m] = make_float4(__uint_as_float(o[4 * i]) * w_own, __uint_as_float(o[4 * i + 1]) * w_own,
                                                                           __uint_as_float(o[4 * i + 2]) * w_own, __uint_as_float(o[4 * i + 3]) * w_own);
                    }
                }
            }
        }
        cluster_arrive();
        cluster_wait();
        if (warp >= 2) {
            const int t_row_m = t0 + row_m / p.G;
            const int c4_per = HD / 4 / ns, c4_0 = (int)my_rank * c4_per;           // this CTA's columns, in float4 units
            if (t_row_m < p.T && l_all > 0.f) {
                const float inv = 1.f / l_all;
                __nv_bfloat16 *orow = (__nv_bfloat16 *)p.out + (((size_t)b * p.T + t_row_m) * p.Hq + kvh * p.G + row_m % p.G) * HD + c4_0 * 4;
#pragma unroll 1
                for (int c4 = 0; c4 < c4_per; c4 += 2) {                            // 8 columns = one 16-byte store at a time
                    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    for (int q = 0; q < ns; ++q) {
                        if (!((live_peers >> q) & 1u)) continue;
                        const uint32_t a = mapa(smem_u32(stage + (c4_0 + c4) * 128 + row_m), (uint32_t)q);
                        float4 v0, v1;
                        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v0.x), "=f"(v0.y), "=f"(v0.z), "=f"(v0.w) : "r"(a) : "memory");
                        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v1.x), "=f"(v1.y), "=f"(v1.z), "=f"(v1.w) : "r"(a + 128 * 16) : "memory");
                        acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
                        acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
                    }
                    uint4 v;
                    uint32_t *vv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(acc[2 * k] * inv, acc[2 * k + 1] * inv);
                        vv[k] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    *reinterpret_cast<uint4 *>(orow + c4 * 4) = v;
                }
            }
        }
        cluster_arrive();
        cluster_wait();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace reflex

#include "attn_tc2.cuh"

namespace reflex {

// ------------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ------------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            return nullptr;
        return (EncodeTiledFn)sym;
    }();
    return fn;
}

// rank-3 map over rows of [rows][Hkv][d] bf16, box = 64 rows x 1 head x 64 elements, 128-byte swizzle
bool make_kv_map(CUtensorMap *m, const void *ptr, uint64_t rows, int Hkv, int d)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)Hkv, rows};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)Hkv * d * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)kBN};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// rank-4 map over q [B][T][Hq][d], box = (64 elements, G heads, 128/G tokens, 1 stream): rows land as (token, head)
bool make_q_map(CUtensorMap *m, const void *ptr, int B, int T, int Hq, int d, int G)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)Hq, (cuuint64_t)T, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)Hq * d * 2, (cuuint64_t)T * Hq * d * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)(kBM / G), 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct MapCache {
    std::mutex mu;
    std::map<std::tuple<const void *, int, int, int, int, int>, CUtensorMap> maps;  // (ptr, kind, a, b, c, d)
    bool get(CUtensorMap *out, const void *ptr, int kind, int a, int b, int c, int d,
             bool (*make)(CUtensorMap *, const void *, int, int, int, int))
    {
        std::lock_guard<std::mutex> lk(mu);
        auto key = std::make_tuple(ptr, kind, a, b, c, d);
        auto it = maps.find(key);
        if (it != maps.end()) { *out = it->second; return true; }
        if (maps.size() > 8192) maps.clear();
        CUtensorMap m;
        if (!make(&m, ptr, a, b, c, d)) return false;
        maps[key] = m;
        *out = m;
        return true;
    }
};

MapCache &cache() { static MapCache c; return c; }

bool mk_slab(CUtensorMap *m, const void *ptr, int rows, int Hkv, int d, int) { return make_kv_map(m, ptr, (uint64_t)rows, Hkv, d); }
bool mk_q(CUtensorMap *m, const void *ptr, int BT /*B<<16|T not used*/, int Hq, int d, int G)
{
    return make_q_map(m, ptr, BT >> 16, BT & 0xFFFF, Hq, d, G);
}

template <int HD>
cudaError_t launch_t(const CUtensorMap *mq, const CUtensorMap *mk, const CUtensorMap *mv, const CUtensorMap *mkd,
                     const CUtensorMap *mvd, const TcParams &tp, dim3 grid, cudaStream_t st)
{
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        return cudaFuncSetAttribute(attn_tc_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TcSmem<HD>::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = TcSmem<HD>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // the key slices of a query tile merge inside a cluster
    attr[1].val.clusterDim.x = 1; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = (unsigned)tp.nsplit;
    cfg.attrs = attr;
    cfg.numAttrs = tp.cluster_merge ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_tc_kernel<HD>, *mq, *mk, *mv, *mkd, *mvd, tp);
    count_launch();
    return e;
}

template <int HD>
cudaError_t launch2_t(const CUtensorMap *mq, const CUtensorMap *mk, const CUtensorMap *mv, const CUtensorMap *mkd,
                      const CUtensorMap *mvd, const CUtensorMap *mo, const TcParams &tp, dim3 grid, cudaStream_t st)
{
    static std::atomic<unsigned long long> attr_set{0};
    cudaError_t e0 = once_per_device(attr_set, [] {
        return cudaFuncSetAttribute(attn_tc2_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Tc2Smem<HD>::TOTAL);
    });
    if (e0 != cudaSuccess) return e0;
    // programmatic stream serialisation: the grid may be scheduled while the preceding kernel drains; it waits
    // (griddepcontrol.wait) before it touches global memory
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kTc2Threads);
    cfg.dynamicSmemBytes = Tc2Smem<HD>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // a pair of CTAs, or all the pairs that merge their key slices
    attr[1].val.clusterDim.x = 2u * (unsigned)(tp.cluster_merge ? tp.nsplit : 1); attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_tc2_kernel<HD>, *mq, *mk, *mv, *mkd, *mvd, *mo, tp);
    count_launch();
    return e;
}

// how many clusters of `cluster_ctas` CTAs of the two-CTA kernel the device holds at once (asked once per shape; clusters
// of 8 fit only once or twice per GPC, far fewer than SMs / 8)
template <int HD>
int tc2_active_clusters_t(int cluster_ctas)
{
    static int cached_dev[64][9] = {};          // per device ordinal (modulo 64): the answer depends on the device
    if (cluster_ctas < 2 || cluster_ctas > 8) return 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    int *cached = cached_dev[dev & 63];
    if (cached[cluster_ctas] != 0) return cached[cluster_ctas] > 0 ? cached[cluster_ctas] : 0;
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cluster_ctas * 64u);
    cfg.blockDim = dim3(kTc2Threads);
    cfg.dynamicSmemBytes = Tc2Smem<HD>::TOTAL;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster_ctas; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaFuncSetAttribute(attn_tc2_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Tc2Smem<HD>::TOTAL);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, attn_tc2_kernel<HD>, &cfg);
    if (e != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    cached[cluster_ctas] = n > 0 ? n : -1;
    return n > 0 ? n : 0;
}

int tc2_active_clusters(int d, int cluster_ctas)
{
    return d == 256 ? tc2_active_clusters_t<256>(cluster_ctas) : d == 128 ? tc2_active_clusters_t<128>(cluster_ctas) : 0;
}

}  // namespace

// rank-2 map over a row-major bf16 matrix [rows][inner], box = box_rows x 64 elements, 128-byte swizzle (cached like the others)
bool tensor_map_2d_bf16(CUtensorMap *out, const void *ptr, int inner, int rows, int box_rows)
{
    return cache().get(out, ptr, 3, inner, rows, box_rows, 0, [](CUtensorMap *m, const void *p_, int inner_, int rows_, int box_rows_, int) -> bool {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return false;
        cuuint64_t dims[2] = {(cuuint64_t)inner_, (cuuint64_t)rows_};
        cuuint64_t strides[1] = {(cuuint64_t)inner_ * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)box_rows_};
        cuuint32_t es[2] = {1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(p_), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

bool tc_supported(const AttnParams &p)
{
    if (p.dtype != REFLEX_DTYPE_BF16) return false;
    if (!(p.d == 64 || p.d == 128 || p.d == 256)) return false;
    const int G = p.Hq / p.Hkv;
    if (G > kBM || (kBM % G) != 0) return false;
    if (p.B > 65535 || p.T > 65535) return false;
    if ((uint64_t)p.L * p.B * (uint64_t)(p.ring_off + p.N) > 0x7FFFFFFFull || (uint64_t)p.B * p.T > 0x7FFFFFFFull) return false;
    return encode_fn() != nullptr;
}

int tc_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count)
{
    const int G = p.Hq / p.Hkv;
    const int tile_tokens = kBM / G;
    const int n_qtiles = (p.T + tile_tokens - 1) / tile_tokens;
    const int ctas = n_qtiles * p.Hkv * p.B;
    const int n_tiles = (p.S_max + kBN - 1) / kBN + (p.N + kBN - 1) / kBN + (p.T + kBN - 1) / kBN;
    if (ctas >= sm_count) return 1;
    int want = (sm_count + ctas - 1) / ctas;

    if (want > n_tiles) want = n_tiles;
    if (want > kMaxSplits) want = kMaxSplits;
    const size_t per_split = (size_t)p.B * p.T * p.Hq * (p.d + 2) * sizeof(float);
    if (per_split > 0 && (size_t)want * per_split > partial_bytes) want = (int)(partial_bytes / per_split);
    // a power of two: measured (one stream, 15 key tiles) 15.5 us per layer with 8 slices and 16.5 with 4, against 18-21 us
    // with 5, 6, 7, 9, 10, 12 or 15 (the stride between a row's partials in the scratch area is then a power of two as well)
    int pow2 = 1;
    while (pow2 * 2 <= want) pow2 *= 2;
    return pow2;
}

bool tc2_supported(const AttnParams &p) { return tc_supported(p) && (p.d == 128 || p.d == 256); }

// Key split of the two-CTA kernel: 1, 2, 4 or 8 slices, whichever a small cost model makes cheapest. A unit (tile pair
// of one stream and KV head) walks its 128-key tiles at about 1.3 us each, units run in waves of one per SM pair, and
// splitting costs a fixed 3 us (merge launch) plus the fp32 partials' round trip through memory. Measured at the
// 898-key shape (before the partial tiles of a cluster's last unit were staged and written as whole rows, which took 1 us
// off the one-stream figure): 1 stream 14.4 us with 8 slices; 2 streams 15.4 with 4; 4 streams 17.5 with 4; 8 to 32 streams 19.5 to
// 21.7 unsplit (split in two: 21.6 to 40); at 4466 keys and 16 streams 41 us split in two, 51 unsplit, 47 in four.
// The nsplit pairs that share a tile pair can merge inside one cluster (no partials, no merge launch) when the cluster stays
// within the portable size of 8 CTAs, all clusters are resident at once with exactly one unit each, and a thread's share of
// the columns is whole 16-byte stores. Measured against the split with partials: 4466 keys, 16 streams 41.2 -> 35.6 us
// (two slices); 898 keys, 4 streams 18.5 -> 16.5 (four slices); one stream 15.5 merged in four against 14.4 with eight
// slices and the merge kernel, and 2 streams 16.5 merged in four against 15.9 with partials. The model therefore charges
// the in-cluster merge 5.5 us (three cluster barriers and the staged reduction keep every CTA of the cluster that long)
// and uses it only where the partials' round trip would cost more.
static constexpr double kTc2MergedUs = 5.5;
static double tc2_partials_us(const AttnParams &p, int nsplit)   // merge launch + fp32 partials written and read back
{
    const double per_split_bytes = (double)p.B * p.T * p.Hq * (p.d + 2) * sizeof(float);
    return 3.0 + 2.0 * per_split_bytes * nsplit / 3.4e6;
}
static bool tc2_cluster_merge_ok(const AttnParams &p, int nsplit, int sm_count)
{
    if (nsplit != 2 && nsplit != 4) return false;
    const int G = p.Hq / p.Hkv;
    const int tile_tokens = kBM / G;
    const int n_pairs = ((p.T + tile_tokens - 1) / tile_tokens + 1) / 2;
    const int base_units = n_pairs * p.Hkv * p.B;
    if (base_units * nsplit * 2 > sm_count) return false;
    // all clusters resident at once (a second wave would wait for whole clusters). Clusters of 8 get a margin: 16 of them,
    // the most the device reports, measured 20.4 us where 12 took 17.5 and the unsplit kernel 19.5.
    const int active = tc2_active_clusters(p.d, 2 * nsplit);
    if (base_units > (nsplit == 4 ? active - active / 4 : active)) return false;
    if (tc2_partials_us(p, nsplit) <= kTc2MergedUs) return false;
    return (p.d / nsplit / kTc2Parts) % 16 == 0 && p.d / nsplit / kTc2Parts >= 16;   // a thread reduces whole 16-column pieces
}

int tc2_choose_splits(const AttnParams &p, size_t partial_bytes, int sm_count)
{
    const int G = p.Hq / p.Hkv;
    const int tile_tokens = kBM / G;
    const int n_pairs = ((p.T + tile_tokens - 1) / tile_tokens + 1) / 2;
    const int units = n_pairs * p.Hkv * p.B;
    const int clusters = sm_count / 2 > 0 ? sm_count / 2 : 1;
    if (units >= clusters) return 1;
    const int halves = (p.S_max + kBN - 1) / kBN + (p.N + kBN - 1) / kBN + (p.T + kBN - 1) / kBN;
    const int tiles = (halves + 1) / 2;
    const double per_split_bytes = (double)p.B * p.T * p.Hq * (p.d + 2) * sizeof(float);
    int best = 1;
    double best_us = 1e30;
    for (int ns = 1; ns <= 8; ns *= 2) {
        if (ns > tiles) break;
        const bool merged = ns > 1 && tc2_cluster_merge_ok(p, ns, sm_count);
        if (ns > 1 && !merged && per_split_bytes * ns > (double)partial_bytes) break;
        const int waves = merged ? 1 : (units * ns + clusters - 1) / clusters;
        const double loop_us = 1.3 * waves * ((tiles + ns - 1) / ns);
        const double split_us = ns == 1 ? 0.0 : (merged ? kTc2MergedUs : tc2_partials_us(p, ns));
        if (loop_us + split_us < best_us - 0.05) { best_us = loop_us + split_us; best = ns; }
    }
    return best;
}

cudaError_t launch_attention_tc(const AttnParams &p, uint32_t *status, bool two_cta, int sm_count, cudaStream_t st)
{
    const int G = p.Hq / p.Hkv;
    const int rows_slab = p.L * p.B * (p.ring_off + p.N);
    CUtensorMap mk, mv, mkd, mvd, mq;
    if (!cache().get(&mk, p.k_slab, 0, rows_slab, p.Hkv, p.d, 0, mk_slab) || !cache().get(&mv, p.v_slab, 0, rows_slab, p.Hkv, p.d, 0, mk_slab) ||
        !cache().get(&mkd, p.k_dyn, 0, p.B * p.T, p.Hkv, p.d, 0, mk_slab) || !cache().get(&mvd, p.v_dyn, 0, p.B * p.T, p.Hkv, p.d, 0, mk_slab) ||
        !cache().get(&mq, p.q, 1, (p.B << 16) | p.T, p.Hq, p.d, G, mk_q))
        return cudaErrorInvalidValue;
    TcParams tp;
    tp.state = p.state; tp.out = p.out; tp.partials = p.partials; tp.status = status;
    tp.B = p.B; tp.L = p.L; tp.Hq = p.Hq; tp.Hkv = p.Hkv; tp.G = G; tp.S_max = p.S_max; tp.N = p.N; tp.T = p.T; tp.layer = p.layer;
    tp.ring_off = p.ring_off;
    tp.dyn_mask = p.dyn_mask; tp.scale = p.scale; tp.scale_log2 = p.scale * 1.4426950408889634f;
    tp.nsplit = p.nsplit;
    tp.tile_tokens = kBM / G;
    tp.live_rows = kBM;
    tp.n_qtiles = (p.T + tp.tile_tokens - 1) / tp.tile_tokens;
    tp.cluster_merge = two_cta ? (tc2_cluster_merge_ok(p, p.nsplit, sm_count) ? 1 : 0)
                               : ((p.nsplit > 1 && p.nsplit <= 8 && (p.d / 4) % (2 * p.nsplit) == 0) ? 1 : 0);
    cudaError_t e;
    if (two_cta) {
        // persistent grid: one cluster (two CTAs) per SM pair walks the (stream, KV head, tile pair) units;
        // an odd tile count leaves the last pair of a stream with one idle half
        CUtensorMap mo;
        if (!cache().get(&mo, p.out, 1, (p.B << 16) | p.T, p.Hq, p.d, G, mk_q)) return cudaErrorInvalidValue;
        tp.n_qtiles = (tp.n_qtiles + 1) / 2;
        // Key-split units that leave fp32 partials: every CTA writes its rows x head_dim x 4 bytes, and an SM's stores leave at
        // about 24 bytes per clock (128 KB: 2.8 us of a 10 us launch). While twice the clusters still fit the device at once,
        // a CTA takes half a tile's tokens (64 live rows of its 128) and the partials are shared by twice the SMs.
        if (p.nsplit > 1 && !tp.cluster_merge && tp.tile_tokens % 2 == 0) {
            const int half_tokens = tp.tile_tokens / 2;
            const int pairs_h = ((p.T + half_tokens - 1) / half_tokens + 1) / 2;
            if (pairs_h > tp.n_qtiles && pairs_h * p.Hkv * p.B * p.nsplit <= tc2_active_clusters(p.d, 2)) {
                tp.tile_tokens = half_tokens; tp.live_rows = kBM / 2; tp.n_qtiles = pairs_h;
            }
        }
        const int units = tp.n_qtiles * p.Hkv * p.B * p.nsplit;
        int clusters = sm_count / 2;
        if (clusters > units) clusters = units;
        if (clusters < 1) clusters = 1;
        dim3 grid2(2 * clusters, 1, 1);                      // with cluster_merge: units pairs = units / nsplit clusters of 2 * nsplit CTAs
        if (p.d == 256) e = launch2_t<256>(&mq, &mk, &mv, &mkd, &mvd, &mo, tp, grid2, st);
        else if (p.d == 128) e = launch2_t<128>(&mq, &mk, &mv, &mkd, &mvd, &mo, tp, grid2, st);
        else return cudaErrorInvalidValue;
        if (e != cudaSuccess || p.nsplit == 1 || tp.cluster_merge) return e;
        return launch_attention_merge(p, st);
    }
    dim3 grid(tp.n_qtiles * p.Hkv, p.B, p.nsplit);
    switch (p.d) {
        case 64: e = launch_t<64>(&mq, &mk, &mv, &mkd, &mvd, tp, grid, st); break;
        case 128: e = launch_t<128>(&mq, &mk, &mv, &mkd, &mvd, tp, grid, st); break;
        case 256: e = launch_t<256>(&mq, &mk, &mv, &mkd, &mvd, tp, grid, st); break;
        default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess || p.nsplit == 1 || tp.cluster_merge) return e;
    return launch_attention_merge(p, st);
}

}  // namespace reflex

#ifdef REFLEX_TRACE
extern "C" int reflex_debug_tc2_trace(long long *out)
{
    return (int)cudaMemcpyFromSymbol(out, reflex::g_tc2_trace, sizeof(long long) * 2 * 4 * 16 * 16);
}
#endif
