// Partitioned attention (Eq. 1), two-CTA persistent form, for batched serving.
//
// A cluster of two CTAs (two SMs) drives tcgen05.mma.cta_group::2 with M = 256: two 128-row query tiles of
// the same (stream, KV head). The B operand of such an MMA is split between the two CTAs' shared memories,
// so each CTA stages only HALF of every K tile (64 of its 128 keys) and HALF of every V tile (128 of the
// head_dim columns): the bytes each SM pulls per key are halved against the one-CTA kernel, which is what
// lets the loads keep up with the tensor pipe at head_dim 256.
//
// The grid is persistent: one cluster per SM pair walks a list of work units (stream, KV head, tile pair).
// Barrier, TMEM and cluster set-up is paid once, and the tail of a unit (last P V, normalisation, store of O)
// overlaps the head of the next one (its Q / K / V loads and first Q K^T).
//
// Per CTA:  warp 0      TMA producer (own Q tile, own K half, own V half)
//           warp 1      MMA issuer (leader CTA only): S = Q K^T (M256 N128), O += P V (M256 N=d)
//           warps 2..9  softmax over this CTA's 128 rows x 128 keys: two threads per row (64 keys each),
//                       P (bf16) into swizzled shared memory, lazy rescale of O in TMEM, and the epilogue:
//                       O / l staged through shared memory and written with TMA stores
// Barriers the leader's MMA thread waits on collect both CTAs (TMA completions through cta_group::2 loads,
// softmax arrivals through shared::cluster arrives); completions fan out with multicast commits.
// Included by attn_tc.cu (shares its tile geometry and tensor maps).
#pragma once

namespace reflex {

// Optional timeline of the first cluster (debug builds only: -DREFLEX_TRACE): clock64 stamps into the (otherwise
// unused) split-K partial area. Compiled out of the product library.
#ifdef REFLEX_TRACE
#define TC2_TRACE(role, slot, ev) do { if (blockIdx.x < 2 && (slot) < 16 && (ev) < 16) \
    reinterpret_cast<long long *>(p.partials)[((blockIdx.x * 4 + (role)) * 16 + (slot)) * 16 + (ev)] = clock64(); } while (0)
#else
#define TC2_TRACE(role, slot, ev) do { } while (0)
#endif

constexpr int kTc2Keys = 128;     // keys per tile = two 64-key halves, one per CTA of the pair
constexpr int kTc2Threads = 320;  // producer warp, MMA warp, eight softmax warps

template <int HD> struct Tc2Smem {
    static constexpr int CH = HD / 64;
    static constexpr int VCH = CH / 2;                          // this CTA's 64-column chunks of head_dim
    static constexpr uint32_t Q_BYTES = CH * 128 * 128;
    static constexpr uint32_t K_STAGE = CH * 64 * 128;          // 64 keys x head_dim
    static constexpr uint32_t V_STAGE = VCH * 128 * 128;        // 128 keys x head_dim/2
    static constexpr uint32_t V_HALF = VCH * 64 * 128;          // bytes one 64-key half contributes
    static constexpr uint32_t P_BYTES = 2 * 128 * 128;          // 128 rows x 128 keys bf16; also the staging area of the epilogue
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = OFF_Q + Q_BYTES;
    static constexpr uint32_t OFF_V = OFF_K + 2 * K_STAGE;
    static constexpr uint32_t OFF_P = OFF_V + 2 * V_STAGE;
    static constexpr uint32_t OFF_BAR = OFF_P + P_BYTES;
    static constexpr uint32_t OFF_XCH = OFF_BAR + 192;              // row max / row sum exchange between the two halves
    static constexpr uint32_t NEED = OFF_XCH + 2 * 2 * 128 * 4;     // bytes used from the 1024-byte aligned base
    static constexpr uint32_t TOTAL = 232448;                       // the whole opt-in shared memory of an SM (227 KB)
};

enum { C_QFULL = 0, C_QEMPTY = 1, C_KFULL = 2, C_KEMPTY = 4, C_VLAND = 6, C_VEMPTY = 8, C_SFULL = 10, C_SEMPTY = 12,
       C_PFULL = 14, C_PVDONE = 15, C_OFREE = 16, C_COUNT = 17 };

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}

template <int HD>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTc2Threads, 1)
attn_tc2_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kd,
                const __grid_constant__ CUtensorMap tm_vd, const __grid_constant__ CUtensorMap tm_o, const TcParams p)
{
    using L = Tc2Smem<HD>;
    constexpr int CH = L::CH, VCH = L::VCH;
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColO = 0, kColS = HD;  // O: HD fp32 columns; S: 2 x 128 columns
    static_assert(HD + 2 * kTc2Keys <= 512 && VCH >= 1, "TMEM budget / head_dim split");
    static_assert(8 * C_COUNT + 8 <= 192, "barrier area");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw_addr);
    const uint32_t bar0 = base + L::OFF_BAR;
    auto bar = [&](int i) -> uint32_t { return bar0 + 8u * (uint32_t)i; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L::OFF_BAR + 8 * C_COUNT);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    if ((base - raw_addr) + L::NEED > L::TOTAL) {
        // the dynamic shared-memory window starts too far from a 1024-byte boundary to hold the tiles: same for every
        // CTA of the launch, so all of them leave here, before any barrier, cluster or TMEM state exists
        if (threadIdx.x == 0) atomicCAS(p.status, 0u, 0x80000000u | (99u << 16));
        return;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 64) TC2_TRACE(2, 15, 0);
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int n_pairs = p.n_qtiles;                    // tile pairs per (stream, KV head)
    const int n_units = p.B * p.Hkv * n_pairs * p.nsplit;   // with nsplit > 1 a unit covers a slice of the key tiles

    // geometry of one work unit
    struct Unit { int b, kvh, t0, H, n_tiles, tile0, split; TileGeom g; };
    auto load_unit = [&](int u) -> Unit {
        Unit w;
        w.split = u % p.nsplit;
        const int uu = u / p.nsplit;
        const int pair = uu % n_pairs;
        w.kvh = (uu / n_pairs) % p.Hkv;
        w.b = uu / (n_pairs * p.Hkv);
        w.t0 = (2 * pair + (int)rank) * p.tile_tokens;
        const StreamState st = p.state[w.b];
        TileGeom &g = w.g;
        g.S = st.static_len > 0 ? st.static_len : 0;
        g.N = p.N; g.T = p.T; g.count = st.count;
        g.oldest = (st.head - st.count) % p.N;
        if (g.oldest < 0) g.oldest += p.N;
        g.ns = (g.S + kBN - 1) / kBN;
        g.nr = g.count > 0 ? (p.N + kBN - 1) / kBN : 0;
        g.nd = (p.T + kBN - 1) / kBN;
        g.row_base = (p.layer * p.B + w.b) * (p.S_max + p.N);
        g.S_max = p.S_max; g.b = w.b;
        w.H = g.ns + g.nr + g.nd;          // 64-key halves
        const int all_tiles = (w.H + 1) / 2;   // >= 1: there is always a dynamic half
        const int per = (all_tiles + p.nsplit - 1) / p.nsplit;
        w.tile0 = w.split * per;               // this unit's slice of the key tiles (may be empty for the last splits)
        w.n_tiles = max(0, min(all_tiles, w.tile0 + per) - w.tile0);
        return w;
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < C_COUNT; ++i) {
            const bool both = (i == C_SEMPTY || i == C_SEMPTY + 1 || i == C_PFULL || i == C_OFREE);
            mbar_init(bar(i), both ? 16u : 1u);   // "both": one arrival per softmax warp of either CTA
        }
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v); prefetch_tmap(&tm_kd); prefetch_tmap(&tm_vd); prefetch_tmap(&tm_o);
    }
    if (warp == 1) tmem_alloc2(smem_u32((const void *)tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // both CTAs' barriers are initialised before anything crosses the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 64) TC2_TRACE(2, 15, 1);

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
        atomicCAS(p.status, 0u, 0x80000000u | ((code + 32u) << 16) | (blockIdx.x & 0xFFFFu));
        return false;
    };

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            bool ok = true;
            int gt = 0, ui = 0;
            for (int u = cluster_id; u < n_units && ok; u += n_clusters, ++ui) {
                const Unit w = load_unit(u);
                if (w.n_tiles == 0) { --ui; continue; }   // an empty key slice: every role skips it the same way
                for (int jj = 0; jj < w.n_tiles && ok; ++jj) {
                    const int gi = gt + jj, st = gi & 1;
                    const uint32_t ph = (uint32_t)((gi >> 1) - 1) & 1u;
                    const int h0 = 2 * (w.tile0 + jj), h1 = h0 + 1;
                    const int live = (h0 < w.H ? 1 : 0) + (h1 < w.H ? 1 : 0);
                    if (gi >= 2) ok = wait(C_KEMPTY + st, ph, 1);
                    if (!ok) break;
                    if (rank == 0) mbar_expect_tx(bar(C_KFULL + st), (uint32_t)live * L::K_STAGE);
                    const int myh = h0 + (int)rank;
                    if (myh < w.H) {
                        const TileRef tr = w.g.decode(myh);
                        for (int c = 0; c < CH; ++c)
                            tma2_load_3d(base + L::OFF_K + st * L::K_STAGE + c * (64 * 128), tr.dyn ? &tm_kd : &tm_k,
                                         bar(C_KFULL + st) & kPeerBitMask, c * 64, w.kvh, tr.row0);
                    }
                    if (jj == 0) {
                        // this unit's Q tile, once the last Q K^T of the previous unit has drained the buffer
                        if (ui >= 1) ok = wait(C_QEMPTY, (uint32_t)(ui - 1) & 1u, 14);
                        if (!ok) break;
                        if (rank == 0) mbar_expect_tx(bar(C_QFULL), 2 * L::Q_BYTES);
                        for (int c = 0; c < CH; ++c)
                            tma2_load_4d(base + L::OFF_Q + c * (128 * 128), &tm_q, bar(C_QFULL) & kPeerBitMask, c * 64, w.kvh * p.G, w.t0, w.b);
                    }
                    if (gi >= 2) ok = wait(C_VEMPTY + st, ph, 2);
                    if (!ok) break;
                    mbar_expect_tx(bar(C_VLAND + st), (uint32_t)live * L::V_HALF);
                    for (int hh = h0; hh <= h1; ++hh) {
                        if (hh >= w.H) break;
                        const TileRef tr = w.g.decode(hh);
                        for (int c = 0; c < VCH; ++c)
                            tma_load_3d(base + L::OFF_V + st * L::V_STAGE + c * (128 * 128) + (hh & 1) * (64 * 128), tr.dyn ? &tm_vd : &tm_v,
                                        bar(C_VLAND + st), ((int)rank * VCH + c) * 64, w.kvh, tr.row0);
                    }
                }
                gt += w.n_tiles;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA) ----------------
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(256, kTc2Keys, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(256, HD, true);
            auto issue_qk = [&](int gi, bool last_of_unit) {
                const int st = gi & 1, buf = gi & 1;
                const uint32_t d_tmem = tmem_base + kColS + buf * kTc2Keys;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t a = base + L::OFF_Q + (kk >> 2) * (128 * 128) + (kk & 3) * 32;
                    const uint32_t bb = base + L::OFF_K + st * L::K_STAGE + (kk >> 2) * (64 * 128) + (kk & 3) * 32;
                    umma2_ss(d_tmem, umma_desc_sw128(a, 16, 1024), umma_desc_sw128(bb, 16, 1024), idesc_qk, kk > 0 ? 1u : 0u);
                }
                umma2_commit_mc(bar(C_KEMPTY + st), 3);
                umma2_commit_mc(bar(C_SFULL + buf), 3);
                if (last_of_unit) umma2_commit_mc(bar(C_QEMPTY), 3);   // Q has been read for the last time
            };
            // wait for the K tile and the S buffer of global tile gi, then issue its Q K^T
            auto qk_when_ready = [&](int gi, bool last_of_unit) -> bool {
                bool ok2 = wait(C_KFULL + (gi & 1), (uint32_t)(gi >> 1) & 1u, 5);
                if (ok2 && gi >= 2) ok2 = wait(C_SEMPTY + (gi & 1), (uint32_t)((gi >> 1) - 1) & 1u, 6);
                if (!ok2) return false;
                tc_fence_after();
                issue_qk(gi, last_of_unit);
                return true;
            };
            // Q K^T of tile jj+1 is issued before waiting for P(jj): S is double buffered in TMEM, so the tensor pipe works
            // on the next tile's logits while the softmax threads finish this tile. (Issuing Q K^T two tiles ahead, or in
            // whichever order inputs arrive, was measured and is slower: with two K stages the extra Q K^T lands in front
            // of a P V that the softmax threads are waiting for.)
            bool ok = true;
            int gt = 0, ui = 0;
            for (int u = cluster_id; u < n_units && ok; u += n_clusters, ++ui) {
                const Unit w = load_unit(u);
                const int n = w.n_tiles;
                if (n == 0) { --ui; continue; }
                ok = wait(C_QFULL, (uint32_t)ui & 1u, 3) && qk_when_ready(gt, n == 1);
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int gi = gt + jj;
                    const int st = gi & 1;
                    if (jj + 1 < n) {
                        ok = qk_when_ready(gi + 1, jj + 2 == n);
                        if (!ok) break;
                    }
                    ok = wait(C_PFULL, (uint32_t)gi & 1u, 8);   // both CTAs: P written, V landed and cleaned
                    if (ok && jj == 0 && ui >= 1) ok = wait(C_OFREE, (uint32_t)(ui - 1) & 1u, 15);   // previous O has been read out
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < kTc2Keys / 16; ++kk) {
                        const uint32_t a = base + L::OFF_P + (kk >> 2) * (128 * 128) + (kk & 3) * 32;
                        const uint32_t bb = base + L::OFF_V + st * L::V_STAGE + kk * (16 * 128);
                        umma2_ss(tmem_base + kColO, umma_desc_sw128(a, 16, 1024), umma_desc_sw128(bb, 128 * 128, 1024), idesc_pv,
                                 (jj > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma2_commit_mc(bar(C_VEMPTY + st), 3);
                    umma2_commit_mc(bar(C_PVDONE), 3);
                }
                gt += n;
            }
        }
    } else {
        // ---------------- softmax / correction / epilogue (both CTAs) ----------------
        // Eight warps: two threads per query row, one per 64-key half of the tile (warps 2..5 take the pair
        // leader's keys, warps 6..9 the partner's). The halves meet once per tile to agree on the row maximum.
        // A wait that ran out never leaves these loops: every softmax warp keeps meeting the others at the named
        // barrier (the remaining waits return at once), so no warp is left behind.
        const int sw = warp - 2;
        const int half = sw >> 2;                 // which 64 columns of S / 64-key chunk of P / half of O's columns
        const int quarter = warp & 3;             // TMEM lane quarter this warp may touch
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const uint32_t leader_pfull = mapa(bar(C_PFULL), 0);
        const uint32_t leader_ofree = mapa(bar(C_OFREE), 0);
        float *exch = reinterpret_cast<float *>(smem + L::OFF_XCH);   // [2 buffers][2 halves][128 rows]
        bool ok = true;
        int gt = 0;
        [[maybe_unused]] int ui_s = 0;
        for (int u = cluster_id; u < n_units; u += n_clusters, ++ui_s) {
            const Unit w = load_unit(u);
            const int t_row = w.t0 + row / p.G;
            if (threadIdx.x == 64) TC2_TRACE(2, ui_s, 0);
            const int rows_total = p.T * p.Hq;
            const size_t n_slots = (size_t)p.B * rows_total * p.nsplit;
            float *pml = nullptr;    // this row's (m, l) slot when the keys are split over several units
            if (p.nsplit > 1 && t_row < p.T)
                pml = partial_ml(p.partials, n_slots, partial_slot(w.b, rows_total, t_row * p.Hq + w.kvh * p.G + row % p.G, p.nsplit, w.split), HD);
            if (w.n_tiles == 0) {
                if (pml && half == 0) { pml[0] = -INFINITY; pml[1] = 0.f; }   // an empty key slice contributes nothing
                continue;
            }
            float m_ref = -INFINITY, l = 0.f;
            for (int jj = 0; jj < w.n_tiles; ++jj) {
                const int gi = gt + jj, buf = gi & 1, st = gi & 1;
                const int h = 2 * (w.tile0 + jj) + half;
                uint64_t tmask = 0ull, rmask = 0ull;
                if (h < w.H) {
                    const TileRef tr = w.g.decode(h);
                    tmask = w.g.tile_mask(tr);
                    rmask = tmask;
                    if (tr.kind == 2 && p.dyn_mask) {
                        const int lim = t_row - tr.idx * kBN;
                        rmask &= (lim < 0) ? 0ull : (lim >= 63 ? ~0ull : ((2ull << lim) - 1ull));
                    }
                }
#define SM_EV(ev) do { if (threadIdx.x == 64 && ui_s == 0) TC2_TRACE(3, jj, ev); } while (0)
                SM_EV(0);
                ok = ok && wait(C_SFULL + buf, (uint32_t)(gi >> 1) & 1u, 9);
                SM_EV(1);
                if (threadIdx.x == 64 && jj == 0) TC2_TRACE(2, ui_s, 1);
                tc_fence_after();
                float s[64];
                {
                    const uint32_t s_addr = tmem_base + lane_addr + kColS + buf * kTc2Keys + half * 64;
                    uint32_t r0[32], r1[32];
                    tmem_ld32(s_addr, r0); tmem_ld32(s_addr + 32, r1);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) { s[c] = __uint_as_float(r0[c]); s[32 + c] = __uint_as_float(r1[c]); }
                }
                SM_EV(2);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(mapa(bar(C_SEMPTY + buf), 0));
                if (tmask != ~0ull) {
                    // dead keys get weight 0, but 0 x (stale NaN/Inf bytes) would still poison O: clear their V rows as soon
                    // as this CTA's V half has landed (long before the P V that reads them)
                    ok = ok && wait(C_VLAND + st, (uint32_t)(gi >> 1) & 1u, 12);
                    if (row < 64 && !((tmask >> row) & 1ull)) {
#pragma unroll
                        for (int c = 0; c < VCH; ++c) {
                            uint4 *vr = reinterpret_cast<uint4 *>(smem + L::OFF_V + st * L::V_STAGE + c * (128 * 128) + (half * 64 + row) * 128);
#pragma unroll
                            for (int i = 0; i < 8; ++i) vr[i] = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                if (rmask != ~0ull) apply_key_mask(s, rmask);
                float mx4[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
                for (int c = 4; c < 64; c += 4) {
                    mx4[0] = fmaxf(mx4[0], s[c]); mx4[1] = fmaxf(mx4[1], s[c + 1]);
                    mx4[2] = fmaxf(mx4[2], s[c + 2]); mx4[3] = fmaxf(mx4[3], s[c + 3]);
                }
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                // meet the thread that holds the other 64 keys of this row (thread 64 first makes sure that the TMA stores of
                // the previous unit have read the staging area, which is the P buffer every thread writes after this barrier)
                SM_EV(3);
                exch[(buf * 2 + half) * 128 + row] = mx;
                if (jj == 0 && threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                asm volatile("bar.sync 1, 256;" ::: "memory");
                SM_EV(4);
                mx = fmaxf(mx, exch[(buf * 2 + (half ^ 1)) * 128 + row]);
                bool pv_waited = false;
                if (jj == 0) {
                    m_ref = mx;
                } else {
                    const bool grow = (mx - m_ref) * p.scale_log2 > kRescaleThreshold;
                    if (__any_sync(0xffffffffu, grow)) {
                        // O (and l) were accumulated against m_ref: bring them to the new reference before this tile's P V.
                        // Both threads of a row see the same mx, so they decide alike; each rescales its half of O's columns.
                        const float alpha = grow ? ex2((m_ref - mx) * p.scale_log2) : 1.f;
                        if (grow) m_ref = mx;
                        l *= alpha;
                        ok = ok && wait(C_PVDONE, (uint32_t)(gi - 1) & 1u, 10);
                        pv_waited = true;
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < HD / 64; ++c) {
                            uint32_t o[32];
                            const uint32_t o_addr = tmem_base + lane_addr + kColO + half * (HD / 2) + c * 32;
                            tmem_ld32(o_addr, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st32(o_addr, o);
                        }
                        tmem_wait_st();
                    }
                }
                const float mr = (m_ref == -INFINITY) ? 0.f : m_ref * p.scale_log2;
                float sum4[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t packed[32];
#pragma unroll
                for (int c = 0; c < 64; c += 2) {
                    // P = 2^(s*scale*log2e - m). One pair in four takes the FMA-pipe exponential so the MUFU unit and the
                    // FMA pipe share the load.
                    const float x0 = fmaf(s[c], p.scale_log2, -mr), x1 = fmaf(s[c + 1], p.scale_log2, -mr);
                    const bool on_fma = ((c >> 1) & 3) == 3;
                    const float p0 = on_fma ? ex2_fma(x0) : ex2(x0);
                    const float p1 = on_fma ? ex2_fma(x1) : ex2(x1);
                    sum4[(c >> 1) & 3] += p0 + p1;
                    __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                    packed[c >> 1] = *reinterpret_cast<uint32_t *>(&hh);
                }
                l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
                SM_EV(5);
                if (gi >= 1 && !pv_waited)
                    ok = ok && wait(C_PVDONE, (uint32_t)(gi - 1) & 1u, 11);  // the single P buffer was read by the previous P V
                SM_EV(6);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint8_t *dst = smem + L::OFF_P + half * (128 * 128) + row * 128 + ((c ^ (row & 7)) << 4);
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                }
                SM_EV(7);
                // the arrive below also tells the leader that this CTA's V half is in place
                if (tmask == ~0ull) ok = ok && wait(C_VLAND + st, (uint32_t)(gi >> 1) & 1u, 12);
                SM_EV(8);
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_pfull);
                SM_EV(9);
            }
            gt += w.n_tiles;
            // ---- epilogue of the unit ----
            // The two threads of a row add their sums; each thread normalises its half of the head_dim columns, 64 at a
            // time, into the (now idle) P buffer laid out like a Q tile, and one thread hands the tile to TMA stores.
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 2); TC2_TRACE(2, ui_s, 2); }
            const int g_last = gt - 1;
            ok = ok && wait(C_PVDONE, (uint32_t)g_last & 1u, 13);
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 3); TC2_TRACE(2, ui_s, 3); }
            const int xb = (g_last + 1) & 1;
            exch[(xb * 2 + half) * 128 + row] = l;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            l += exch[(xb * 2 + (half ^ 1)) * 128 + row];
            tc_fence_after();
            if (p.nsplit > 1) {
                // key-split unit: leave (m, l, unnormalised O) for the merge kernel; m in natural-log units like the other
                // kernels. O goes out 32 columns per thread at a time through the idle P buffer (fp32, swizzled 128-byte
                // rows), so that the global stores are whole 128-byte row segments instead of one scattered row per lane.
                if (pml && half == 0) { pml[0] = (m_ref == -INFINITY) ? -INFINITY : m_ref * p.scale; pml[1] = l; }
#pragma unroll 1
                for (int sub = 0; sub < HD / 64; ++sub) {
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + half * (HD / 2) + sub * 32, o);
                    tmem_wait_ld();
                    if (sub == HD / 64 - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(leader_ofree);
                    }
                    uint8_t *srow = smem + L::OFF_P + half * (128 * 128) + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    const int tid = threadIdx.x - 64;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int idx = it * 256 + tid;
                        const int hh = idx >> 10, rr = (idx >> 3) & 127, cc = idx & 7;
                        const int tt = w.t0 + rr / p.G;
                        if (tt < p.T) {
                            const uint4 v = *reinterpret_cast<const uint4 *>(smem + L::OFF_P + hh * (128 * 128) + rr * 128 + ((cc ^ (rr & 7)) << 4));
                            float *dst = partial_o(p.partials, partial_slot(w.b, rows_total, tt * p.Hq + w.kvh * p.G + rr % p.G, p.nsplit, w.split), HD) +
                                         hh * (HD / 2) + sub * 32 + cc * 4;
                            *reinterpret_cast<uint4 *>(dst) = v;
                        }
                    }
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
                continue;
            }
            const float inv = 1.f / l;
            const bool store_unit = w.t0 < p.T;   // an idle partner tile (odd tile count) has nothing to write
#pragma unroll 1
            for (int rnd = 0; rnd < HD / 128; ++rnd) {
                uint32_t o0[32], o1[32];
                const uint32_t o_addr = tmem_base + lane_addr + kColO + half * (HD / 2) + rnd * 64;
                tmem_ld32(o_addr, o0); tmem_ld32(o_addr + 32, o1);
                tmem_wait_ld();
                if (rnd == HD / 128 - 1) {
                    // all of O is in registers: the next unit's first P V may overwrite the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_ofree);
                }
                uint8_t *srow = smem + L::OFF_P + half * (128 * 128) + row * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t *src = (c < 4) ? (o0 + 8 * c) : (o1 + 8 * (c - 4));
                    uint4 v;
                    uint32_t *vv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(src[2 * k]) * inv, __uint_as_float(src[2 * k + 1]) * inv);
                        vv[k] = *reinterpret_cast<uint32_t *>(&hh);
                    }
                    *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) = v;
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (threadIdx.x == 64) {
                    if (store_unit) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
                            tma_store_4d(&tm_o, base + L::OFF_P + hh * (128 * 128), hh * (HD / 2) + rnd * 64, w.kvh * p.G, w.t0, w.b);
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    // before the staging area is rewritten the store must have read it: at once between rounds, but after
                    // the last round only when the next unit is about to write P (see the top of the tile loop)
                    if (rnd + 1 < HD / 128) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                if (rnd + 1 < HD / 128) asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 4); TC2_TRACE(2, ui_s, 4); }
        }
        if (threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores of this CTA are complete
    }

    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // neither CTA retires while its partner can still touch its shared memory or barriers
    if (warp == 1) tmem_dealloc2(tmem_base, kTmemCols);
    if (threadIdx.x == 64) TC2_TRACE(2, 15, 5);
}

}  // namespace reflex
