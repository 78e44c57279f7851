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
//           warps 2..   softmax over this CTA's 128 rows x 128 keys: NP threads per row (128 / NP keys each),
//                       P (bf16) written back into tensor memory over the logits it came from, lazy rescale
//                       of O in tensor memory, and the epilogue: O / l through a 32 KB staging area and TMA stores
// P never touches shared memory: P V takes its A operand from tensor memory. With head_dim 256 the Q K^T
// MMAs alone read shared memory at its full bandwidth (a 4 KB slice of Q plus 4 KB of K per 64-cycle
// instruction), so every byte of shared-memory traffic that is not an operand read or a TMA fill stretches
// the tensor pipe; the 32 KB a P buffer would take pays for a third V stage instead.
// Barriers the leader's MMA thread waits on collect both CTAs (TMA completions through cta_group::2 loads,
// softmax arrivals through shared::cluster arrives); completions fan out with multicast commits.
// Included by attn_tc.cu (shares its tile geometry and tensor maps).
#pragma once
#include <type_traits>

namespace reflex {

// Optional timeline of the first cluster (debug builds only: -DREFLEX_TRACE): clock64 stamps into a device array that
// reflex_debug_tc2_trace() copies out. Compiled out of the product library.
#ifdef REFLEX_TRACE
__device__ long long g_tc2_trace[2 * 4 * 16 * 16];
#define TC2_TRACE(role, slot, ev) do { if (blockIdx.x < 2 && (slot) < 16 && (ev) < 16) \
    g_tc2_trace[((blockIdx.x * 4 + (role)) * 16 + (slot)) * 16 + (ev)] = clock64(); } while (0)
#else
#define TC2_TRACE(role, slot, ev) do { } while (0)
#endif
#ifndef REFLEX_TRACE_UNIT
#define REFLEX_TRACE_UNIT 0     // which unit of the cluster the per-tile stamps are taken in
#endif

constexpr int kTc2Keys = 128;     // keys per tile = two 64-key halves, one per CTA of the pair
#ifndef REFLEX_TC2_NP
#define REFLEX_TC2_NP 2
#endif
#ifndef REFLEX_TC2_POLY
#define REFLEX_TC2_POLY 2
#endif
constexpr int kTc2PolyEighths = REFLEX_TC2_POLY;   // of every 8 key pairs, how many take their exponentials on the FMA pipe
constexpr int kTc2Parts = REFLEX_TC2_NP;            // softmax threads per query row (2 or 4)
constexpr int kTc2Threads = 64 + 128 * kTc2Parts;   // producer warp, MMA warp, 4 * kTc2Parts softmax warps
static_assert(kTc2Parts == 2 || kTc2Parts == 4, "softmax threads per row");

// s[c] = -inf for every key c < K of a slice that `mask` marks dead
template <int K>
__device__ __forceinline__ void apply_slice_mask(float (&s)[K], uint64_t mask)
{
    const uint32_t lo = (uint32_t)mask, hi = (uint32_t)(mask >> 32);
#pragma unroll
    for (int c = 0; c < K; ++c) {
        const uint32_t w = c < 32 ? lo : hi;
        if (!(w & (1u << (c & 31)))) s[c] = -INFINITY;
    }
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}

template <int HD> struct Tc2Smem {
    static constexpr int CH = HD / 64;
    static constexpr int VCH = CH / 2;                          // this CTA's 64-column chunks of head_dim
    static constexpr int NKS = (HD == 256) ? 2 : 4;             // K stages
    static constexpr int NVS = (HD == 256) ? 2 : 4;             // V stages (P lives in tensor memory, which pays for the third)
    static constexpr uint32_t Q_BYTES = CH * 128 * 128;
    static constexpr uint32_t K_STAGE = CH * 64 * 128;          // 64 keys x head_dim
    static constexpr uint32_t V_STAGE = VCH * 128 * 128;        // 128 keys x head_dim/2
    static constexpr uint32_t V_HALF = VCH * 64 * 128;          // bytes one 64-key half contributes
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = OFF_Q + Q_BYTES;
    static constexpr uint32_t OFF_V = OFF_K + NKS * K_STAGE;
    static constexpr uint32_t OFF_STAGE = OFF_V + NVS * V_STAGE;      // epilogue staging: 128 rows x 128 columns of O in bf16
    static constexpr uint32_t STAGE_BYTES = 2 * 128 * 128;
    static constexpr uint32_t OFF_BAR = OFF_STAGE + STAGE_BYTES;
    static constexpr uint32_t BAR_BYTES = 256;
    // Row maxima of the NP threads of a row: 2 buffers (one per S/P buffer) x 128 rows x NP fp32, exact (rounded to 16 bits
    // the common reference overshot the true maximum by up to |max| / 128, which empties a row by underflow once logits
    // reach tens of thousands). The row sums exchanged at the end of a unit (NP x 128 fp32: one buffer's size) use the
    // buffer the unit's last tile did NOT use: every thread is past its last read of it, and the next tile writes to it
    // only after the barriers of the epilogue, which every thread reaches after it has read the sums.
    static constexpr uint32_t OFF_XMAX = OFF_BAR + BAR_BYTES;
    static constexpr uint32_t XBUF_BYTES = 128 * kTc2Parts * 4;
    static constexpr uint32_t XMAX_BYTES = 2 * XBUF_BYTES;
    static constexpr uint32_t TOTAL = 232448;                                   // the whole opt-in shared memory of an SM (227 KB)
    static constexpr uint32_t NEED = OFF_XMAX + XMAX_BYTES;                     // from the 1024-byte aligned base
    static_assert(NEED <= TOTAL, "shared memory budget");
    // mbarrier indices
    static constexpr int C_QFULL = 0, C_QEMPTY = 1, C_KFULL = 2, C_KEMPTY = C_KFULL + NKS, C_VLAND = C_KEMPTY + NKS,
                         C_VEMPTY = C_VLAND + NVS, C_SFULL = C_VEMPTY + NVS, C_PFULL = C_SFULL + 2, C_PVDONE = C_PFULL + 2,
                         C_OFREE = C_PVDONE + 2, C_COUNT = C_OFREE + 1;   // P V completion: one barrier per S/P buffer
    static_assert(8 * C_COUNT + 8 <= BAR_BYTES, "barrier area");
};

// (18 warps are five on at least one of the four schedulers, whose 16 K registers then allow 96 per thread)
template <int HD>
__global__ void __launch_bounds__(kTc2Threads, 1)   // launched as clusters of 2 CTAs, or of 2 * nsplit (cluster_merge)
attn_tc2_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kd,
                const __grid_constant__ CUtensorMap tm_vd, const __grid_constant__ CUtensorMap tm_o, const TcParams p)
{
    using L = Tc2Smem<HD>;
    constexpr int CH = L::CH, VCH = L::VCH, NKS = L::NKS, NVS = L::NVS;
    constexpr int C_QFULL = L::C_QFULL, C_QEMPTY = L::C_QEMPTY, C_KFULL = L::C_KFULL, C_KEMPTY = L::C_KEMPTY, C_VLAND = L::C_VLAND,
                  C_VEMPTY = L::C_VEMPTY, C_SFULL = L::C_SFULL, C_PFULL = L::C_PFULL, C_PVDONE = L::C_PVDONE, C_OFREE = L::C_OFREE,
                  C_COUNT = L::C_COUNT;
    constexpr uint32_t kTmemCols = 512;
    // O: HD fp32 columns. S: 2 x 128 fp32 columns; P(j) (bf16, two keys per column) overwrites the first 64 columns of
    // S(j)'s buffer once every thread of the row has taken its logits out, and is the A operand of P V from there.
    constexpr uint32_t kColO = 0, kColS = HD;
    static_assert(HD + 2 * kTc2Keys <= 512 && VCH >= 1, "TMEM budget / head_dim split");

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
    // A pair of CTAs (cluster ranks 2k, 2k+1) drives the cta_group::2 MMAs. Normally the cluster is one pair and walks a
    // list of units; with cluster_merge the cluster holds the nsplit pairs that share one query tile pair, each taking a
    // slice of the keys, and merges their (m, l, O) through distributed shared memory at the end (one unit per cluster).
    const uint32_t crank = cluster_ctarank();
    const uint32_t rank = crank & 1u, lead = crank & ~1u;      // rank inside the pair; cluster rank of the pair's leader
    const uint16_t pair_mask = (uint16_t)(3u << lead);         // both CTAs of this pair, for multicast commits
    const int pairs_per_cluster = p.cluster_merge ? p.nsplit : 1;
    const int cluster_id = blockIdx.x / (2 * pairs_per_cluster);
    const int n_clusters = gridDim.x / (2 * pairs_per_cluster);
    const int n_pairs = p.n_qtiles;                    // tile pairs per (stream, KV head)
    const int n_units = p.B * p.Hkv * n_pairs * p.nsplit;   // with nsplit > 1 a unit covers a slice of the key tiles
    // this pair's first unit and the stride to its next one
    const int u_start = p.cluster_merge ? cluster_id * p.nsplit + (int)(crank >> 1) : cluster_id;
    const int u_stride = p.cluster_merge ? n_units : n_clusters;

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
        g.row_base = (p.layer * p.B + w.b) * (p.ring_off + p.N);
        g.s_off = st.bank * p.S_max; g.ring_off = p.ring_off; g.b = w.b;
        w.H = g.ns + g.nr + g.nd;          // 64-key halves
        const int all_tiles = (w.H + 1) / 2;   // >= 1: there is always a dynamic half
        const int per = (all_tiles + p.nsplit - 1) / p.nsplit;
        w.tile0 = w.split * per;               // this unit's slice of the key tiles (may be empty for the last splits)
        w.n_tiles = max(0, min(all_tiles, w.tile0 + per) - w.tile0);
        return w;
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < C_COUNT; ++i) {
            const bool both = (i == C_PFULL || i == C_PFULL + 1 || i == C_OFREE);
            mbar_init(bar(i), both ? (uint32_t)(8 * kTc2Parts) : 1u);   // "both": one arrival per softmax warp of either CTA
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
    // Programmatic dependent launch: this grid may have been scheduled while the kernel ahead of it on the stream was still
    // running (its set-up above touches no global memory); from here on everything that kernel wrote is visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");

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

    // what a softmax thread carries into the in-cluster merge: its row's reference maximum (log2 units) and sum
    float fin_m = -INFINITY, fin_l = 0.f;
    bool fin_ok = true;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (lane == 0) {
            // The loads are issued in the order in which the tensor pipe frees their stages. The MMA warp issues
            // Q K^T(j+1) before P V(j), so the completions come as QK(0) QK(1) PV(0) QK(2) PV(1) ...: K(g) may go once
            // QK(g - NKS) is done (position 2(g-NKS)-1 in that sequence), V(g) once PV(g - NVS) is done (position
            // 2(g-NVS)+2). A K cursor therefore runs kLead = NKS - NVS + 1 tiles ahead of a V cursor through the same
            // list of units, and neither load waits behind a stage that frees later than its own.
            constexpr int kLead = NKS - NVS + 1;
            static_assert(kLead == 0 || kLead == 1, "order of K and V loads");
            struct Cursor { int u, ui, jj, g; bool valid; Unit w; };
            auto settle = [&](Cursor &c) {   // first unit at or after c.u with a non-empty key slice
                c.valid = false;
                for (; c.u < n_units; c.u += u_stride) {
                    c.w = load_unit(c.u);
                    if (c.w.n_tiles > 0) { c.valid = true; c.jj = 0; return; }
                }
            };
            auto advance = [&](Cursor &c) {
                ++c.g;
                if (++c.jj == c.w.n_tiles) { c.u += u_stride; ++c.ui; settle(c); }
            };
            bool ok = true;
            auto issue_k = [&](const Cursor &c) {
                const Unit &w = c.w;
                const int gi = c.g, st = gi % NKS;
                const uint32_t ph = (uint32_t)(gi / NKS - 1) & 1u;
                const int h0 = 2 * (w.tile0 + c.jj), h1 = h0 + 1;
                const int live = (h0 < w.H ? 1 : 0) + (h1 < w.H ? 1 : 0);
                if (c.ui == REFLEX_TRACE_UNIT) TC2_TRACE(0, c.jj, 0);
                if (gi >= NKS) ok = wait(C_KEMPTY + st, ph, 1);
                if (!ok) return;
                if (c.ui == REFLEX_TRACE_UNIT) TC2_TRACE(0, c.jj, 1);
                if (rank == 0) mbar_expect_tx(bar(C_KFULL + st), (uint32_t)live * L::K_STAGE);
                const int myh = h0 + (int)rank;
                if (myh < w.H) {
                    const TileRef tr = w.g.decode(myh);
                    for (int ch = 0; ch < CH; ++ch)
                        tma2_load_3d(base + L::OFF_K + st * L::K_STAGE + ch * (64 * 128), tr.dyn ? &tm_kd : &tm_k,
                                     bar(C_KFULL + st) & kPeerBitMask, ch * 64, w.kvh, tr.row0);
                }
            };
            auto issue_q = [&](const Cursor &c) {
                // a unit's Q tile, once the last Q K^T of the previous unit has drained the buffer
                const Unit &w = c.w;
                if (c.ui >= 1) ok = wait(C_QEMPTY, (uint32_t)(c.ui - 1) & 1u, 14);
                if (!ok) return;
                if (rank == 0) mbar_expect_tx(bar(C_QFULL), 2 * L::Q_BYTES);
                for (int ch = 0; ch < CH; ++ch)
                    tma2_load_4d(base + L::OFF_Q + ch * (128 * 128), &tm_q, bar(C_QFULL) & kPeerBitMask, ch * 64, w.kvh * p.G, w.t0, w.b);
            };
            auto issue_v = [&](const Cursor &c) {
                const Unit &w = c.w;
                const int gi = c.g, st = gi % NVS;
                const uint32_t ph = (uint32_t)(gi / NVS - 1) & 1u;
                const int h0 = 2 * (w.tile0 + c.jj), h1 = h0 + 1;
                const int live = (h0 < w.H ? 1 : 0) + (h1 < w.H ? 1 : 0);
                if (gi >= NVS) ok = wait(C_VEMPTY + st, ph, 2);
                if (!ok) return;
                if (c.ui == REFLEX_TRACE_UNIT) TC2_TRACE(0, c.jj, 2);
                mbar_expect_tx(bar(C_VLAND + st), (uint32_t)live * L::V_HALF);
                for (int hh = h0; hh <= h1; ++hh) {
                    if (hh >= w.H) break;
                    const TileRef tr = w.g.decode(hh);
                    for (int ch = 0; ch < VCH; ++ch)
                        tma_load_3d(base + L::OFF_V + st * L::V_STAGE + ch * (128 * 128) + (hh & 1) * (64 * 128), tr.dyn ? &tm_vd : &tm_v,
                                    bar(C_VLAND + st), ((int)rank * VCH + ch) * 64, w.kvh, tr.row0);
                }
            };
            Cursor ck, cv;
            ck.u = u_start; ck.ui = 0; ck.jj = 0; ck.g = 0;
            // Where a Q tile lies follows from the unit's number alone: with unsplit keys (no unit is ever empty) the first
            // one is requested before the stream state, which everything else about the unit hangs on, has come in.
            const bool q_early = p.nsplit == 1 && u_start < n_units;
            if (q_early) {
                const int pair = u_start % n_pairs, kvh = (u_start / n_pairs) % p.Hkv, b = u_start / (n_pairs * p.Hkv);
                if (rank == 0) mbar_expect_tx(bar(C_QFULL), 2 * L::Q_BYTES);
                for (int ch = 0; ch < CH; ++ch)
                    tma2_load_4d(base + L::OFF_Q + ch * (128 * 128), &tm_q, bar(C_QFULL) & kPeerBitMask, ch * 64, kvh * p.G,
                                 (2 * pair + (int)rank) * p.tile_tokens, b);
            }
            settle(ck);
            cv = ck;
            if (kLead == 1 && ck.valid) { issue_k(ck); if (!q_early) issue_q(ck); advance(ck); }
            // At a unit boundary the pipe's completions come as QK(last - 1) PV(last - 2) QK(last): the next unit's first K
            // tile, the V tile of this unit's last P V and then the next unit's Q tile go out in that order, and the next
            // unit's geometry (a global load and some divisions) is worked out only after the V tile is on its way.
            while (cv.valid && ok) {
                const bool k_now = ck.valid;
                if (k_now) { issue_k(ck); if (!ok) break; }
                issue_v(cv);
                if (!ok) break;
                if (k_now) {
                    if (ck.jj == 0 && !(q_early && ck.ui == 0)) { issue_q(ck); if (!ok) break; }
                    advance(ck);
                }
                advance(cv);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA) ----------------
        // Q K^T of tile j+1 is issued before waiting for P(j): S is double buffered in TMEM, so the tensor pipe works on the
        // next tile's logits while the softmax threads finish this tile. S(j+2) overwrites the buffer that held P(j); the MMAs
        // of one thread run in issue order, and Q K^T(j+2) is issued after P V(j), so the pipe itself keeps that hazard away.
        // (Two issuing threads in two warps, one per kind of MMA with the hazard made explicit by a completion barrier, were
        // measured 3 % slower: Q K^T(j+2) then starts a P V latency later. This thread shares its scheduler with two softmax
        // warps and is short of issue slots whenever they run dense arithmetic; a stand-alone issue loop beside pure-FMA
        // warps took 600 cycles per MMA instead of 65.)
        // The whole warp runs these loops converged and one elected lane issues (see umma2_ss_elect).
        if (rank == 0) {
            constexpr uint32_t idesc_qk = umma_idesc_bf16(256, kTc2Keys, false);
            constexpr uint32_t idesc_pv = umma_idesc_bf16(256, HD, true);
            const uint64_t qdesc0 = umma_desc_sw128(base + L::OFF_Q, 16, 1024), kdesc0 = umma_desc_sw128(base + L::OFF_K, 16, 1024);
            const uint64_t vdesc0 = umma_desc_sw128(base + L::OFF_V, 128 * 128, 1024);
            auto qk = [&](int gi, bool last) -> bool {
                const int st = gi % NKS, buf = gi & 1;
                if (!wait(C_KFULL + st, (uint32_t)(gi / NKS) & 1u, 5)) return false;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + kColS + buf * kTc2Keys;
                uint64_t qd = qdesc0, kd = kdesc0;
                umma_desc_advance(kd, (uint32_t)st * L::K_STAGE);
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    umma2_ss_elect(d_tmem, qd, kd, idesc_qk, kk > 0 ? 1u : 0u);
                    // next 16 columns of head_dim: 32 bytes on inside a 64-column chunk, else on to the next chunk
                    umma_desc_advance(qd, (kk & 3) == 3 ? 128 * 128 - 96 : 32);
                    umma_desc_advance(kd, (kk & 3) == 3 ? 64 * 128 - 96 : 32);
                }
                umma2_commit_mc_elect(bar(C_KEMPTY + st), pair_mask);
                umma2_commit_mc_elect(bar(C_SFULL + buf), pair_mask);
                if (last) umma2_commit_mc_elect(bar(C_QEMPTY), pair_mask);
                return true;
            };
            bool ok = true;
            int gt = 0, ui = 0;
            for (int u = u_start; u < n_units && ok; u += u_stride, ++ui) {
                const Unit w = load_unit(u);
                const int n = w.n_tiles;
                if (n == 0) { --ui; continue; }
                ok = wait(C_QFULL, (uint32_t)ui & 1u, 3) && qk(gt, n == 1);
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int gi = gt + jj, st = gi % NVS, buf = gi & 1;
                    if (jj + 1 < n) { ok = qk(gi + 1, jj + 2 == n); if (!ok) break; }
                    ok = wait(C_PFULL + buf, (uint32_t)(gi >> 1) & 1u, 8);
                    if (ok && jj == 0 && ui >= 1) ok = wait(C_OFREE, (uint32_t)(ui - 1) & 1u, 15);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t p_tmem = tmem_base + kColS + buf * kTc2Keys;
                    uint64_t vd = vdesc0;
                    umma_desc_advance(vd, (uint32_t)st * L::V_STAGE);
                    // a tile whose second 64-key half lies past the unit's last key (odd number of halves) contributes
                    // nothing from it: its P is zero and its V rows were never loaded, so those four MMAs are left out
                    const int ksteps = (2 * (w.tile0 + jj) + 1 < w.H) ? kTc2Keys / 16 : kTc2Keys / 32;
#pragma unroll 4
                    for (int kk = 0; kk < ksteps; ++kk) {
                        umma2_ts_elect(tmem_base + kColO, p_tmem + kk * 8, vd, idesc_pv, (jj > 0 || kk > 0) ? 1u : 0u);
                        umma_desc_advance(vd, 16 * 128);   // the next 16 keys
                    }
                    umma2_commit_mc_elect(bar(C_VEMPTY + st), pair_mask);
                    umma2_commit_mc_elect(bar(C_PVDONE + buf), pair_mask);
                }
                gt += n;
            }
        }
    } else {
        // ---------------- softmax / correction / epilogue (both CTAs) ----------------
        // 4 * NP warps: NP threads per query row, one per KT-key slice of the 128-key tile (slice `part`; a warp's TMEM
        // lane quarter fixes which 32 rows it serves). The threads of a row meet once per tile to agree on the row
        // maximum. A wait that ran out never leaves these loops: every softmax warp keeps meeting the others at the
        // named barrier (the remaining waits return at once), so no warp is left behind.
        constexpr int NP = kTc2Parts, KT = kTc2Keys / NP, SMT = 128 * NP;
        constexpr uint64_t kSliceFull = (KT == 64) ? ~0ull : ((1ull << (KT & 63)) - 1ull);
        const int sw = warp - 2;
        const int part = sw >> 2;                 // which KT-key slice of the tile
        const int half = (part * KT) >> 6;        // the 64-key half (one CTA's K rows) that slice lies in
        const int koff = (part * KT) & 63;        // first key of the slice inside its half
        const int quarter = warp & 3;             // TMEM lane quarter this warp may touch
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const uint32_t leader_pfull[2] = {mapa(bar(C_PFULL), lead), mapa(bar(C_PFULL + 1), lead)};
        const uint32_t leader_ofree = mapa(bar(C_OFREE), lead);
        float *xmax = reinterpret_cast<float *>(smem + L::OFF_XMAX);         // [2 buffers][128 rows][NP]
        bool ok = true;
        int gt = 0;
        [[maybe_unused]] int ui_s = 0;
        // (the next unit's geometry -- a global load of the stream state and a handful of integer divisions, about 800 cycles --
        // is worked out while this unit's last P V completes, not at the top of the next unit)
        Unit w_next;
        bool have_next = false;
        for (int u = u_start; u < n_units; u += u_stride, ++ui_s) {
            const Unit w = have_next ? w_next : load_unit(u);
            have_next = false;
            // (key-split units of a few streams may cover half a tile's tokens per CTA, rows past them idle: twice the CTAs then
            // share the fp32 partials, which leave an SM at about 24 bytes per clock whatever else it does)
            const int t_row = row < p.live_rows ? w.t0 + row / p.G : 0x3fffffff;
            if (threadIdx.x == 64) TC2_TRACE(2, ui_s, 0);
            const int rows_total = p.T * p.Hq;
            const size_t n_slots = (size_t)p.B * rows_total * p.nsplit;
            float *pml = nullptr;    // this row's (m, l) slot when the keys are split over several units
            if (p.nsplit > 1 && !p.cluster_merge && t_row < p.T)   // (merged inside the cluster: no partials exist)
                pml = partial_ml(p.partials, n_slots, partial_slot(w.b, rows_total, t_row * p.Hq + w.kvh * p.G + row % p.G, p.nsplit, w.split), HD);
            if (w.n_tiles == 0) {
                if (pml && part == 0) { pml[0] = -INFINITY; pml[1] = 0.f; }   // an empty key slice contributes nothing
                continue;
            }
            float m_ref = -INFINITY, l = 0.f;
            const int full_halves = w.g.S / kBN;      // 64-key halves that lie entirely inside the static prefix
            // one tile of the softmax, compiled twice: for a half that lies entirely inside the static prefix (every key live:
            // no masks, nothing to clear) and for the rest
            auto tile = [&](auto mode_c, const int jj) {
                constexpr bool FULL = decltype(mode_c)::value == 0;
                // a half past the unit's last key (odd number of halves: second half of the last tile) has no logits to read and
                // no P to write: its threads only take part in the row exchange, rescale their columns of O and arrive
                constexpr bool DEAD = decltype(mode_c)::value == 2;
                const int gi = gt + jj, buf = gi & 1, st = gi % NVS;
                const uint32_t vph = (uint32_t)(gi / NVS) & 1u;
                const int h = 2 * (w.tile0 + jj) + half;
                uint64_t tmask = ~0ull, rmask = ~0ull;   // liveness of the 64 keys of this half: for every row / for this row
                if constexpr (!FULL) {
                  tmask = rmask = 0ull;
                  if (h < w.H) {
                    const TileRef tr = w.g.decode(h);
                    tmask = w.g.tile_mask(tr);
                    rmask = tmask;
                    if (tr.kind == 2 && p.dyn_mask) {
                        const int lim = t_row - tr.idx * kBN;
                        rmask &= (lim < 0) ? 0ull : (lim >= 63 ? ~0ull : ((2ull << lim) - 1ull));
                    }
                  }
                }
                const uint64_t smask = FULL ? kSliceFull : ((rmask >> koff) & kSliceFull);   // this thread's KT keys
#define SM_EV(ev) do { if (threadIdx.x == 64 && ui_s == REFLEX_TRACE_UNIT) TC2_TRACE(3, jj, ev); } while (0)
                SM_EV(0);
                float s[KT];
                if constexpr (!DEAD) {
                    ok = ok && wait(C_SFULL + buf, (uint32_t)(gi >> 1) & 1u, 9);
                    SM_EV(1);
                    if (threadIdx.x == 64 && jj == 0) TC2_TRACE(2, ui_s, 1);
                    tc_fence_after();
                    const uint32_t s_addr = tmem_base + lane_addr + kColS + buf * kTc2Keys + part * KT;
                    uint32_t r[KT];
#pragma unroll
                    for (int q = 0; q < KT / 32; ++q) tmem_ld32(s_addr + 32 * q, *reinterpret_cast<uint32_t(*)[32]>(r + 32 * q));
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < KT; ++c) s[c] = __uint_as_float(r[c]);
                }
                SM_EV(2);
                if (!FULL && !DEAD && tmask != ~0ull) {   // (a half past the unit's last key is never read by P V: nothing to clear)
                    // dead keys get weight 0, but 0 x (stale NaN/Inf bytes) would still poison O: clear their V rows as soon
                    // as this CTA's V half has landed. (Doing it at the end of the tile, where every thread waits for V anyway,
                    // puts the clearing stores and their proxy fence in front of the P-ready arrival: measured slower.)
                    ok = ok && wait(C_VLAND + st, vph, 12);
                    // (all 128 threads of the slice share the stores: thread `row` takes half of V row `row % 64`. Two warps
                    // clearing a whole dead half alone, 32 stores each, held their next shared-memory load for 700 cycles.)
                    if (koff == 0 && !((tmask >> (row & 63)) & 1ull)) {
#pragma unroll
                        for (int c = 0; c < VCH; ++c) {
                            uint4 *vr = reinterpret_cast<uint4 *>(smem + L::OFF_V + st * L::V_STAGE + c * (128 * 128) + (half * 64 + (row & 63)) * 128) + (row >> 6) * 4;
#pragma unroll
                            for (int i = 0; i < 4; ++i) vr[i] = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                float mx = -INFINITY;
                if constexpr (!DEAD) {
                if (!FULL && smask != kSliceFull) apply_slice_mask<KT>(s, smask);
                // three-input maxima: half the instructions of a two-input chain (the single MMA-issuing thread shares its
                // scheduler with two of these warps, and every issue slot they do not take is one it can have)
                float mx4[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
                for (int c = 4; c + 7 < KT; c += 8) {
                    mx4[0] = max3_f32(mx4[0], s[c], s[c + 1]); mx4[1] = max3_f32(mx4[1], s[c + 2], s[c + 3]);
                    mx4[2] = max3_f32(mx4[2], s[c + 4], s[c + 5]); mx4[3] = max3_f32(mx4[3], s[c + 6], s[c + 7]);
                }
                static_assert((KT - 4) % 8 == 4 || (KT - 4) % 8 == 0, "tail of the maximum loop");
                if constexpr ((KT - 4) % 8 == 4) {
                    mx4[0] = max3_f32(mx4[0], s[KT - 4], s[KT - 3]); mx4[1] = max3_f32(mx4[1], s[KT - 2], s[KT - 1]);
                }
                mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                }
                // meet the threads that hold the other keys of this row: every one of them publishes its maximum and takes the
                // largest of the NP published values, so all agree. Past this barrier every thread of the row has its logits
                // in registers, so P may overwrite them in tensor memory.
                SM_EV(3);
                xmax[(buf * 128 + row) * NP + part] = mx;
                asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");
                SM_EV(4);
                {
                    const float *xr = xmax + (buf * 128 + row) * NP;
                    mx = xr[0];
#pragma unroll
                    for (int q = 1; q < NP; ++q) mx = fmaxf(mx, xr[q]);
                }
                if (jj == 0) {
                    m_ref = mx;
                } else {
                    const bool grow = (mx - m_ref) * p.scale_log2 > kRescaleThreshold;
                    if (__any_sync(0xffffffffu, grow)) {
                        // O (and l) were accumulated against m_ref: bring them to the new reference before this tile's P V.
                        // All threads of a row see the same mx, so they decide alike; each rescales its share of O's columns.
                        const float alpha = grow ? ex2((m_ref - mx) * p.scale_log2) : 1.f;
                        if (grow) m_ref = mx;
                        l *= alpha;
                        ok = ok && wait(C_PVDONE + ((gi - 1) & 1), (uint32_t)((gi - 1) >> 1) & 1u, 10);
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < HD / NP / 32; ++c) {
                            uint32_t o[32];
                            const uint32_t o_addr = tmem_base + lane_addr + kColO + part * (HD / NP) + c * 32;
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
                // P = 2^(s*scale*log2e - m), two keys per instruction wherever the hardware has a packed form (the scaling FMA,
                // the running sums, the polynomial). A quarter of the key pairs take a cubic on the FMA pipe, the rest the MUFU
                // unit (4 results per clock and scheduler): measured 2/8 35.4 us, 0/8 35.6, 3/8 35.9, 4/8 36.4 per launch.
                SM_EV(6);
                if constexpr (!DEAD) {
                const uint64_t sc2 = pack_f32x2(p.scale_log2, p.scale_log2), nm2 = pack_f32x2(-mr, -mr);
                const Ex2PolyConsts pk = ex2_poly_consts();
                uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
                uint32_t packed[KT / 2];
#pragma unroll
                for (int c = 0; c < KT; c += 2) {
                    float x0, x1;
                    unpack_f32x2(fma_f32x2(pack_f32x2(s[c], s[c + 1]), sc2, nm2), x0, x1);
                    float p0, p1;
                    if (((c >> 1) & 7) < kTc2PolyEighths) ex2_poly_f32x2(x0, x1, pk, p0, p1);
                    else { p0 = ex2(x0); p1 = ex2(x1); }
                    sum2[(c >> 1) & 3] = add_f32x2(sum2[(c >> 1) & 3], pack_f32x2(p0, p1));
                    __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
                    packed[c >> 1] = *reinterpret_cast<uint32_t *>(&hh);
                }
                {
                    float a, b;
                    unpack_f32x2(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), a, b);
                    l += a + b;
                }
                if (!FULL && kTc2PolyEighths > 0 && smask != kSliceFull) {
                    // the polynomial gives a masked key 2^-125 instead of 0 (nothing for the sum, but P must be exactly 0
                    // there): clear those halves of the packed words
#pragma unroll
                    for (int c = 0; c < KT; c += 2) {
                        if (((c >> 1) & 7) < kTc2PolyEighths) {
                            const uint32_t two = (uint32_t)(smask >> c) & 3u;
                            packed[c >> 1] &= ((two & 1u) ? 0x0000FFFFu : 0u) | ((two & 2u) ? 0xFFFF0000u : 0u);
                        }
                    }
                }
                SM_EV(5);
                // P goes into the first 64 columns of S's buffer (two keys per column): the A operand of this tile's P V.
                // (No wait for an earlier P V: the one that read this buffer, two tiles back, was issued before the Q K^T
                // that produced the logits just consumed.)
                {
                    const uint32_t p_addr = tmem_base + lane_addr + kColS + buf * kTc2Keys + part * (KT / 2);
                    if constexpr (KT == 64) tmem_st32(p_addr, *reinterpret_cast<const uint32_t(*)[32]>(packed));
                    else tmem_st16(p_addr, *reinterpret_cast<const uint32_t(*)[16]>(packed));
                    tmem_wait_st();
                }
                }
                SM_EV(7);
                // (The waits on a P V barrier, one barrier per S/P buffer, come at irregular times: before rescaling O and before
                // reading O out. Their parity test stays unambiguous because S(g) exists only after P V(g-2) completed, so the
                // barrier of tile g-1 has finished the phase of tile g-3 and cannot have passed that of tile g+1.)
                // the arrive below also tells the leader that this CTA's V half is in place
                if (FULL || DEAD || tmask == ~0ull) ok = ok && wait(C_VLAND + st, vph, 12);
                SM_EV(8);
                fence_proxy_async_smem();   // V rows cleared above are read by the tensor pipe
                tc_fence_before();
                __syncwarp();
                // (one barrier per S/P buffer: the two CTAs' softmax warps are not synchronised with each other, and on a single
                // barrier a CTA one tile ahead would complete this tile's phase with its arrivals for the next)
                if (lane == 0) mbar_arrive_cluster(leader_pfull[buf]);
                SM_EV(9);
            };
            for (int jj = 0; jj < w.n_tiles; ++jj) {
                const int hh = 2 * (w.tile0 + jj) + half;
                if (hh < full_halves) tile(std::integral_constant<int, 0>{}, jj);
                else if (hh < w.H) tile(std::integral_constant<int, 1>{}, jj);
                else tile(std::integral_constant<int, 2>{}, jj);
            }
            gt += w.n_tiles;
            if (u + u_stride < n_units) { w_next = load_unit(u + u_stride); have_next = true; }
            // ---- epilogue of the unit ----
            // (before this cluster's last epilogue: let the next kernel on the stream be scheduled; it waits for this grid's end)
            if (threadIdx.x == 64 && u + u_stride >= n_units) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            // The threads of a row add their sums; each thread takes its share of the head_dim columns out of tensor
            // memory, 32 at a time, and stores its row segment straight to global memory in 32-byte pieces (whole sectors).
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 2); TC2_TRACE(2, ui_s, 2); }
            const int g_last = gt - 1;
            ok = ok && wait(C_PVDONE + (g_last & 1), (uint32_t)(g_last >> 1) & 1u, 13);
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 3); TC2_TRACE(2, ui_s, 3); }
            float *xsum = xmax + ((g_last & 1) ^ 1) * (128 * NP);      // [NP][128 rows], in the maxima buffer the last tile did not use
            xsum[part * 128 + row] = l;
            asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");
#pragma unroll
            for (int q = 1; q < NP; ++q) l += xsum[((part + q) % NP) * 128 + row];
            tc_fence_after();
            if (threadIdx.x == 64) TC2_TRACE(2, ui_s, 5);
            const bool row_live = t_row < p.T;
            const int hq = w.kvh * p.G + row % p.G;
            constexpr int EC = HD / NP;            // this thread's columns of O
            if (p.cluster_merge) {
                // the slices of this tile pair meet in the merge phase at the end of the kernel (this pair has no other unit)
                fin_m = (m_ref == -INFINITY) ? -INFINITY : m_ref * p.scale_log2;
                fin_l = l;
                fin_ok = ok;
                continue;
            }
            if (p.nsplit > 1) {
                // key-split unit: leave (m, l, unnormalised O) for the merge kernel; m in natural-log units like the other kernels
                if (pml && part == 0) { pml[0] = (m_ref == -INFINITY) ? -INFINITY : m_ref * p.scale; pml[1] = l; }
                if (threadIdx.x == 64) TC2_TRACE(2, ui_s, 6);
                if (u + u_stride >= n_units) {
                    // The cluster's last unit (its only one when few streams are split finely): the Q tile and the K stages are
                    // idle, so the whole fp32 tile (128 rows x head_dim) is staged there, every thread dropping its half row as
                    // 16-byte pieces at [row][piece ^ (row % 32)], and each warp then writes whole rows of the partial area, 512
                    // contiguous bytes per instruction. (Straight from registers every store instruction touched 32 rows
                    // 8 KB apart: 4.5 of the 10.3 us of a one-stream launch.)
                    static_assert(L::OFF_K == L::OFF_Q + L::Q_BYTES && L::Q_BYTES + L::NKS * L::K_STAGE >= (uint32_t)HD * 128 * 4, "staging area of the partial tile");
                    constexpr int PR = HD / 4;                          // 16-byte pieces per row
                    uint4 *stage = reinterpret_cast<uint4 *>(smem + L::OFF_Q);
#pragma unroll 1
                    for (int c = 0; c < EC / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tmem_base + lane_addr + kColO + part * EC + c * 32, o);
                        tmem_wait_ld();
                        if (c == EC / 32 - 1) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(leader_ofree);
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            stage[row * PR + (((part * EC + c * 32) / 4 + i) ^ (row & 31))] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");
                    constexpr int RW = 128 / (4 * NP);                  // rows per warp
#pragma unroll 2
                    for (int rr = 0; rr < RW; ++rr) {
                        const int r = sw * RW + rr;
                        const int tr = w.t0 + r / p.G;
                        if (tr >= p.T || r >= p.live_rows) continue;
                        float *dst = partial_o(p.partials, partial_slot(w.b, rows_total, tr * p.Hq + w.kvh * p.G + r % p.G, p.nsplit, w.split), HD);
#pragma unroll
                        for (int h = 0; h < PR / 32; ++h) {
                            const int piece = h * 32 + lane;
                            reinterpret_cast<uint4 *>(dst)[piece] = stage[r * PR + (piece ^ (r & 31))];
                        }
                    }
                } else {
                float *po = row_live ? partial_o(p.partials, partial_slot(w.b, rows_total, t_row * p.Hq + hq, p.nsplit, w.split), HD) + part * EC : nullptr;
#pragma unroll 1
                for (int c = 0; c < EC / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + part * EC + c * 32, o);
                    tmem_wait_ld();
                    if (c == EC / 32 - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(leader_ofree);
                    }
                    if (row_live) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) st_global_v8(po + c * 32 + 8 * i, *reinterpret_cast<const uint32_t(*)[8]>(o + 8 * i));
                    }
                }
                }
                if (threadIdx.x == 64) TC2_TRACE(2, ui_s, 7);
                asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");   // every thread has read the row sums before the next unit's maxima land there
                continue;
            }
            // O / l goes out through a 32 KB staging area laid out like a Q tile (two 64-column chunks of 128 swizzled rows)
            // and TMA stores: the threads are done once the tile sits in shared memory, and the store drains underneath the
            // next unit. (Stores straight from registers kept every thread until its 64 KB were accepted by a memory system
            // that all clusters hit at the same moment: 4.4 k cycles per unit.)
            const float inv = 1.f / l;
            const bool store_unit = w.t0 < p.T;   // an idle partner tile (odd tile count) has nothing to write
            // Rounds of 64 columns, alternating between the two 16 KB halves of the staging area: the TMA store of one round
            // reads its half while the threads convert the next round into the other (one store of 32 KB per 128 columns made
            // every second round wait about 900 cycles for the first to be read).
            constexpr int SC = 64 / NP;            // columns per thread and round
            static_assert(SC == 32 || SC == 16, "columns per thread and epilogue round");
#pragma unroll 1
            for (int rnd = 0; rnd < HD / 64; ++rnd) {
                uint32_t o[SC];
                const uint32_t o_addr = tmem_base + lane_addr + kColO + rnd * 64 + part * SC;
                if constexpr (SC == 32) tmem_ld32(o_addr, *reinterpret_cast<uint32_t(*)[32]>(o));
                else tmem_ld16(o_addr, *reinterpret_cast<uint32_t(*)[16]>(o));
                // this half may still be read by the store issued two rounds ago (this unit's or the previous one's)
                if (threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                tmem_wait_ld();
                if (rnd == HD / 64 - 1) {
                    // all of O is in registers: the next unit's first P V may overwrite the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(leader_ofree);
                }
                asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");
                uint8_t *srow = smem + L::OFF_STAGE + (rnd & 1) * (128 * 128) + row * 128;
                const int c16 = part * (SC / 8);
#pragma unroll
                for (int c = 0; c < SC / 8; ++c) {
                    uint4 v;
                    uint32_t *vv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(o[8 * c + 2 * k]) * inv, __uint_as_float(o[8 * c + 2 * k + 1]) * inv);
                        vv[k] = *reinterpret_cast<uint32_t *>(&hh);
                    }
                    *reinterpret_cast<uint4 *>(srow + (((c16 + c) ^ (row & 7)) << 4)) = v;
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, %0;" ::"n"(SMT) : "memory");
                if (threadIdx.x == 64) {
                    if (store_unit) tma_store_4d(&tm_o, base + L::OFF_STAGE + (rnd & 1) * (128 * 128), rnd * 64, w.kvh * p.G, w.t0, w.b);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            if (threadIdx.x == 64) { TC2_TRACE(2, 15, 4); TC2_TRACE(2, ui_s, 4); }
        }
        if (threadIdx.x == 64) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores of this CTA are complete
    }

    if (p.cluster_merge) {
        // ---- merge of the key slices inside the cluster ----
        // Pair q of the cluster holds slice q of the keys for the same 256 query rows; CTAs of equal rank inside their pairs
        // hold the same 128 rows. 1. every row's (m, l) is published; 2. with all slices' (m, l) each thread scales its
        // share of its O row to the common maximum and stages it in shared memory (Q and K buffers, idle now), column-major
        // in 16-byte units; 3. pair q adds up columns [q, q+1) * head_dim / nsplit of all slices through distributed shared
        // memory, divides by the common sum and writes bf16. A cluster barrier after 1 and after 2; the one at the end of
        // the kernel keeps every CTA alive while a peer may still read its staging area.
        constexpr int NP = kTc2Parts;
        const int ns = p.nsplit;
        const int sw = warp - 2, part = sw >> 2;
        const int row = (warp & 3) * 32 + lane;
        float2 *ml_own = reinterpret_cast<float2 *>(smem + L::OFF_STAGE);      // [128 rows]
        float4 *stage = reinterpret_cast<float4 *>(smem + L::OFF_Q);           // [HD / 4][128 rows]
        static_assert(L::OFF_K == L::OFF_Q + L::Q_BYTES && L::Q_BYTES + L::NKS * L::K_STAGE >= (uint32_t)HD * 128 * 4, "staging area of the merge");
        // (the cluster barriers are warp-aligned instructions: the lanes of the producer warp that idled while lane 0 ran the
        // loads must not reach them before lane 0 does, so the CTA meets here first)
        __syncthreads();
        if (warp >= 2 && part == 0) ml_own[row] = make_float2(fin_m, fin_l);
        cluster_arrive();
        cluster_wait();
        float wgt[8], l_all = 0.f;
        if (warp >= 2) {
            float pm[8], mstar = -INFINITY;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                pm[q] = -INFINITY; wgt[q] = 0.f;
                if (q < ns) {
                    float lq;
                    const uint32_t a = mapa(smem_u32(ml_own + row), (uint32_t)(2 * q) + rank);
                    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(pm[q]), "=f"(lq) : "r"(a) : "memory");
                    wgt[q] = lq;                                   // the sum for now
                    if (!(lq > 0.f)) pm[q] = -INFINITY;            // a slice that saw nothing live has no say
                    mstar = fmaxf(mstar, pm[q]);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float e = (pm[q] == -INFINITY) ? 0.f : ex2(pm[q] - mstar);
                l_all = fmaf(wgt[q], e, l_all);
                wgt[q] = e;
            }
            float w_own = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q == (int)(crank >> 1)) w_own = wgt[q];
            {
                // Only the columns that OTHER pairs reduce are staged; this pair's own columns stay in tensor memory until the
                // reduction below. (The tensor-memory loads are warp-wide: every lane takes part, whatever its own row's
                // weight; a row without weight in this slice, or a slice without tiles whose accumulator was never written,
                // stages nothing.)
                tc_fence_after();
                const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
                constexpr int EC = HD / NP;
                const bool mine = w_own > 0.f && fin_ok;
                const int own_lo = (int)(crank >> 1) * (HD / ns), own_hi = own_lo + HD / ns;     // columns this pair reduces
#pragma unroll 1
                for (int c = 0; c < EC / 32; ++c) {
                    const int col0 = part * EC + c * 32;
                    if (col0 >= own_lo && col0 < own_hi) continue;        // (uniform over the CTA; HD / ns is a multiple of 32)
                    uint32_t o[32];
                    tmem_ld32(tmem_base + lane_addr + kColO + col0, o);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            stage[(col0 / 4 + i) * 128 + row] =
                                make_float4(__uint_as_float(o[4 * i]) * w_own, __uint_as_float(o[4 * i + 1]) * w_own,
                                            __uint_as_float(o[4 * i + 2]) * w_own, __uint_as_float(o[4 * i + 3]) * w_own);
                    }
                }
            }
        }
        cluster_arrive();
        cluster_wait();
        if (warp >= 2) {
            // this pair's columns [crank/2 * HD/ns, +HD/ns), split between the NP threads of the row: its own share comes
            // straight from tensor memory, the other slices' shares from their staging areas
            const int uu = u_start / p.nsplit, pair = uu % n_pairs, kvh = (uu / n_pairs) % p.Hkv, b = uu / (n_pairs * p.Hkv);
            const int t_row = (2 * pair + (int)rank) * p.tile_tokens + row / p.G;
            const int own = (int)(crank >> 1);
            const int cols_thread = HD / ns / NP;                                       // columns per thread: 16, 32 or 64
            const int col_0 = own * (HD / ns) + part * cols_thread;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const bool live = fin_ok && t_row < p.T && l_all > 0.f;
            float w_own = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (q == own) w_own = wgt[q];
            if (!(fin_l > 0.f)) w_own = 0.f;                                            // an accumulator that was never written
            const float inv = live ? 1.f / l_all : 0.f;
            __nv_bfloat16 *orow = (__nv_bfloat16 *)p.out + (((size_t)b * p.T + (live ? t_row : 0)) * p.Hq + kvh * p.G + row % p.G) * HD + col_0;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < cols_thread; c0 += 16) {
                uint32_t o[16];
                tmem_ld16(tmem_base + lane_addr + kColO + col_0 + c0, o);              // warp-wide, whatever the row's state
                tmem_wait_ld();
                if (!live) continue;
                float acc[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = w_own > 0.f ? __uint_as_float(o[i]) * w_own : 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q < ns && q != own && wgt[q] > 0.f) {
                        const uint32_t a = mapa(smem_u32(stage + ((col_0 + c0) / 4) * 128 + row), (uint32_t)(2 * q) + rank);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float4 v;
                            asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a + j * 128 * 16) : "memory");
                            acc[4 * j] += v.x; acc[4 * j + 1] += v.y; acc[4 * j + 2] += v.z; acc[4 * j + 3] += v.w;
                        }
                    }
                }
#pragma unroll
                for (int h8 = 0; h8 < 2; ++h8) {
                    uint4 v;
                    uint32_t *vv = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(acc[8 * h8 + 2 * k] * inv, acc[8 * h8 + 2 * k + 1] * inv);
                        vv[k] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    *reinterpret_cast<uint4 *>(orow + c0 + 8 * h8) = v;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();   // neither CTA retires while its partner can still touch its shared memory or barriers
    if (warp == 1) tmem_dealloc2(tmem_base, kTmemCols);
    if (threadIdx.x == 64) TC2_TRACE(2, 15, 5);
}

}  // namespace reflex
