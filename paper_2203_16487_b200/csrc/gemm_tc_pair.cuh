// Two-SM variant of the tensor-core GEMM (tcgen05 cta_group::2) for the wide GEMMs over many rows.
//
// A cluster of two CTAs works on one 256-row x BN-column tile.  Each CTA stages its own 128 activation
// rows and HALF of the weight tile (BN / 2 weight rows); one thread of the leader CTA (cluster rank 0)
// issues tcgen05.mma.cta_group::2 with M = 256, which reads both CTAs' shared memory and leaves rows
// 0..127 of the result in the leader's tensor memory and rows 128..255 in the peer's.  A CTA therefore
// ingests (128 + BN / 2) * K * 2 bytes per 128 x BN outputs instead of (128 + BN) * K * 2: the single-SM
// kernel is bound by exactly that ingest, not by the MMAs.
//
// Synchronisation (every wait is bounded, as in the single-SM kernel):
//   full[s]      in the leader: its producer expects the bytes of BOTH CTAs' loads; both CTAs' TMA loads
//                (cta_group::2 form, no multicast) complete their bytes on it;
//   empty[s]     in each CTA, acc_full[i] in each CTA: signalled by the leader's MMA thread with one
//                multicast tcgen05.commit (same barrier offset in both CTAs);
//   acc_empty[i] in the leader: the eight epilogue warps of both CTAs arrive on it (the peer's remotely).
// Cluster barriers bracket the kernel so that no CTA touches the other's barriers before they exist or
// leaves while the other may still read its shared memory.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

__device__ __forceinline__ uint32_t pair_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t pair_map(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void pair_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA tile load into this CTA's shared memory whose bytes are counted on a barrier given by its cluster address
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// arrives, once the MMAs issued so far have completed, on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

template <int BN, bool STG = true> struct TcPairCfg {
    static constexpr int BNH = BN / 2;                                    // weight rows a CTA stages per tile
    static constexpr int STAGE_BYTES = (TC_BM + BNH) * TC_BK * 2;
    static constexpr int STG_BYTES = STG ? TC_EPI_WARPS * 32 * 32 * 4 : 0;
    static constexpr int FIT = (232448 - 1024 - STG_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = FIT > 8 ? 8 : FIT;
    static constexpr int SMEM = STAGES * STAGE_BYTES + STG_BYTES + 1024;
    static constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);   // two accumulators
    static_assert(BN % 32 == 0 && BN >= 64 && BN <= 256, "pair tile width");
};

// Persistent over pair tiles: pair p works on tiles p, p + pairs, ... (row pair fastest, so pairs running
// together share one weight tile).  Ring and accumulators run across tiles as in the single-SM kernel.
template <int EPI, int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
k_gemm_tc_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g,
               int* err_word) {
    using Cfg = TcPairCfg<BN, EPI != EPI_STATS>;
    constexpr int STAGES = Cfg::STAGES, BNH = Cfg::BNH;
    constexpr int A_BYTES = TC_BM * TC_BK * 2;
    if (threadIdx.x == 0) tc_stamp(g.trace, 0);
    const bool early = g.rows_static >= 0;
    if (!early) pdl_wait();
    const int R = early ? g.rows_static : *g.n_rows;
    const int m_pairs = (R + 2 * TC_BM - 1) / (2 * TC_BM), n_tiles = (g.N + BN - 1) / BN;
    const int total = m_pairs * n_tiles;
    const int pair = (int)blockIdx.x >> 1, pairs = (int)gridDim.x >> 1;
    if (pair >= total) return;                       // both CTAs of the pair leave together, before any cluster barrier

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[STAGES], bar_empty[STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = pair_cta_rank();
    const bool leader = rank == 0;
    const int nkb = g.K / TC_BK;
    float* stg = reinterpret_cast<float*>(smem_raw + (tiles - smem_u32(smem_raw)) + STAGES * Cfg::STAGE_BYTES) + (warp >= 2 ? warp - 2 : 0) * 1024;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_empty[i]), 2 * TC_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&tmem_base_s), Cfg::TMEM_COLS);
    tc_fence_before();
    pair_sync();                                     // both CTAs' barriers and tensor memory exist from here on
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0 && tmem_d != 0xffffffffu) tc_stamp(g.trace, 1);
    int pre = 0;                                     // stages whose weight halves were requested before the wait
    if (early) {
        if (threadIdx.x == 0) {
            const int n0 = (pair / m_pairs) * BN + (int)rank * BNH;
            for (; pre < STAGES && pre < nkb; ++pre) {
                if (leader) mbar_expect_tx(smem_u32(&bar_full[pre]), 2 * Cfg::STAGE_BYTES);
                tma_load_2d_pair(tiles + pre * Cfg::STAGE_BYTES + A_BYTES, &tmW, pre * TC_BK, n0, pair_map(smem_u32(&bar_full[pre]), 0));
            }
        }
        pdl_launch_dependents();
        pdl_wait();                                  // activations, residual and outputs belong to the predecessors until here
    }

    if (warp == 0) {
        if (lane == 0) {
            int kbi = 0;
            int ps = 0; uint32_t ppar = 0; bool wrapped = false, dead = false;   // producer's ring position (incremental: see k_vocab_pair)
            for (int t = pair; t < total && !dead && !*abort_flag; t += pairs) {
                const int m0 = (t % m_pairs) * 2 * TC_BM + (int)rank * TC_BM, n0 = (t / m_pairs) * BN + (int)rank * BNH;
                for (int kb = 0; kb < nkb; ++kb, ++kbi) {
                    if (wrapped && !mbar_wait(smem_u32(&bar_empty[ps]), ppar, abort_flag, err_word, 1)) { dead = true; break; }
                    const uint32_t a_dst = tiles + ps * Cfg::STAGE_BYTES, w_dst = a_dst + A_BYTES;
                    const uint32_t bar = pair_map(smem_u32(&bar_full[ps]), 0);
                    if (kbi >= pre) {
                        if (leader) mbar_expect_tx(smem_u32(&bar_full[ps]), 2 * Cfg::STAGE_BYTES);
                        tma_load_2d_pair(w_dst, &tmW, kb * TC_BK, n0, bar);
                    }
                    tma_load_2d_pair(a_dst, &tmA, kb * TC_BK, m0, bar);
                    if (++ps == STAGES) { ps = 0; if (wrapped) ppar ^= 1u; wrapped = true; }
                }
            }
            tc_stamp(g.trace, 3);
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * TC_BM, BN);
            int kbi = 0, i = 0;
            int s = 0; uint32_t par = 0;                      // ring position kept incrementally; bookkeeping between the issues (see k_gemm_tc)
            const bool stamps = g.trace != nullptr && blockIdx.x == 0;
            for (int t = pair; t < total && !*abort_flag; t += pairs, ++i) {
                const int ab = i & 1;
                if (i >= 2) mbar_wait(smem_u32(&bar_acc_empty[ab]), ((i >> 1) - 1) & 1, abort_flag, err_word, 4);
                tc_fence_after();
                const uint32_t acc = tmem_d + ab * BN;
                bool ok = mbar_wait(smem_u32(&bar_full[s]), par, abort_flag, err_word, 2);
                if (stamps && kbi == 0) tc_stamp(g.trace, 4);
                for (int kb = 0; kb < nkb && ok; ++kb, ++kbi) {
                    const uint32_t a_src = tiles + s * Cfg::STAGE_BYTES, w_src = a_src + A_BYTES;
                    const uint64_t ad = umma_desc_k_sw128(a_src), wd = umma_desc_k_sw128(w_src);
                    umma_bf16_pair(acc, ad, wd, idesc, kb ? 1u : 0u);
                    int sn = s + 1; uint32_t parn = par;
                    if (sn == STAGES) { sn = 0; parn ^= 1u; }
                    const uint32_t next_bar = smem_u32(&bar_full[sn]);
                    umma_bf16_pair(acc, ad + 2, wd + 2, idesc, 1u);
                    const uint32_t early_ok = (kb + 1 < nkb) ? mbar_try_wait(next_bar, parn) : 1u;
                    umma_bf16_pair(acc, ad + 4, wd + 4, idesc, 1u);
                    if (stamps && kbi < 16) tc_stamp(g.trace, 40 + kbi);
                    umma_bf16_pair(acc, ad + 6, wd + 6, idesc, 1u);
                    umma_commit_pair(smem_u32(&bar_empty[s]));       // both CTAs may refill the stage
                    if (!early_ok) ok = mbar_wait(next_bar, parn, abort_flag, err_word, 2);
                    s = sn; par = parn;
                }
                if (!ok) break;
                umma_commit_pair(smem_u32(&bar_acc_full[ab]));       // both CTAs' halves of the accumulator are complete
                if (stamps) tc_stamp(g.trace, 5 + (i > 0));
            }
        }
    } else {
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        int i = 0;
        for (int t = pair; t < total; t += pairs, ++i) {
            const int ab = i & 1;
            const int m0 = (t % m_pairs) * 2 * TC_BM + (int)rank * TC_BM, n_tile = t / m_pairs;
            tc_epilogue_tile<EPI, BN>(g, R, m0, n_tile, q, half, lane, tmem_d + ab * BN, stg, smem_u32(&bar_acc_full[ab]),
                                      (i >> 1) & 1, abort_flag, err_word, i > 0);
            if (lane == 0) mbar_arrive_cluster(pair_map(smem_u32(&bar_acc_empty[ab]), 0));
            if (threadIdx.x == 64) tc_stamp(g.trace, 8 + 2 * (i > 0));
        }
    }
    tc_fence_before();
    pair_sync();                                     // nobody reads the other's memory or barriers past this point
    if (warp == 1) tmem_dealloc_pair(tmem_d, Cfg::TMEM_COLS);
    if (threadIdx.x == 0) tc_stamp(g.trace, 11);
}

// Vocabulary projection + row statistics on two-SM tiles with the activation rows RESIDENT in shared memory:
// a pair of CTAs takes a contiguous run of (row pair, column tile) tiles, column tile fastest, so its 2 x 128
// activation rows (K <= 512: at most 128 KB per CTA) are loaded once per row pair and only the weight halves
// (128 rows x 64 per k-block and CTA) stream through the ring.  Per k-block a CTA then ingests 16 KB instead of
// 32 KB (two-SM tile with streamed activations) or 48 KB (single-SM 128 x 256 tile).
constexpr int VP_BN = 256, VP_BNH = 128, VP_MAX_STAGES = 8;
constexpr int VP_KB_BYTES = TC_BM * TC_BK * 2;                    // 16 KB: one k-block of 128 rows, activations or weights
inline int vp_stages(int K) {
    const int fit = (232448 - 1024 - (K / TC_BK) * VP_KB_BYTES) / VP_KB_BYTES;
    return fit > VP_MAX_STAGES ? VP_MAX_STAGES : fit;
}
inline size_t vp_smem(int K) { return (size_t)(K / TC_BK + vp_stages(K)) * VP_KB_BYTES + 1024; }

// Work units: a unit is (row pair m, segment sg of the column tiles); pair p takes units p, p + pairs, ... with m fastest,
// so the pairs that run together walk the SAME column tiles in the same order for different row pairs: a weight tile is
// then fetched by many SMs of a die within a short time and served by the near half of the L2 (with one private run of
// column tiles per pair, 23 % of the kernel's L2 traffic came from the far half and the ring landed 40 GB/s per CTA).
__device__ __forceinline__ int vp_pick_segs(int m_pairs, int n_tiles, int pairs) {
    int best = 1; long long best_cost = -1;
    for (int k = 1; k <= 4; ++k) {
        int sg = (k * pairs) / m_pairs;
        sg = sg < 1 ? 1 : (sg > n_tiles ? n_tiles : sg);
        const long long cost = (long long)((m_pairs * sg + pairs - 1) / pairs) * ((n_tiles + sg - 1) / sg);   // rounds x tiles per unit
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = sg; }
    }
    return best;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
k_vocab_pair(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g,
             int* err_word, int stages) {
    if (threadIdx.x == 0) tc_stamp(g.trace, 0);
    const bool early = g.rows_static >= 0;
    if (!early) pdl_wait();
    const int R = early ? g.rows_static : *g.n_rows;
    const int m_pairs = (R + 2 * TC_BM - 1) / (2 * TC_BM), n_tiles = (g.N + VP_BN - 1) / VP_BN;
    const int pair = (int)blockIdx.x >> 1, pairs = (int)gridDim.x >> 1;
    const int segs = m_pairs > 0 ? vp_pick_segs(m_pairs, n_tiles, pairs) : 1;
    const int units = m_pairs * segs;
    if (pair >= units) return;                       // both CTAs of the pair leave together, before any cluster barrier
    // unit u: row pair u % m_pairs, column tiles [nb, ne) of segment u / m_pairs
#define VP_UNIT(u, m, nb, ne) const int m = (u) % m_pairs, nb = (((u) / m_pairs) * n_tiles) / segs, ne = (((u) / m_pairs + 1) * n_tiles) / segs

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_w_full[VP_MAX_STAGES], bar_w_empty[VP_MAX_STAGES], bar_a_full, bar_a_empty,
        bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = pair_cta_rank();
    const bool leader = rank == 0;
    const int nkb = g.K / TC_BK;
    const uint32_t a_base = (smem_u32(smem_raw) + 1023u) & ~1023u, w_base = a_base + nkb * VP_KB_BYTES;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < VP_MAX_STAGES; ++s) { mbar_init(smem_u32(&bar_w_full[s]), 1); mbar_init(smem_u32(&bar_w_empty[s]), 1); }
        mbar_init(smem_u32(&bar_a_full), 1); mbar_init(smem_u32(&bar_a_empty), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_empty[i]), 2 * TC_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&tmem_base_s), 512);
    tc_fence_before();
    pair_sync();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0 && tmem_d != 0xffffffffu) tc_stamp(g.trace, 1);
    int pre = 0;                                     // ring stages requested before the wait (weights only)
    if (early) {
        if (threadIdx.x == 0) {
            VP_UNIT(pair, m_first, nb_first, ne_first);
            (void)m_first; (void)ne_first;
            const int n0 = nb_first * VP_BN + (int)rank * VP_BNH;
            for (; pre < stages && pre < nkb; ++pre) {
                if (leader) mbar_expect_tx(smem_u32(&bar_w_full[pre]), 2 * VP_KB_BYTES);
                tma_load_2d_pair(w_base + pre * VP_KB_BYTES, &tmW, pre * TC_BK, n0, pair_map(smem_u32(&bar_w_full[pre]), 0));
            }
        }
        pdl_launch_dependents();
        pdl_wait();
    }

    if (warp == 0) {
        if (lane == 0) {
            int kbi = 0, a_loads = 0;
            int ps = 0; uint32_t ppar = 0; bool wrapped = false, dead = false;   // producer's ring position; ppar = parity of the empty phase awaited
            for (int u = pair; u < units && !dead && !*abort_flag; u += pairs) {
                VP_UNIT(u, m_pair, nb, ne);
                // this unit's activation rows replace the resident ones
                if (a_loads > 0 && !mbar_wait(smem_u32(&bar_a_empty), (a_loads - 1) & 1, abort_flag, err_word, 5)) break;
                if (leader) mbar_expect_tx(smem_u32(&bar_a_full), 2 * nkb * VP_KB_BYTES);
                const uint32_t abar = pair_map(smem_u32(&bar_a_full), 0);
                for (int kb = 0; kb < nkb; ++kb)
                    tma_load_2d_pair(a_base + kb * VP_KB_BYTES, &tmA, kb * TC_BK, m_pair * 2 * TC_BM + (int)rank * TC_BM, abar);
                ++a_loads;
                if (a_loads == 1) tc_stamp(g.trace, 2);
                for (int n = nb; n < ne && !dead; ++n) {
                    const int n0 = n * VP_BN + (int)rank * VP_BNH;
                    for (int kb = 0; kb < nkb; ++kb, ++kbi) {
                        if (wrapped && !mbar_wait(smem_u32(&bar_w_empty[ps]), ppar, abort_flag, err_word, 1)) { dead = true; break; }
                        if (kbi >= pre) {
                            if (leader) mbar_expect_tx(smem_u32(&bar_w_full[ps]), 2 * VP_KB_BYTES);
                            tma_load_2d_pair(w_base + ps * VP_KB_BYTES, &tmW, kb * TC_BK, n0, pair_map(smem_u32(&bar_w_full[ps]), 0));
                        }
                        if (++ps == stages) { ps = 0; if (wrapped) ppar ^= 1u; wrapped = true; }
                    }
                }
            }
            tc_stamp(g.trace, 3);
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * TC_BM, VP_BN);
            int kbi = 0, i = 0, a_uses = 0;
            int s = 0; uint32_t par = 0;                      // ring position kept incrementally; bookkeeping between the issues (see k_gemm_tc)
            const bool stamps = g.trace != nullptr && blockIdx.x == 0;
            bool ok = true;
            for (int u = pair; u < units && ok && !*abort_flag; u += pairs) {
                VP_UNIT(u, m_pair, nb, ne);
                (void)m_pair;
                ok = mbar_wait(smem_u32(&bar_a_full), a_uses & 1, abort_flag, err_word, 6);
                ++a_uses;
                for (int n = nb; n < ne && ok; ++n, ++i) {
                    const int ab = i & 1;
                    if (i >= 2) ok = mbar_wait(smem_u32(&bar_acc_empty[ab]), ((i >> 1) - 1) & 1, abort_flag, err_word, 4);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t acc = tmem_d + ab * VP_BN;
                    ok = mbar_wait(smem_u32(&bar_w_full[s]), par, abort_flag, err_word, 2);
                    if (stamps && kbi == 0) tc_stamp(g.trace, 4);
                    for (int kb = 0; kb < nkb && ok; ++kb, ++kbi) {
                        const uint64_t ad = umma_desc_k_sw128(a_base + kb * VP_KB_BYTES), wd = umma_desc_k_sw128(w_base + s * VP_KB_BYTES);
                        umma_bf16_pair(acc, ad, wd, idesc, kb ? 1u : 0u);
                        int sn = s + 1; uint32_t parn = par;
                        if (sn == stages) { sn = 0; parn ^= 1u; }
                        const uint32_t next_bar = smem_u32(&bar_w_full[sn]);
                        umma_bf16_pair(acc, ad + 2, wd + 2, idesc, 1u);
                        const uint32_t early_ok = (kb + 1 < nkb) ? mbar_try_wait(next_bar, parn) : 1u;
                        umma_bf16_pair(acc, ad + 4, wd + 4, idesc, 1u);
                        if (stamps && kbi < 16) tc_stamp(g.trace, 40 + kbi);
                        umma_bf16_pair(acc, ad + 6, wd + 6, idesc, 1u);
                        umma_commit_pair(smem_u32(&bar_w_empty[s]));
                        if (!early_ok) ok = mbar_wait(next_bar, parn, abort_flag, err_word, 2);
                        s = sn; par = parn;
                    }
                    if (!ok) break;
                    if (n + 1 == ne) umma_commit_pair(smem_u32(&bar_a_empty));   // the unit's rows may be replaced
                    umma_commit_pair(smem_u32(&bar_acc_full[ab]));
                    if (stamps) tc_stamp(g.trace, 5 + (i > 0));
                }
            }
        }
    } else {
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        int i = 0;
        for (int u = pair; u < units; u += pairs) {
            VP_UNIT(u, m_pair, nb, ne);
            for (int n = nb; n < ne; ++n, ++i) {
                const int ab = i & 1;
                const int m0 = m_pair * 2 * TC_BM + (int)rank * TC_BM;
                tc_epilogue_tile<EPI_STATS, VP_BN>(g, R, m0, n, q, half, lane, tmem_d + ab * VP_BN, nullptr,
                                                   smem_u32(&bar_acc_full[ab]), (i >> 1) & 1, abort_flag, err_word, i > 0);
                if (lane == 0) mbar_arrive_cluster(pair_map(smem_u32(&bar_acc_empty[ab]), 0));
                if (threadIdx.x == 64) tc_stamp(g.trace, 8 + 2 * (i > 0));
            }
        }
    }
#undef VP_UNIT
    tc_fence_before();
    pair_sync();
    if (warp == 1) tmem_dealloc_pair(tmem_d, 512);
    if (threadIdx.x == 0) tc_stamp(g.trace, 11);
}

// ------------------------------------------------------------------ host side
template <int EPI, int BN>
inline cudaError_t tc_pair_set_smem() {
    return cudaFuncSetAttribute(k_gemm_tc_pair<EPI, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TcPairCfg<BN, EPI != EPI_STATS>::SMEM);
}
inline cudaError_t tc_pair_init() {
    cudaError_t e = tc_pair_set_smem<EPI_QKV, 256>();
    if (e == cudaSuccess) e = tc_pair_set_smem<EPI_RELU, 256>();
    if (e == cudaSuccess) e = tc_pair_set_smem<EPI_STORE, 256>();
    if (e == cudaSuccess) e = tc_pair_set_smem<EPI_STATS, 256>();
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_vocab_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024);
    return e;
}

// Worth it for wide weight matrices over many rows: the weight half of the ingest is what the pair saves.
inline bool tc_pair_wanted(int epi, int N, int K, int rows_ub) {
    if (epi != EPI_QKV && epi != EPI_RELU && epi != EPI_STORE && epi != EPI_STATS) return false;   // (the GELU variant stays on single-SM tiles)
    return rows_ub >= 4 * 2 * TC_BM && N >= 1024 && N % 128 == 0 && K % TC_BK == 0;
}

template <int EPI, int BN>
inline int tc_pair_launch_one(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, TC_BM);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, BN / 2);
    if (!ta || !tw) return -1;
    const long long tiles_ub = (long long)((g.N + BN - 1) / BN) * ((rows_ub + 2 * TC_BM - 1) / (2 * TC_BM));
    const int grid = 2 * (int)std::min<long long>(tiles_ub, enc.n_sm / 2);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = TcPairCfg<BN, EPI != EPI_STATS>::SMEM; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemm_tc_pair<EPI, BN>, *ta, *tw, g, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("pair launch: ") + cudaGetErrorString(e); return -1; }
    return 0;
}

inline int vocab_pair_launch(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, TC_BM);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, VP_BNH);
    if (!ta || !tw) return -1;
    const long long tiles_ub = (long long)((g.N + VP_BN - 1) / VP_BN) * ((rows_ub + 2 * TC_BM - 1) / (2 * TC_BM));
    const int grid = 2 * (int)std::min<long long>(tiles_ub, enc.n_sm / 2);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = vp_smem(g.K); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_vocab_pair, *ta, *tw, g, enc.err_word, vp_stages(g.K));
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("vocabulary pair launch: ") + cudaGetErrorString(e); return -1; }
    return 0;
}

inline int gemm_tc_pair_launch(TmaEncoder& enc, int epi, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st, int* n_tiles_out) {
    if (!enc.ready) return -1;
    g.one_m_tile = 0;
    switch (epi) {
        case EPI_QKV: return tc_pair_launch_one<EPI_QKV, 256>(enc, g, rows_ub, st);
        case EPI_RELU: return tc_pair_launch_one<EPI_RELU, 256>(enc, g, rows_ub, st);
        case EPI_STORE: return tc_pair_launch_one<EPI_STORE, 256>(enc, g, rows_ub, st);
        case EPI_STATS:
            g.n_tiles = 2 * ((g.N + 255) / 256);
            if (n_tiles_out) *n_tiles_out = g.n_tiles;
            if (g.K <= 512 && vp_stages(g.K) >= 4) return vocab_pair_launch(enc, g, rows_ub, st);
            return tc_pair_launch_one<EPI_STATS, 256>(enc, g, rows_ub, st);
        default: return -2;
    }
}

}  // namespace sd
