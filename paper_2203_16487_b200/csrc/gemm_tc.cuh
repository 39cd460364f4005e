// Tensor-core GEMM for sm_100a:  C[r, n] = sum_k A[r, k] * W[n, k]  (bf16 operands, fp32 accumulate).
//
//   * operands are staged by TMA (cp.async.bulk.tensor, 128-byte swizzle) into a ring of shared
//     memory stages, 64 K-elements (128 B) per row;
//   * one elected thread issues tcgen05.mma (M = 128 activation rows, N = BN weight rows, K = 16
//     per instruction) with the accumulator in tensor memory;
//   * four epilogue warps read the accumulator back with tcgen05.ld (one TMEM lane = one output
//     row per thread) and apply the fused epilogue: bias / ReLU / residual add / fp32 store / the
//     per-row vocabulary statistics that replace the logits tensor.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, warps 2..9 = epilogue
// (two warps per TMEM lane quadrant, each taking half of the tile's columns).
// Every mbarrier wait is bounded; on a timeout the CTA flags an error word in global memory,
// stops waiting everywhere, still releases its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <map>
#include <string>
#include <tuple>

#include "kernels.cuh"

namespace sd {

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait: gives up after ~2e8 clocks, raises the CTA-wide abort flag and the global error word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* err_word,
                                          int code) {
    if (*abort_flag) return false;
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > 200000000LL) {
            *abort_flag = 1;
            atomicExch(err_word, code);
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile, rows of 128 B, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                             // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                             // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tc_stamp(long long* trace, int slot) {
    if (trace && blockIdx.x == 0) { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); trace[slot] = t; }
}
constexpr int TC_BM = 128, TC_BK = 64;
constexpr int TC_EPI_WARPS = 8;                      // two per TMEM lane quadrant: each takes half the columns
constexpr int TC_THREADS = (2 + TC_EPI_WARPS) * 32;  // + TMA warp + MMA warp
template <int BN> struct TcCfg {
    static constexpr int STAGES = BN >= 256 ? 4 : (BN >= 128 ? 6 : 8);
    static constexpr int STAGE_BYTES = (TC_BM + BN) * TC_BK * 2;
    static constexpr int STG_BYTES = TC_EPI_WARPS * 32 * 32 * 4;      // per-warp 32 x 32 fp32 transpose buffers
    static constexpr int SMEM = STAGES * STAGE_BYTES + STG_BYTES + 1024;
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;      // two accumulators
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// CW consecutive fp32 columns (CW = 16 or 32) of this thread's TMEM lane.
template <int CW>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float* v) {
    if constexpr (CW == 32) { tmem_ld32(taddr, v); return; }
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Persistent kernel: CTA c works on tiles c, c + gridDim.x, ... (row tile fastest, so CTAs running
// together share one weight tile).  The TMA ring and the two TMEM accumulators run across tiles, so the
// epilogue of tile i overlaps the loads and MMAs of tile i + 1.
template <int EPI, int BN>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g,
          int* err_word) {
    using Cfg = TcCfg<BN>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int HALF = BN / 2;                     // columns per epilogue warp
    if (threadIdx.x == 0) tc_stamp(g.trace, 0);
    constexpr int CW = HALF >= 32 ? 32 : 16;         // columns per TMEM read
    // With a row count known on the host the kernel can set itself up and start streaming weight tiles before
    // its predecessor has finished (programmatic dependent launch); a device-side count must be waited for.
    const bool early = g.rows_static >= 0;
    if (!early) pdl_wait();
    const int R = early ? g.rows_static : *g.n_rows;
    const int m_tiles = (R + TC_BM - 1) / TC_BM, n_tiles = (g.N + BN - 1) / BN;
    const int total = m_tiles * n_tiles;
    if ((int)blockIdx.x >= total) return;            // whole CTA leaves before touching barriers or tensor memory

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[STAGES], bar_empty[STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = g.K / TC_BK;
    float* stg = reinterpret_cast<float*>(smem_raw + (tiles - smem_u32(smem_raw)) + STAGES * Cfg::STAGE_BYTES) + (warp >= 2 ? warp - 2 : 0) * 1024;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&bar_acc_full[i]), 1); mbar_init(smem_u32(&bar_acc_empty[i]), TC_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0) tc_stamp(g.trace, 1);
    int pre = 0;                                       // stages whose weight half was requested before the wait
    if (early) {
        if (threadIdx.x == 0) {
            const int n0 = ((int)blockIdx.x / m_tiles) * BN;
            for (; pre < STAGES && pre < nkb; ++pre) {
                const uint32_t bar = smem_u32(&bar_full[pre]);
                mbar_expect_tx(bar, Cfg::STAGE_BYTES);
                tma_load_2d(tiles + pre * Cfg::STAGE_BYTES + TC_BM * TC_BK * 2, &tmW, pre * TC_BK, n0, bar);
            }
        }
        pdl_launch_dependents();
        pdl_wait();                                    // activations, residual and outputs belong to the predecessors until here
    }

    if (warp == 0) {
        if (lane == 0) {
            int kbi = 0;                               // k-blocks issued so far, over all tiles
            for (int t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x) {
                const int m0 = (t % m_tiles) * TC_BM, n0 = (t / m_tiles) * BN;
                for (int kb = 0; kb < nkb; ++kb, ++kbi) {
                    const int s = kbi % STAGES;
                    if (kbi >= STAGES) mbar_wait(smem_u32(&bar_empty[s]), ((kbi / STAGES) - 1) & 1, abort_flag, err_word, 1);
                    if (*abort_flag) break;
                    const uint32_t a_dst = tiles + s * Cfg::STAGE_BYTES, w_dst = a_dst + TC_BM * TC_BK * 2;
                    const uint32_t bar = smem_u32(&bar_full[s]);
                    if (kbi >= pre) {
                        mbar_expect_tx(bar, Cfg::STAGE_BYTES);
                        tma_load_2d(w_dst, &tmW, kb * TC_BK, n0, bar);
                    }
                    tma_load_2d(a_dst, &tmA, kb * TC_BK, m0, bar);
                    if (kbi == 0) tc_stamp(g.trace, 2);
                }
            }
            tc_stamp(g.trace, 3);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, BN);
            int kbi = 0, i = 0;
            for (int t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++i) {
                const int ab = i & 1;
                if (i >= 2) mbar_wait(smem_u32(&bar_acc_empty[ab]), ((i >> 1) - 1) & 1, abort_flag, err_word, 4);
                tc_fence_after();
                const uint32_t acc = tmem_d + ab * BN;
                for (int kb = 0; kb < nkb; ++kb, ++kbi) {
                    const int s = kbi % STAGES;
                    mbar_wait(smem_u32(&bar_full[s]), (kbi / STAGES) & 1, abort_flag, err_word, 2);
                    if (*abort_flag) break;
                    if (kbi == 0) tc_stamp(g.trace, 4);
                    tc_fence_after();
                    const uint32_t a_src = tiles + s * Cfg::STAGE_BYTES, w_src = a_src + TC_BM * TC_BK * 2;
                    const uint64_t ad = umma_desc_k_sw128(a_src), wd = umma_desc_k_sw128(w_src);
#pragma unroll
                    for (int k4 = 0; k4 < TC_BK / 16; ++k4)      // +32 bytes along K per instruction: 2 address units
                        umma_bf16(acc, ad + (uint64_t)(k4 * 2), wd + (uint64_t)(k4 * 2), idesc, (kb | k4) ? 1u : 0u);
                    umma_commit(smem_u32(&bar_empty[s]));        // stage reusable once these MMAs have read it
                }
                umma_commit(smem_u32(&bar_acc_full[ab]));        // accumulator of this tile complete
                tc_stamp(g.trace, 5 + (i > 0));
            }
        }
    } else {
        const int q = warp & 3;                                  // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;                        // which half of the tile's columns
        int i = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++i) {
            const int ab = i & 1;
            const int m0 = (t % m_tiles) * TC_BM, n_tile = t / m_tiles, n0 = n_tile * BN + half * HALF;
            const int r = m0 + q * 32 + lane;
            const bool live = mbar_wait(smem_u32(&bar_acc_full[ab]), (i >> 1) & 1, abort_flag, err_word, 3);
            if (threadIdx.x == 64) tc_stamp(g.trace, 7 + 2 * (i > 0));
            tc_fence_after();
            const uint32_t trow = tmem_d + ((uint32_t)(q * 32) << 16) + ab * BN + half * HALF;
            const bool warp_live = live && (m0 + q * 32 < R);    // warp-uniform: any live row in this quadrant
            float v[CW];
            long long my_cache_row = 0;                          // EPI_QKV: cache row of this lane's output row
            if (EPI == EPI_QKV && warp_live && r < R) my_cache_row = (long long)g.pg.row(g.seq[r], g.pos[r]);
            if (warp_live && EPI == EPI_STATS) {
                const float ld = (g.ld && r < R) ? g.ld[r] : CUDART_INF_F;
                const int id = (g.ld_id && r < R) ? g.ld_id[r] : -1;
                // four interleaved running statistics shorten the dependent chain; merged in column order
                float mx[4]; int arg[4]; int cnt = 0;
#pragma unroll
                for (int u = 0; u < 4; ++u) { mx[u] = -CUDART_INF_F; arg[u] = 0x7fffffff; }
                for (int c = 0; c < HALF / CW; ++c) {
                    tmem_ld<CW>(trow + c * CW, v);
#pragma unroll
                    for (int j = 0; j < CW; ++j) {
                        const int n = n0 + c * CW + j;
                        const float x = (n >= g.N) ? -CUDART_INF_F : ((n == id) ? ld : v[j]);   // draft column: pre-pass value
                        if (x > mx[j & 3]) { mx[j & 3] = x; arg[j & 3] = n; }
                        cnt += (x > ld) ? 1 : 0;
                    }
                }
                RowPart p; p.mx = mx[0]; p.arg = arg[0]; p.sum = 0.f; p.cnt = cnt;
#pragma unroll
                for (int u = 1; u < 4; ++u)
                    if (mx[u] > p.mx || (mx[u] == p.mx && arg[u] < p.arg)) { p.mx = mx[u]; p.arg = arg[u]; }
                if (g.want_sum) {
                    for (int c = 0; c < HALF / CW; ++c) {
                        tmem_ld<CW>(trow + c * CW, v);
#pragma unroll
                        for (int j = 0; j < CW; ++j) {
                            const int n = n0 + c * CW + j;
                            if (n < g.N) p.sum += expf(((n == id) ? ld : v[j]) - p.mx);
                        }
                    }
                }
                if (r < R) g.part[(size_t)r * g.n_tiles + n_tile * 2 + half] = p;
            } else if (warp_live) {
                for (int c = 0; c < HALF / CW; ++c) {
                    tmem_ld<CW>(trow + c * CW, v);
                    const int nb = n0 + c * CW;
                    if (g.bias) {
#pragma unroll
                        for (int j = 0; j < CW; ++j) v[j] += (nb + j < g.N) ? __ldg(g.bias + nb + j) : 0.f;
                    }
                    if (EPI == EPI_RELU) {
#pragma unroll
                        for (int j = 0; j < CW; ++j) v[j] = fmaxf(v[j], 0.f);
                    }
                    const bool full = nb + CW <= g.N;
                    const bool bf_out = (EPI == EPI_STORE || EPI == EPI_RELU || EPI == EPI_QKV);
                    if (CW == 32 && full && (bf_out ? (g.ldo % 2 == 0 && (EPI != EPI_QKV || g.kv_d % 32 == 0)) : true)) {
                        // Transpose through shared memory: a thread owns one output ROW in tensor memory, but global
                        // memory wants a warp to touch one row at a time.  The 32 x 32 block is written row-wise with
                        // its 16-byte chunks XOR-swizzled by the row, then read back one row per warp instruction.
                        float* srow = stg + lane * 32;
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4)
                            *reinterpret_cast<float4*>(srow + ((j4 ^ (lane & 7)) << 2)) = make_float4(v[j4 * 4], v[j4 * 4 + 1], v[j4 * 4 + 2], v[j4 * 4 + 3]);
                        __syncwarp();
                        const int rbase = m0 + q * 32;
                        if (!bf_out) {
                            float* gcol = g.resid + nb + lane;
#pragma unroll
                            for (int r8 = 0; r8 < 32; r8 += 8) {
                                float xin[8];
                                if (EPI == EPI_RESID) {
#pragma unroll
                                    for (int u = 0; u < 8; ++u) xin[u] = (rbase + r8 + u < R) ? gcol[(size_t)(rbase + r8 + u) * g.N] : 0.f;
                                }
#pragma unroll
                                for (int u = 0; u < 8; ++u) {
                                    const int rr = r8 + u;
                                    float val = stg[rr * 32 + ((((lane >> 2) ^ (rr & 7))) << 2) + (lane & 3)];
                                    if (EPI == EPI_RESID) val += xin[u];
                                    if (rbase + rr < R) gcol[(size_t)(rbase + rr) * g.N] = val;
                                }
                            }
                        } else {
                            const int hl = lane >> 4, cl = lane & 15;           // half-warp per row, two columns per lane
#pragma unroll 4
                            for (int r2 = 0; r2 < 32; r2 += 2) {
                                const int rr = r2 + hl, gr = rbase + rr;
                                const long long row_of = (EPI == EPI_QKV) ? __shfl_sync(0xffffffffu, my_cache_row, rr) : 0;
                                const float2 pv = *reinterpret_cast<const float2*>(stg + rr * 32 + (((cl >> 1) ^ (rr & 7)) << 2) + (cl & 1) * 2);
                                if (gr < R) {
                                    bf16* o = g.out + (size_t)gr * g.ldo + nb;
                                    if (EPI == EPI_QKV && nb >= g.kv_d) {          // K or V part: straight into the paged cache
                                        const size_t row = (size_t)row_of;
                                        o = (nb < 2 * g.kv_d ? g.kc + row * g.kv_d + (nb - g.kv_d) : g.vc + row * g.kv_d + (nb - 2 * g.kv_d));
                                    }
                                    __nv_bfloat162 b2;
                                    b2.x = __float2bfloat16_rn(pv.x); b2.y = __float2bfloat16_rn(pv.y);
                                    *reinterpret_cast<__nv_bfloat162*>(o + cl * 2) = b2;
                                }
                            }
                        }
                        __syncwarp();
                        continue;
                    }
                    if (r >= R) continue;
                    if (bf_out) {
                        bf16* o = g.out + (size_t)r * g.ldo + nb;
                        if (EPI == EPI_QKV && nb >= g.kv_d) {
                            const size_t row = g.pg.row(g.seq[r], g.pos[r]);
                            o = (nb < 2 * g.kv_d ? g.kc + row * g.kv_d + (nb - g.kv_d) : g.vc + row * g.kv_d + (nb - 2 * g.kv_d));
                        }
                        for (int j = 0; j < CW; ++j)
                            if (nb + j < g.N) o[j] = __float2bfloat16_rn(v[j]);
                    } else {
                        float* o = g.resid + (size_t)r * g.N + nb;
                        for (int j = 0; j < CW; ++j)
                            if (nb + j < g.N) o[j] = (EPI == EPI_RESID ? o[j] : 0.f) + v[j];
                    }
                }
            }
            // this warp is done with the accumulator: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[ab]));
            if (threadIdx.x == 64) tc_stamp(g.trace, 8 + 2 * (i > 0));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, Cfg::TMEM_COLS);
    if (threadIdx.x == 0) tc_stamp(g.trace, 11);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TmaEncoder {
    bool ready = false;
    std::string err = "not initialised";
    PFN_encodeTiled encode = nullptr;
    int* err_word = nullptr;            // device word the kernels raise on a wait timeout
    int n_sm = 148;
    int force_bn = 0;                   // experiments: 0 = choose, else 32 / 64 / 128 / 256
    bool pdl = true;                    // launch with programmatic stream serialization
    std::map<std::tuple<const void*, long long, int, int, int>, CUtensorMap> cache;

    // 2-D bf16 tensor [rows, K] with row pitch ld elements; box = 64 x box_rows, 128-byte swizzle.
    const CUtensorMap* get(const void* base, long long rows, int K, int ld, int box_rows) {
        auto key = std::make_tuple(base, rows, K, ld, box_rows);
        auto it = cache.find(key);
        if (it != cache.end()) return &it->second;
        CUtensorMap tm;
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
        cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
        cuuint32_t estr[2] = {1, 1};
        CUresult rc = encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (rc != CUDA_SUCCESS) { err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)rc); return nullptr; }
        if (cache.size() > 4096) cache.clear();
        return &(cache[key] = tm);
    }
};

inline bool tc_supported(int N, int K) { return K % TC_BK == 0 && K >= TC_BK && N >= 32; }

template <int EPI, int BN>
inline cudaError_t tc_set_smem() {
    return cudaFuncSetAttribute(k_gemm_tc<EPI, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<BN>::SMEM);
}
template <int EPI>
inline cudaError_t tc_set_smem_all() {
    cudaError_t e = tc_set_smem<EPI, 32>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 64>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 128>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 256>();
    return e;
}

inline int tc_init(TmaEncoder& enc, int* err_word) {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        enc.err = "cannot query the device"; return -1;
    }
    if (major != 10) { enc.err = "device is not sm_100"; return -1; }
    cudaDeviceGetAttribute(&enc.n_sm, cudaDevAttrMultiProcessorCount, dev);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) { enc.err = "cuTensorMapEncodeTiled not found in the driver"; return -1; }
    enc.encode = (PFN_encodeTiled)fn;
    cudaError_t e = tc_set_smem_all<EPI_STORE>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_RELU>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_RESID>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_F32>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_QKV>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 128>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 256>();
    if (e != cudaSuccess) { enc.err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return -1; }
    enc.err_word = err_word;
    enc.ready = true;
    enc.err.clear();
    return 0;
}

template <int EPI, int BN>
inline int tc_launch_one(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, TC_BM);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, BN);
    if (!ta || !tw) return -1;
    const long long tiles_ub = (long long)((g.N + BN - 1) / BN) * ((rows_ub + TC_BM - 1) / TC_BM);
    const int grid = (int)std::min<long long>(tiles_ub, enc.n_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = TcCfg<BN>::SMEM; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemm_tc<EPI, BN>, *ta, *tw, g, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("launch: ") + cudaGetErrorString(e); return -1; }
    return 0;
}

template <int EPI>
inline int tc_launch_bn(TmaEncoder& enc, int bn, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    switch (bn) {
        case 256: return tc_launch_one<EPI, 256>(enc, g, rows_ub, st);
        case 128: return tc_launch_one<EPI, 128>(enc, g, rows_ub, st);
        case 64: return tc_launch_one<EPI, 64>(enc, g, rows_ub, st);
        default: return tc_launch_one<EPI, 32>(enc, g, rows_ub, st);
    }
}

// Tile width: a CTA ingests (128 + BN) * K * 2 bytes per tile and the SMs are ingest-bound long before
// they are math-bound, so pick the BN that minimises waves * (128 + BN); ties go to the narrower tile
// (more tiles per CTA, so more of the epilogue overlaps the next tile's loads).
inline int tc_pick_bn(int N, int rows_ub, int n_sm) {
    const int m_tiles = (rows_ub + TC_BM - 1) / TC_BM;
    const int cand[4] = {256, 128, 64, 32};
    int best = 32; long long best_cost = -1;
    for (int i = 0; i < 4; ++i) {
        const int bn = cand[i];
        if (bn > N && bn != 32) continue;
        if (bn == 32 && m_tiles > 1) continue;                 // the narrow tile only pays for a single row tile
        const long long tiles = (long long)((N + bn - 1) / bn) * m_tiles;
        const long long cost = ((tiles + n_sm - 1) / n_sm) * (TC_BM + bn);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

inline int gemm_tc_launch(TmaEncoder& enc, int epi, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st, int* n_tiles_out) {
    if (!enc.ready) return -1;
    if (epi == EPI_STATS) {
        if (g.N < 128) return -2;
        const bool wide = rows_ub > 4 * TC_BM && g.N >= 256;    // many row tiles: wider tiles halve the re-reads of A
        const int bn = wide ? 256 : 128;
        g.n_tiles = 2 * ((g.N + bn - 1) / bn);                   // two column halves per tile
        if (n_tiles_out) *n_tiles_out = g.n_tiles;
        return wide ? tc_launch_one<EPI_STATS, 256>(enc, g, rows_ub, st) : tc_launch_one<EPI_STATS, 128>(enc, g, rows_ub, st);
    }
    const int bn = (enc.force_bn && enc.force_bn <= g.N) ? enc.force_bn : tc_pick_bn(g.N, rows_ub, enc.n_sm);
    switch (epi) {
        case EPI_STORE: return tc_launch_bn<EPI_STORE>(enc, bn, g, rows_ub, st);
        case EPI_RELU: return tc_launch_bn<EPI_RELU>(enc, bn, g, rows_ub, st);
        case EPI_RESID: return tc_launch_bn<EPI_RESID>(enc, bn, g, rows_ub, st);
        case EPI_QKV: return tc_launch_bn<EPI_QKV>(enc, bn, g, rows_ub, st);
        default: return tc_launch_bn<EPI_F32>(enc, bn, g, rows_ub, st);
    }
}

}  // namespace sd
