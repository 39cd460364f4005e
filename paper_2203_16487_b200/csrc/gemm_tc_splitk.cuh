// Residual GEMM over a few 128-row tiles with a long reduction (FFN2: K = 4 d), split along K inside a cluster:
//     resid[r, n] += x[r, :] . W[n, :] + bias[n],   x bf16 [R, K], W bf16 [N, K], resid fp32 [R, N],
// for row counts whose tiles x N / 64 x SPLIT CTAs still fit one wave.
//
// With 64-wide column tiles such a GEMM has N / 64 CTAs (8 for d = 512), each walking the whole K: 32 k-blocks at
// the tensor core's 0.35 us per block is what the kernel costs.  Here SPLIT CTAs of a cluster share one column
// tile: each requests its K / SPLIT slice of the weights before the programmatic-launch dependency wait and of the
// activation rows after it (everything resident: at most 8 k-blocks per CTA), accumulates its partial product in
// tensor memory, and the CTAs of rank > 0 send their fp32 partials to the rank-0 CTA's shared memory (st.async,
// counted on its mbarrier; the operand tiles there are dead by then, which a cluster barrier guarantees).  Rank 0
// adds the partials in rank order -- a fixed order, so the result does not depend on timing -- then bias and the
// residual, and stores.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

constexpr int SPK_BN = 64;
constexpr int SPK_MAX_KB = 8;                                  // k-blocks per CTA
constexpr int SPK_A_KB = TC_BM * TC_BK * 2, SPK_W_KB = SPK_BN * TC_BK * 2;
constexpr int SPK_PROW = SPK_BN * 4 + 16;                      // byte pitch of a partial row (16 bytes of padding: conflict-free float4 reads)
constexpr int SPK_PART = TC_BM * SPK_PROW;                     // one peer's partial tile
inline size_t spk_smem(int nkb, int split) {
    const size_t ops = (size_t)nkb * (SPK_A_KB + SPK_W_KB), parts = (size_t)(split - 1) * SPK_PART;
    return (ops > parts ? ops : parts) + 1024;
}
// 4 CTAs per column tile when their K / 4 slices fit (K <= 2048), else 6 (K = 3072: FFN2 of a 768-wide model); more
// partial tiles than 5 would not fit beside each other in rank 0's shared memory
inline int spk_split(int K) {
    for (int s : {4, 6})
        if (K % (s * TC_BK) == 0 && K / (s * TC_BK) <= SPK_MAX_KB) return s;
    return 0;
}
inline bool spk_supported(int N, int K, int rows_ub, int n_sm) {
    const int split = spk_split(K);
    return split != 0 && N % SPK_BN == 0 && K >= 1024 &&
           (long long)((rows_ub + TC_BM - 1) / TC_BM) * (N / SPK_BN) * split <= n_sm;
}

template <int SPLIT>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc_splitk(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g,
                 int* err_word) {
    const int nkb = g.K / TC_BK / SPLIT;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[SPK_MAX_KB], bar_acc, bar_part;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t a_base = (smem_u32(smem_raw) + 1023u) & ~1023u, w_base = a_base + nkb * SPK_A_KB;
    uint8_t* base_ptr = smem_raw + (a_base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int n_tile = blockIdx.x / SPLIT, kb0 = (int)rank * nkb, m0 = blockIdx.y * TC_BM;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < SPK_MAX_KB; ++s) mbar_init(smem_u32(&bar_full[s]), 1);
        mbar_init(smem_u32(&bar_acc), 1);
        mbar_init(smem_u32(&bar_part), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 64);
    tc_fence_before();
    tc_cluster_sync();                               // rank 0's barrier exists before anybody sends
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0) {                          // this CTA's slice of the weights: before the dependency wait
        for (int kb = 0; kb < nkb; ++kb) {
            mbar_expect_tx(smem_u32(&bar_full[kb]), SPK_A_KB + SPK_W_KB);
            tma_load_2d(w_base + kb * SPK_W_KB, &tmW, (kb0 + kb) * TC_BK, n_tile * SPK_BN, smem_u32(&bar_full[kb]));
        }
    }
    pdl_launch_dependents();
    pdl_wait();
    // rows of this CTA's 128-row tile (none: the tile still runs, on zero-filled rows, and stores nothing)
    const int R = min(max((g.rows_static >= 0 ? g.rows_static : *g.n_rows) - m0, 0), TC_BM);
    if (threadIdx.x == 0) {
        for (int kb = 0; kb < nkb; ++kb)
            tma_load_2d(a_base + kb * SPK_A_KB, &tmA, (kb0 + kb) * TC_BK, m0, smem_u32(&bar_full[kb]));
        if (rank == 0) mbar_expect_tx(smem_u32(&bar_part), (uint32_t)(SPLIT - 1) * R * SPK_BN * 4);
    }
    const int q = warp & 3, half = (warp - 2) >> 2, row = q * 32 + lane;
    const int n0 = n_tile * SPK_BN + half * 32;
    // rank 0: residual values and bias of this thread's 32 outputs, requested before the accumulator is ready
    float4 xin[8], bz[8];
    if (warp >= 2 && rank == 0) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            bz[j] = g.bias ? __ldg(reinterpret_cast<const float4*>(g.bias + n0) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
            xin[j] = row < R ? *(reinterpret_cast<const float4*>(g.resid + (size_t)(m0 + row) * g.N + n0) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    bool ok = true;
    if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, SPK_BN);
            for (int kb = 0; kb < nkb && ok; ++kb) {
                ok = mbar_wait(smem_u32(&bar_full[kb]), 0, abort_flag, err_word, 2);
                if (!ok) break;
                tc_fence_after();
                const uint64_t ad = umma_desc_k_sw128(a_base + kb * SPK_A_KB), wd = umma_desc_k_sw128(w_base + kb * SPK_W_KB);
#pragma unroll
                for (int k4 = 0; k4 < TC_BK / 16; ++k4)
                    umma_bf16(tmem_d, ad + (uint64_t)(k4 * 2), wd + (uint64_t)(k4 * 2), idesc, (kb | k4) ? 1u : 0u);
            }
            umma_commit(smem_u32(&bar_acc));
        }
    } else if (warp >= 2) {
        ok = mbar_wait(smem_u32(&bar_acc), 0, abort_flag, err_word, 3);      // this CTA's MMAs are done: its operand tiles are dead
        tc_fence_after();
    }
    // every CTA's operand tiles are dead (rank 0's are about to be overwritten by the partials).  A CTA whose wait
    // gave up still arrives here, so nobody hangs; the error word tells the host.
    __syncwarp();
    tc_cluster_sync();
    if (warp >= 2) {
        float v[32];
        tmem_ld32(tmem_d + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 32), v);
        if (rank != 0) {
            if (row < R) {
                const uint32_t dst = a_base + (rank - 1) * SPK_PART + row * SPK_PROW + half * 128;
                uint32_t ra, rb;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(smem_u32(&bar_part)), "r"(0));
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(dst + j * 16), "r"(0));
                    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                                 ::"r"(ra), "r"(__float_as_uint(v[4 * j])), "r"(__float_as_uint(v[4 * j + 1])),
                                   "r"(__float_as_uint(v[4 * j + 2])), "r"(__float_as_uint(v[4 * j + 3])), "r"(rb) : "memory");
                }
            }
        } else {
            if (ok) ok = mbar_wait(smem_u32(&bar_part), 0, abort_flag, err_word, 10);   // the peers' partials have landed
            if (ok && row < R) {
                const uint8_t* prow = base_ptr + row * SPK_PROW + half * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 a = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
#pragma unroll
                    for (int p = 0; p < SPLIT - 1; ++p) {                                // rank order: fixed summation order
                        const float4 t = *reinterpret_cast<const float4*>(prow + p * SPK_PART + j * 16);
                        a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
                    }
                    a.x += bz[j].x; a.y += bz[j].y; a.z += bz[j].z; a.w += bz[j].w;
                    a.x += xin[j].x; a.y += xin[j].y; a.z += xin[j].z; a.w += xin[j].w;
                    *(reinterpret_cast<float4*>(g.resid + (size_t)(m0 + row) * g.N + n0) + j) = a;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, 64);
}

inline cudaError_t spk_init() {
    cudaError_t e = cudaFuncSetAttribute(k_gemm_tc_splitk<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)spk_smem(SPK_MAX_KB, 4));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc_splitk<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)spk_smem(SPK_MAX_KB, 6));
    return e;
}

inline int spk_launch(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    if (!enc.ready) return -1;
    const int split = spk_split(g.K);
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, TC_BM);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, SPK_BN);
    if (!ta || !tw || split == 0) return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.N / SPK_BN * split, (rows_ub + TC_BM - 1) / TC_BM); cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = spk_smem(g.K / TC_BK / split, split); cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 2 : 1;
    cudaError_t e = split == 4 ? cudaLaunchKernelEx(&cfg, k_gemm_tc_splitk<4>, *ta, *tw, g, enc.err_word)
                               : cudaLaunchKernelEx(&cfg, k_gemm_tc_splitk<6>, *ta, *tw, g, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("launch (split-K): ") + cudaGetErrorString(e); return -1; }
    return 0;
}

}  // namespace sd
