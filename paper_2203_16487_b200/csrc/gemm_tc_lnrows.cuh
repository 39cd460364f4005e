// Tensor-core GEMM over at most 128 rows with the LayerNorm of its input fused in front:
//     out = epilogue( LayerNorm(x) W^T + bias ),   x fp32 [R <= 128, K <= 512], W bf16 [N, K].
//
// Passes of a few dozen rows (a batch-1..4 verify block, the drafter's first layer, short encoder inputs) are
// chains of small kernels, and a separate LayerNorm launch costs about as much as the GEMM it feeds.  Here one
// CTA per 64 weight rows; the CTAs form clusters of up to 8, and each CTA normalises only the rows rank, rank + C, ...
// of its cluster: its eight epilogue warps read those fp32 rows, compute the statistics (two passes over registers,
// as the stand-alone kernel does) and write the bf16 operand into shared memory in the layout the tensor core reads
// (128-byte rows, 16-byte chunks XOR-swizzled by the row within 8-row groups: what a 128B-swizzled TMA load would
// have produced) -- their own and, with st.async counted on the receiver's mbarrier, every peer's.  (Every CTA of
// the grid normalising all rows itself was tried first and lost to the separate LayerNorm launch: all CTAs queue up
// on the same L2 lines.)  The whole weight tile
// (64 x K) fits the ring and is requested before the programmatic-launch dependency wait, so after the wait the
// kernel is: read rows, normalise, K / 16 MMAs, epilogue.  Rows past the count are left as they are in shared
// memory: they only feed accumulator lanes nobody reads.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

constexpr int LR_BN = 64;                                     // weight rows (output columns) per CTA
constexpr int LR_MAX_KB = 8;                                  // K <= 512
constexpr int LR_A_KB_BYTES = TC_BM * TC_BK * 2;              // 16 KB: 128 rows x 64 columns of the operand
constexpr int LR_W_KB_BYTES = LR_BN * TC_BK * 2;              // 8 KB
constexpr int LR_STG_BYTES = TC_EPI_WARPS * 32 * 32 * 4;      // epilogue transpose buffers
inline size_t lr_smem(int K) { return (size_t)(K / TC_BK) * (LR_A_KB_BYTES + LR_W_KB_BYTES) + LR_STG_BYTES + 1024; }
inline bool lr_supported(int epi, int N, int K, int rows_ub) {
    return rows_ub <= TC_BM && K % TC_BK == 0 && K >= TC_BK && K <= LR_MAX_KB * TC_BK && N % LR_BN == 0 &&
           (epi == EPI_STORE || epi == EPI_RELU || epi == EPI_GELU || epi == EPI_QKV);
}

__device__ __forceinline__ void lr_st_peer16(uint32_t local_addr, uint32_t local_bar, uint32_t rank, uint4 v) {
    uint32_t ra, rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(ra), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(rb) : "memory");
}

struct LnRowsArgs { const float* x; const float* gam; const float* bet; float eps; };

template <int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc_lnrows(const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g, LnRowsArgs ln, int* err_word) {
    const int nkb = g.K / TC_BK, K = g.K;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_w[LR_MAX_KB], bar_a, bar_acc;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t a_base = (smem_u32(smem_raw) + 1023u) & ~1023u, w_base = a_base + nkb * LR_A_KB_BYTES;
    uint8_t* a_ptr = smem_raw + (a_base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* stg = reinterpret_cast<float*>(a_ptr + nkb * (LR_A_KB_BYTES + LR_W_KB_BYTES)) + (warp >= 2 ? warp - 2 : 0) * 1024;
    const int n_tile = blockIdx.x;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < LR_MAX_KB; ++s) mbar_init(smem_u32(&bar_w[s]), 1);
        mbar_init(smem_u32(&bar_a), TC_EPI_WARPS + 1);      // eight local warps + the thread that announces the peers' bytes
        mbar_init(smem_u32(&bar_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_s), 64);
    tc_fence_before();
    tc_cluster_sync();                               // peers' barriers exist before anybody sends (still before the dependency wait)
    tc_fence_after();
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const uint32_t csize = tc_cluster_nctas();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    // weights and LayerNorm parameters before the dependency wait
    if (threadIdx.x == 0) {
        for (int kb = 0; kb < nkb; ++kb) {
            mbar_expect_tx(smem_u32(&bar_w[kb]), LR_W_KB_BYTES);
            tma_load_2d(w_base + kb * LR_W_KB_BYTES, &tmW, kb * TC_BK, n_tile * LR_BN, smem_u32(&bar_w[kb]));
        }
    }
    // a lane owns 16 consecutive columns of a row (two 16-byte operand chunks): columns 16 lane .. 16 lane + 15
    float4 gm[4], bt[4];
    const bool col_ok = lane * 16 < K;
    if (warp >= 2 && col_ok) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            gm[c] = __ldg(reinterpret_cast<const float4*>(ln.gam + lane * 16) + c);
            bt[c] = __ldg(reinterpret_cast<const float4*>(ln.bet + lane * 16) + c);
        }
    }
    pdl_launch_dependents();
    pdl_wait();
    const int R = min(g.rows_static >= 0 ? g.rows_static : *g.n_rows, TC_BM);
    const int own = (R > (int)rank) ? (R - 1 - (int)rank) / (int)csize + 1 : 0;       // rows rank, rank + csize, ... below R
    if (threadIdx.x == 0) mbar_expect_tx(smem_u32(&bar_a), (uint32_t)(R - own) * K * 2);

    if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, LR_BN);
            bool ok = mbar_wait(smem_u32(&bar_a), 0, abort_flag, err_word, 9);      // the normalised rows are in place
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_after();
            for (int kb = 0; kb < nkb && ok; ++kb) {
                ok = mbar_wait(smem_u32(&bar_w[kb]), 0, abort_flag, err_word, 2);
                if (!ok) break;
                const uint64_t ad = umma_desc_k_sw128(a_base + kb * LR_A_KB_BYTES), wd = umma_desc_k_sw128(w_base + kb * LR_W_KB_BYTES);
#pragma unroll
                for (int k4 = 0; k4 < TC_BK / 16; ++k4)
                    umma_bf16(tmem_d, ad + (uint64_t)(k4 * 2), wd + (uint64_t)(k4 * 2), idesc, (kb | k4) ? 1u : 0u);
            }
            umma_commit(smem_u32(&bar_acc));
        }
    } else if (warp >= 2) {
        // ---- LayerNorm of rows (warp - 2), (warp - 2) + 8, ... into the operand tile
        const int w8 = warp - 2;
        const int rstep = TC_EPI_WARPS * (int)csize;                // this CTA's rows: rank + csize * (w8 + 8 i)
        for (int r0 = (int)rank + (int)csize * w8; r0 < R; r0 += 4 * rstep) {   // four rows in flight per warp: one round trip
            float4 v[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = r0 + i * rstep;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    v[i][c] = (r < R && col_ok) ? *(reinterpret_cast<const float4*>(ln.x + (size_t)r * K + lane * 16) + c)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = r0 + i * rstep;
                if (r >= R) break;                                 // warp-uniform
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) s += (v[i][c].x + v[i][c].y) + (v[i][c].z + v[i][c].w);
                const float mu = warp_sum(s) / K;
                float q = 0.f;
                if (col_ok) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const float c0 = v[i][c].x - mu, c1 = v[i][c].y - mu, c2 = v[i][c].z - mu, c3 = v[i][c].w - mu;
                        q += (c0 * c0 + c1 * c1) + (c2 * c2 + c3 * c3);
                    }
                }
                const float rstd = 1.0f / sqrtf(warp_sum(q) / K + ln.eps);
                if (col_ok) {
                    uint32_t pk[8];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        __nv_bfloat162 p0 = __floats2bfloat162_rn((v[i][c].x - mu) * rstd * gm[c].x + bt[c].x, (v[i][c].y - mu) * rstd * gm[c].y + bt[c].y);
                        __nv_bfloat162 p1 = __floats2bfloat162_rn((v[i][c].z - mu) * rstd * gm[c].z + bt[c].z, (v[i][c].w - mu) * rstd * gm[c].w + bt[c].w);
                        pk[c * 2] = *reinterpret_cast<uint32_t*>(&p0); pk[c * 2 + 1] = *reinterpret_cast<uint32_t*>(&p1);
                    }
                    // columns 16 lane .. : k-block lane / 4, 16-byte chunks 2 (lane % 4) and 2 (lane % 4) + 1 of the 128-byte row
                    uint8_t* rowp = a_ptr + (lane >> 2) * LR_A_KB_BYTES + r * 128;
                    const int c0 = (lane & 3) * 2;
                    uint8_t* q0 = rowp + ((c0 ^ (r & 7)) << 4);
                    uint8_t* q1 = rowp + (((c0 + 1) ^ (r & 7)) << 4);
                    const uint4 v0 = make_uint4(pk[0], pk[1], pk[2], pk[3]), v1 = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    *reinterpret_cast<uint4*>(q0) = v0;
                    *reinterpret_cast<uint4*>(q1) = v1;
                    for (uint32_t rk = 0; rk < csize; ++rk)
                        if (rk != rank) {
                            lr_st_peer16(smem_u32(q0), smem_u32(&bar_a), rk, v0);
                            lr_st_peer16(smem_u32(q1), smem_u32(&bar_a), rk, v1);
                        }
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these stores are read by the tensor core (async proxy)
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_a));
        // ---- epilogue of the single tile
        tc_epilogue_tile<EPI, LR_BN>(g, R, 0, n_tile, warp & 3, (warp - 2) >> 2, lane, tmem_d, stg, smem_u32(&bar_acc), 0,
                                     abort_flag, err_word, false);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, 64);
}

template <int EPI>
inline int lr_launch_one(TmaEncoder& enc, GemmArgs<bf16>& g, const LnRowsArgs& ln, cudaStream_t st) {
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, LR_BN);
    if (!tw) return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.N / LR_BN); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = lr_smem(g.K); cfg.stream = st;
    const int ctas = g.N / LR_BN;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ctas % 8 == 0 ? 8 : (ctas % 4 == 0 ? 4 : (ctas % 2 == 0 ? 2 : 1));
    attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemm_tc_lnrows<EPI>, *tw, g, ln, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("launch (LayerNorm rows): ") + cudaGetErrorString(e); return -1; }
    return 0;
}
inline cudaError_t lr_init() {
    const int bytes = (int)lr_smem(LR_MAX_KB * TC_BK);
    cudaError_t e = cudaFuncSetAttribute(k_gemm_tc_lnrows<EPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc_lnrows<EPI_RELU>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc_lnrows<EPI_GELU>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc_lnrows<EPI_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}
inline int lr_launch(TmaEncoder& enc, int epi, GemmArgs<bf16>& g, const LnRowsArgs& ln, cudaStream_t st) {
    if (!enc.ready) return -1;
    switch (epi) {
        case EPI_STORE: return lr_launch_one<EPI_STORE>(enc, g, ln, st);
        case EPI_RELU: return lr_launch_one<EPI_RELU>(enc, g, ln, st);
        case EPI_GELU: return lr_launch_one<EPI_GELU>(enc, g, ln, st);
        case EPI_QKV: return lr_launch_one<EPI_QKV>(enc, g, ln, st);
        default: return -2;
    }
}

}  // namespace sd
