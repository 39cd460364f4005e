// Issue rate of tcgen05.mma with the operands already resident in shared memory (diagnostics).
//
// The tile GEMMs' main loops are fed by TMA; to tell a loop that waits for operands from one that is limited by the
// tensor pipe itself, this kernel takes the loads out: one CTA per SM fills two operand stages once, then one thread
// issues `n_mma` MMAs back to back (alternating between the two stages and two accumulators), commits, and the
// elapsed clocks are divided by the count.  PAIR: the two-SM form (cta_group::2, M = 256 over a cluster of two CTAs).
#pragma once
#include "gemm_tc_pair.cuh"

namespace sd {

template <int BN, bool PAIR>
__global__ void __launch_bounds__(128, 1) k_mma_rate(int n_mma, long long* __restrict__ out_clocks, int* err_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_done;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    constexpr int BNL = PAIR ? BN / 2 : BN;                       // weight rows this CTA holds
    constexpr int A_BYTES = TC_BM * TC_BK * 2, STAGE = A_BYTES + BNL * TC_BK * 2;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    uint32_t rank = 0;
    if (PAIR) rank = pair_cta_rank();
    // operands: any finite bit pattern will do for timing
    for (int i = threadIdx.x; i < 2 * STAGE / 16; i += blockDim.x)
        *reinterpret_cast<uint4*>(smem_raw + (tiles - smem_u32(smem_raw)) + (size_t)i * 16) = make_uint4(0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u);
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar_done), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);
    if (warp == 1) { if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_s), TMEM_COLS); else tmem_alloc(smem_u32(&tmem_base_s), TMEM_COLS); }
    tc_fence_before();
    if (PAIR) pair_sync(); else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    if (threadIdx.x == 0 && (!PAIR || rank == 0)) {
        constexpr uint32_t idesc = umma_idesc_bf16(PAIR ? 2 * TC_BM : TC_BM, BN);
        const long long t0 = clock64();
        for (int i = 0; i < n_mma; ++i) {
            const uint32_t a_src = tiles + (i & 1) * STAGE, w_src = a_src + A_BYTES;
            const uint64_t ad = umma_desc_k_sw128(a_src) + (uint64_t)((i >> 1) & 3) * 2, wd = umma_desc_k_sw128(w_src) + (uint64_t)((i >> 1) & 3) * 2;
            const uint32_t acc = tmem_d + ((i >> 3) & 1) * BN;
            if (PAIR) umma_bf16_pair(acc, ad, wd, idesc, i >= 16 ? 1u : 0u); else umma_bf16(acc, ad, wd, idesc, i >= 16 ? 1u : 0u);
        }
        const long long t1 = clock64();                           // the thread is done issuing
        if (PAIR) umma_commit_pair(smem_u32(&bar_done)); else umma_commit(smem_u32(&bar_done));
        mbar_wait(smem_u32(&bar_done), 0, &abort_s, err_word, 9);
        const long long t2 = clock64();                           // the last MMA has completed
        out_clocks[2 * (blockIdx.x >> (PAIR ? 1 : 0))] = t1 - t0;
        out_clocks[2 * (blockIdx.x >> (PAIR ? 1 : 0)) + 1] = t2 - t0;
    } else if (PAIR && threadIdx.x == 0) {
        mbar_wait(smem_u32(&bar_done), 0, &abort_s, err_word, 9);  // the multicast commit arrives here too
    }
    tc_fence_before();
    if (PAIR) pair_sync(); else __syncthreads();
    if (warp == 1) { if (PAIR) tmem_dealloc_pair(tmem_d, TMEM_COLS); else tmem_dealloc(tmem_d, TMEM_COLS); }
}

// clocks per MMA (issue, completion) averaged over the grid; returns a CUDA error code
template <int BN, bool PAIR>
inline cudaError_t mma_rate_run(int n_sm, int n_mma, long long* d_scratch, int* err_word, cudaStream_t st, double* issue, double* done) {
    constexpr int BNL = PAIR ? BN / 2 : BN;
    const int smem = 2 * (TC_BM * TC_BK * 2 + BNL * TC_BK * 2) + 1024;
    cudaError_t e = cudaFuncSetAttribute(k_mma_rate<BN, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int ctas = PAIR ? (n_sm / 2) * 2 : n_sm, groups = PAIR ? ctas / 2 : ctas;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = PAIR ? 1 : 0;
    for (int rep = 0; rep < 2; ++rep) {                           // the second run is the one that is read
        e = cudaLaunchKernelEx(&cfg, k_mma_rate<BN, PAIR>, n_mma, d_scratch, err_word);
        if (e != cudaSuccess) return e;
    }
    std::vector<long long> hbuf(2 * groups);
    e = cudaMemcpyAsync(hbuf.data(), d_scratch, hbuf.size() * 8, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    double a = 0, b = 0;
    for (int i = 0; i < groups; ++i) { a += (double)hbuf[2 * i]; b += (double)hbuf[2 * i + 1]; }
    *issue = a / groups / n_mma; *done = b / groups / n_mma;
    return cudaSuccess;
}

}  // namespace sd
