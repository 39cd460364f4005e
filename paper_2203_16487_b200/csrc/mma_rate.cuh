// Issue rate of tcgen05.mma with the operands already resident in shared memory (diagnostics).
//
// The tile GEMMs' main loops are fed by TMA; to tell a loop that waits for operands from one that is limited by the
// tensor pipe itself, this kernel takes the loads out: one CTA per SM fills two operand stages once, then one thread
// issues `n_mma` MMAs back to back (alternating between the two stages and two accumulators), commits, and the
// elapsed clocks are divided by the count.  PAIR: the two-SM form (cta_group::2, M = 256 over a cluster of two CTAs).
// bg_stages > 0: meanwhile another thread keeps bg_stages bulk copies of 16 KB each in flight from global memory into a
// separate region of shared memory -- what a TMA producer does to the shared memory the MMAs read from -- and the
// bytes it landed per clock are reported beside the MMA rate.  commit_every > 0: a tcgen05.commit (to a barrier nobody
// waits on; the multicast form for PAIR) after every k-block of four MMAs, as a main loop issues one.  op_stages: how many
// distinct resident operand stages the k-blocks walk (four without the background stream, two with it; walking two to six
// stages measured the same rate: the pipe keeps no operands across MMAs).
#pragma once
#include "gemm_tc_pair.cuh"

namespace sd {

template <int BN, bool PAIR>
__global__ void __launch_bounds__(128, 1) k_mma_rate(int n_mma, long long* __restrict__ out_clocks, int* err_word,
                                                     const uint8_t* __restrict__ bg_src, int bg_stages, long long bg_window, int commit_every, int op_stages) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_done, bar_bg, bar_dummy;   // bar_dummy: target of the in-loop commits (commit_every > 0), never waited on
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ volatile int stop_s;
    constexpr int BNL = PAIR ? BN / 2 : BN;                       // weight rows this CTA holds
    constexpr int A_BYTES = TC_BM * TC_BK * 2, STAGE = A_BYTES + BNL * TC_BK * 2;
    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    uint32_t rank = 0;
    if (PAIR) rank = pair_cta_rank();
    // operands: any finite bit pattern will do for timing
    for (int i = threadIdx.x; i < op_stages * STAGE / 16; i += blockDim.x)
        *reinterpret_cast<uint4*>(smem_raw + (tiles - smem_u32(smem_raw)) + (size_t)i * 16) = make_uint4(0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u);
    if (threadIdx.x == 0) {
        abort_s = 0; stop_s = 0;
        mbar_init(smem_u32(&bar_done), 1);
        mbar_init(smem_u32(&bar_bg), 1);
        mbar_init(smem_u32(&bar_dummy), 1);
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
        // k-blocks of four MMAs (64 K-elements), as the GEMM main loops issue them; optionally one commit per k-block
        int st = 0;                                   // the k-blocks walk op_stages resident operand stages round robin
        for (int kb = 0; kb < n_mma / 4; ++kb) {
            const uint32_t a_src = tiles + st * STAGE, w_src = a_src + A_BYTES;
            if (++st == op_stages) st = 0;
            const uint64_t ad = umma_desc_k_sw128(a_src), wd = umma_desc_k_sw128(w_src);
            const uint32_t acc = tmem_d + ((kb >> 1) & 1) * BN;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {
                if (PAIR) umma_bf16_pair(acc, ad + (uint64_t)(k4 * 2), wd + (uint64_t)(k4 * 2), idesc, kb >= 4 ? 1u : 0u);
                else umma_bf16(acc, ad + (uint64_t)(k4 * 2), wd + (uint64_t)(k4 * 2), idesc, kb >= 4 ? 1u : 0u);
            }
            if (commit_every > 0) {                   // as a main loop does once per k-block, to free the stage
                if (PAIR) umma_commit_pair(smem_u32(&bar_dummy)); else umma_commit(smem_u32(&bar_dummy));
            }
        }
        const long long t1 = clock64();                           // the thread is done issuing
        if (PAIR) umma_commit_pair(smem_u32(&bar_done)); else umma_commit(smem_u32(&bar_done));
        mbar_wait(smem_u32(&bar_done), 0, &abort_s, err_word, 9);
        const long long t2 = clock64();                           // the last MMA has completed
        out_clocks[4 * (blockIdx.x >> (PAIR ? 1 : 0))] = t1 - t0;
        out_clocks[4 * (blockIdx.x >> (PAIR ? 1 : 0)) + 1] = t2 - t0;
        stop_s = 1;
    } else if (PAIR && threadIdx.x == 0) {
        mbar_wait(smem_u32(&bar_done), 0, &abort_s, err_word, 9);  // the multicast commit arrives here too
        stop_s = 1;
    } else if (threadIdx.x == 64 && bg_stages > 0) {
        // background stream into shared memory: batches of bg_stages x 16 KB, the next batch once this one has landed
        const uint32_t dst0 = tiles + op_stages * STAGE, bar = smem_u32(&bar_bg);
        long long off = ((long long)blockIdx.x << 20) % bg_window, batches = 0;
        if (off + (long long)bg_stages * 16384 > bg_window) off = 0;
        uint32_t ph = 0;
        const long long t0 = clock64();
        while (!stop_s && !abort_s) {
            mbar_expect_tx(bar, (uint32_t)bg_stages * 16384u);
            for (int sg = 0; sg < bg_stages; ++sg)
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst0 + sg * 16384), "l"(bg_src + off + (long long)sg * 16384), "r"(16384), "r"(bar) : "memory");
            if (!mbar_wait(bar, ph, &abort_s, err_word, 10)) break;     // bounded; every copy of the batch has landed
            ph ^= 1; ++batches;
            off += (long long)bg_stages * 16384;
            if (off + (long long)bg_stages * 16384 > bg_window) off = 0;
        }
        const long long t1 = clock64();
        if (!PAIR || rank == 0) {
            out_clocks[4 * (blockIdx.x >> (PAIR ? 1 : 0)) + 2] = batches * bg_stages * 16384;
            out_clocks[4 * (blockIdx.x >> (PAIR ? 1 : 0)) + 3] = t1 - t0;
        }
    }
    tc_fence_before();
    if (PAIR) pair_sync(); else __syncthreads();
    if (warp == 1) { if (PAIR) tmem_dealloc_pair(tmem_d, TMEM_COLS); else tmem_dealloc(tmem_d, TMEM_COLS); }
}

// clocks per MMA (issue, completion) averaged over the grid; returns a CUDA error code
template <int BN, bool PAIR>
inline cudaError_t mma_rate_run(int n_sm, int n_mma, long long* d_scratch, int* err_word, cudaStream_t st, double* issue, double* done,
                                const void* bg_src = nullptr, int bg_stages = 0, long long bg_window = 0, double* bg_bytes_per_clock = nullptr,
                                int commit_every = 0, int op_stages = 2) {
    constexpr int BNL = PAIR ? BN / 2 : BN;
    if (bg_stages < 0 || bg_stages > 6 || (bg_stages > 0 && (!bg_src || bg_window < (8ll << 20)))) return cudaErrorInvalidValue;
    if (op_stages < 1) return cudaErrorInvalidValue;
    const int smem = op_stages * (TC_BM * TC_BK * 2 + BNL * TC_BK * 2) + bg_stages * 16384 + 1024;
    if (smem > 232448 - 1024) return cudaErrorInvalidValue;
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
        e = cudaLaunchKernelEx(&cfg, k_mma_rate<BN, PAIR>, n_mma, d_scratch, err_word, (const uint8_t*)bg_src, bg_stages, bg_window, commit_every, op_stages);
        if (e != cudaSuccess) return e;
    }
    std::vector<long long> hbuf(4 * groups);
    e = cudaMemcpyAsync(hbuf.data(), d_scratch, hbuf.size() * 8, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    double a = 0, b = 0, by = 0, cl = 0;
    for (int i = 0; i < groups; ++i) { a += (double)hbuf[4 * i]; b += (double)hbuf[4 * i + 1]; by += (double)hbuf[4 * i + 2]; cl += (double)hbuf[4 * i + 3]; }
    *issue = a / groups / n_mma; *done = b / groups / n_mma;
    if (bg_bytes_per_clock) *bg_bytes_per_clock = (bg_stages > 0 && cl > 0) ? by / cl : 0.0;
    return cudaSuccess;
}

}  // namespace sd
