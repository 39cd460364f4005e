// Cost of one exchange round between the CTAs of a thread-block cluster through distributed shared memory
// (diagnostics).  Fusing the kernels of a decoder layer into one cluster kernel replaces kernel boundaries by such
// rounds (every CTA sends its share of a small operand tile to every peer, then all wait for all): this measures
// what a round costs, empty and with data, so the two can be compared.
#pragma once
#include "gemm_tc.cuh"

namespace sd {

// One round: the CTA stores `n16` 16-byte pieces into each peer's receive buffer (plain remote stores), the CTA
// synchronises, one warp arrives (release, cluster scope) on every peer's barrier, one warp waits for all CS arrivals
// (acquire) and releases the rest of the CTA through the CTA barrier.  CS = cluster size.
template <int CS>
__global__ void __launch_bounds__(256, 1) k_cluster_round(int rounds, int n16, long long* __restrict__ out_ns, int* err_word) {
    extern __shared__ __align__(16) uint8_t cr_smem[];         // receive buffer: CS * n16 * 16 bytes
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_s;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar), CS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc_cluster_sync();
    long long t0 = 0;
    if (tid == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    uint32_t phase = 0;
    for (int r = 0; r < rounds; ++r) {
        const uint4 v = make_uint4(r, tid, rank, 0);
        for (int d = 0; d < CS; ++d) {
            uint32_t base;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(base) : "r"(smem_u32(cr_smem)), "r"(d));
            for (int i = tid; i < n16; i += 256)
                asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};"
                             ::"r"(base + (rank * n16 + i) * 16), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
        __syncthreads();
        if (warp == 0) {
            if (lane < CS) {
                uint32_t rb;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(smem_u32(&bar)), "r"(lane));
                asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(rb) : "memory");
            }
            // bounded wait with cluster-scope acquire
            const long long c0 = clock64();
            while (true) {
                uint32_t ok;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(ok) : "r"(smem_u32(&bar)), "r"(phase) : "memory");
                if (ok || abort_s) break;
                if (clock64() - c0 > 200000000LL) { abort_s = 1; atomicExch(err_word, 11); break; }
            }
        }
        phase ^= 1;
        __syncthreads();
    }
    if (tid == 0 && blockIdx.x == 0) {
        long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        out_ns[0] = t1 - t0;
    }
    tc_cluster_sync();                                          // nobody leaves while a peer may still write to it
}

template <int CS>
inline cudaError_t cluster_round_run(int rounds, int bytes_per_cta_per_peer, long long* d_scratch, int* err_word, cudaStream_t st, double* ns_per_round) {
    const int n16 = bytes_per_cta_per_peer / 16;
    const int smem = CS * (n16 > 0 ? n16 : 1) * 16;
    cudaError_t e = cudaFuncSetAttribute(k_cluster_round<CS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess && CS > 8) e = cudaFuncSetAttribute(k_cluster_round<CS>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    for (int rep = 0; rep < 2; ++rep) {
        e = cudaLaunchKernelEx(&cfg, k_cluster_round<CS>, rounds, n16, d_scratch, err_word);
        if (e != cudaSuccess) return e;
    }
    long long ns = 0;
    e = cudaMemcpyAsync(&ns, d_scratch, 8, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    *ns_per_round = (double)ns / rounds;
    return cudaSuccess;
}

}  // namespace sd
