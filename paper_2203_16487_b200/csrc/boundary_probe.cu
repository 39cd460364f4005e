// What does a dependency between two small kernels cost?  A chain of N kernels (G CTAs x 256 threads each, replayed from a
// CUDA graph, every launch programmatic) in which CTA c of link i reads what CTA c + 1 of link i - 1 wrote.  Two ways to wait:
//   mode 0  griddepcontrol.wait: the predecessor GRID has completed and flushed (what the library's kernels do);
//   mode 1  a counter per link: every CTA adds 1 after its stores (fence, atomic), a successor CTA spins (bounded) until
//           the predecessor's counter reaches epoch x G.  A programmatically launched grid starts only after every CTA of
//           its predecessor has started, so the CTAs waited for are always resident: the spin cannot starve them.
// Prints microseconds per link for both, and checks the chain's result (every element = N after one replay).
// Build: nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o boundary_probe boundary_probe.cu
#include <cuda_runtime.h>
#include <cstdio>
#include <vector>

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void k_head(unsigned* epoch, float* buf, int n) {      // plain launch: opens a replay
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) *epoch += 1;
    if (i < n) buf[i] = 0.f;
}

template <int MODE>
__global__ void __launch_bounds__(256) k_link(const float* in, float* out, unsigned* flags, const unsigned* epoch, int idx,
                                              int G, int* err) {
    __shared__ unsigned ep_s;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (MODE == 0) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
    } else {
        if (threadIdx.x == 0) {
            // the epoch was written by the head kernel, which completed before link 1 started (plain dependency)
            const unsigned ep = ld_acquire(epoch);
            ep_s = ep;
            if (idx > 0) {
                const unsigned want = ep * (unsigned)G;
                const long long t0 = clock64();
                while (ld_acquire(flags + idx - 1) < want) {
                    if (*(volatile int*)err) break;                                            // somebody gave up: nobody waits on
                    if (clock64() - t0 > 400000000LL) { atomicExch(err, idx + 1); break; }     // ~0.2 s: give up, report
                }
            } else {
                asm volatile("griddepcontrol.wait;" ::: "memory");      // first link: behind the head kernel
            }
        }
        __syncthreads();
    }
    const int n = G * 256, i = blockIdx.x * 256 + threadIdx.x;
    const float v = in[(i + 256) % n];                                  // written by the next CTA of the predecessor
    out[i] = v + 1.f;
    if (MODE == 1) {
        __syncthreads();
        if (threadIdx.x == 0) { __threadfence(); atomicAdd(flags + idx, 1u); }
    }
}

template <int MODE>
static float run(int N, int G, int reps, bool check) {
    float *a, *b; unsigned *flags, *epoch; int* err;
    const int n = G * 256;
    cudaMalloc(&a, n * 4); cudaMalloc(&b, n * 4); cudaMalloc(&flags, N * 4); cudaMalloc(&epoch, 4); cudaMalloc(&err, 4);
    cudaMemset(flags, 0, N * 4); cudaMemset(epoch, 0, 4); cudaMemset(err, 0, 4);
    cudaStream_t st; cudaStreamCreate(&st);
    cudaGraph_t g; cudaGraphExec_t ex;
    cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal);
    k_head<<<(n + 255) / 256, 256, 0, st>>>(epoch, a, n);
    for (int i = 0; i < N; ++i) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(G); cfg.blockDim = dim3(256); cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        const float* in = (i & 1) ? b : a; float* out = (i & 1) ? a : b;
        cudaLaunchKernelEx(&cfg, k_link<MODE>, in, out, flags, (const unsigned*)epoch, i, G, err);
    }
    cudaStreamEndCapture(st, &g);
    cudaGraphInstantiate(&ex, g, 0);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    for (int w = 0; w < 3; ++w) cudaGraphLaunch(ex, st);
    cudaStreamSynchronize(st);
    cudaEventRecord(e0, st);
    for (int r = 0; r < reps; ++r) cudaGraphLaunch(ex, st);
    cudaEventRecord(e1, st);
    cudaStreamSynchronize(st);
    float ms = 0.f; cudaEventElapsedTime(&ms, e0, e1);
    if (check) {
        std::vector<float> h(n);
        cudaMemcpy(h.data(), (N & 1) ? b : a, n * 4, cudaMemcpyDeviceToHost);
        int bad = 0, herr = 0;
        for (int i = 0; i < n; ++i) bad += h[i] != (float)N;
        cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
        printf("  mode %d N=%d G=%d: %d wrong elements of %d, error word %d (%s)\n", MODE, N, G, bad, n, herr,
               cudaGetErrorString(cudaGetLastError()));
    }
    cudaGraphExecDestroy(ex); cudaGraphDestroy(g); cudaStreamDestroy(st);
    cudaFree(a); cudaFree(b); cudaFree(flags); cudaFree(epoch); cudaFree(err);
    return ms * 1e3f / reps / N;
}

int main() {
    const int N = 64, reps = 50;
    for (int G : {8, 64, 148, 256}) {
        const float t0 = run<0>(N, G, reps, true), t1 = run<1>(N, G, reps, true);
        printf("G=%3d CTAs: %.2f us per link with griddepcontrol.wait, %.2f us per link with per-link counters\n", G, t0, t1);
    }
    return 0;
}
