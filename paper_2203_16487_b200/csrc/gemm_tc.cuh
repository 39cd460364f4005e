// Tensor-core GEMM interface (tcgen05 / TMEM / TMA).  Placeholder until the kernel lands:
// reports "unavailable" so every contraction runs in the SIMT reference GEMM on the GPU.
#pragma once
#include <string>
#include "kernels.cuh"

namespace sd {

struct TmaEncoder {
    bool ready = false;
    std::string err = "not built";
};

inline bool tc_supported(int, int) { return false; }
inline int tc_init(TmaEncoder&) { return -1; }
inline int gemm_tc_launch(TmaEncoder&, int, GemmArgs<bf16>&, int, cudaStream_t, int*) { return -1; }

}  // namespace sd
