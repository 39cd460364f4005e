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
    if (mbar_try_wait(bar, parity)) return true;      // fast path: no other shared-memory access
    if (*abort_flag) return false;
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
constexpr int TC_BM = 128, TC_BK = 64;
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
    if (trace && blockIdx.x == 0 && (unsigned)slot < 56u) {          // the trace window holds 56 slots
        long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); trace[slot] = t;
    }
}
constexpr int TC_EPI_WARPS = 8;                      // two per TMEM lane quadrant: each takes half the columns
constexpr int TC_THREADS = (2 + TC_EPI_WARPS) * 32;  // + TMA warp + MMA warp
// AR = rows of the activation box a stage holds (the MMA always spans 128 rows; with AR < 128 the rows beyond
// the box are whatever shared memory holds and only feed accumulator lanes that nobody reads).  STG = the
// epilogue needs its transpose buffers.
template <int BN, int AR = 128, bool STG = true, bool LNF = false> struct TcCfg {   // LNF: room for the row statistics
    static constexpr int STAGE_BYTES = (AR + BN) * TC_BK * 2;
    static constexpr int STG_BYTES = STG ? TC_EPI_WARPS * 32 * 32 * 4 : 0;   // per-warp 32 x 32 fp32 transpose buffers
    static_assert(BN >= 128 - AR, "the 128-row MMA read of a short activation box must stay inside its stage");
    static constexpr int FIT = (232448 - 1024 - STG_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = (AR < 128 || !STG ? (FIT > 8 ? 8 : FIT) : (BN > 128 ? 4 : (BN >= 128 ? 6 : 8))) - (LNF ? 1 : 0);
    static constexpr int SMEM = STAGES * STAGE_BYTES + STG_BYTES + 1024;
    static constexpr int TMEM_COLS = 2 * BN <= 32 ? 32 : (2 * BN <= 64 ? 64 : (2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512)));  // two accumulators, power of two
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

// The same loads split in two, so that the next chunk's load runs under this chunk's arithmetic: tmem_ld_issue starts the
// load, tmem_ld_done waits for every load issued so far (tcgen05.wait::ld) and names the registers as in/out operands, so no
// use of them can be scheduled ahead of the wait.
template <int CW>
__device__ __forceinline__ void tmem_ld_issue(uint32_t taddr, uint32_t* r) {
    if constexpr (CW == 32) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
              "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
              "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
              "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
            : "r"(taddr) : "memory");
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
              "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
            : "r"(taddr) : "memory");
    }
}
template <int CW>
__device__ __forceinline__ void tmem_ld_done(uint32_t* r) {
    if constexpr (CW == 32) {
        asm volatile("tcgen05.wait::ld.sync.aligned;"
            : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
              "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
              "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
              "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
            : : "memory");
    } else {
        asm volatile("tcgen05.wait::ld.sync.aligned;"
            : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
              "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
            : : "memory");
    }
}

__device__ __forceinline__ void tc_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t tc_cluster_nctas() {
    uint32_t n;
    asm volatile("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(n));
    return n;
}
// Two floats to shared-memory address `local_addr` of CTA `rank` of this cluster, counted (8 bytes) on the mbarrier at
// `local_bar` of that same CTA: the receiver learns of the data through its own barrier, no cluster-wide fence needed.
__device__ __forceinline__ void tc_st_peer2(uint32_t local_addr, uint32_t local_bar, uint32_t rank, float a, float b) {
    uint32_t ra, rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 ::"r"(ra), "f"(a), "f"(b), "r"(rb) : "memory");
}

// One tile of the epilogue, for one of the eight epilogue warps: q = the TMEM lane quadrant the warp may read,
// half = which half of the tile's BN columns it takes; tmem_acc = the tile's accumulator.  Requests what it can
// before waiting for the accumulator (residual tile, bias, cache rows, draft logits), then reads tensor memory
// chunk by chunk.  The caller hands the accumulator back afterwards.
// LNF (residual epilogue only): per row, the sum and sum of squares of the new residual values over the warp's columns
// are written into EVERY cluster peer's ln_part[row][2 * rank + half] for the fused LayerNorm that follows.
template <int EPI, int BN, bool LNF = false>
__device__ __forceinline__ void tc_epilogue_tile(const GemmArgs<bf16>& g, int R, int m0, int n_tile, int q, int half, int lane,
                                                 uint32_t tmem_acc, float* stg, uint32_t bar_acc_full_addr, uint32_t parity,
                                                 volatile int* abort_flag, int* err_word, bool later_tile,
                                                 float* ln_part = nullptr, uint32_t ln_bar = 0) {
    static_assert(!LNF || (EPI == EPI_RESID && BN <= 128 && BN % 64 == 0), "fused LayerNorm: residual epilogue, 64 or 128 columns");
    constexpr int HALF = BN / 2;                     // columns per epilogue warp
    constexpr int CW = HALF % 32 == 0 ? 32 : 16;     // columns per TMEM read
    constexpr bool bf_out = (EPI == EPI_STORE || EPI == EPI_RELU || EPI == EPI_GELU || EPI == EPI_QKV);
    constexpr int NCH = HALF / CW;                   // column chunks per warp and tile
    // 16-byte accesses after the transpose need aligned rows
    const bool vec_ok = CW == 32 && (bf_out ? (g.ldo % 8 == 0 && (EPI != EPI_QKV || g.kv_d % 32 == 0)) : (g.N % 4 == 0));
    const int n0 = n_tile * BN + half * HALF;
    const int r = m0 + q * 32 + lane;
    const int rbase = m0 + q * 32;
    // EPI_RESID: the residual values of the first two column chunks are requested before the accumulator
    // is awaited, so their latency hides behind the MMAs
    float4 xin[2][8];
    if (EPI == EPI_RESID && vec_ok && rbase < R) {
#pragma unroll
        for (int c = 0; c < (NCH < 2 ? NCH : 2); ++c) {
            const int nb = n0 + c * CW;
            if (nb + CW <= g.N) {
#pragma unroll
                for (int ps = 0; ps < 8; ++ps) {
                    const int gr = rbase + ps * 4 + (lane >> 3);
                    xin[c][ps] = gr < R ? *reinterpret_cast<const float4*>(g.resid + (size_t)gr * g.N + nb + (lane & 7) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
    }
    float ln_s1[8], ln_s2[8];                        // LNF: per pass, sum and sum of squares of row 4 ps + lane / 8 over this lane's columns
#pragma unroll
    for (int ps = 0; ps < 8; ++ps) { ln_s1[ps] = 0.f; ln_s2[ps] = 0.f; }
    // ... and so are this lane's bias columns, its cache row and its draft logit
    float4 bzv[NCH][2];
    if (EPI != EPI_STATS && vec_ok && g.bias) {
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int nb = n0 + c * CW;
            if (nb + CW <= g.N) {
                const float4* bp = reinterpret_cast<const float4*>(g.bias + nb);
                if (bf_out) { bzv[c][0] = __ldg(bp + 2 * (lane & 3)); bzv[c][1] = __ldg(bp + 2 * (lane & 3) + 1); }
                else bzv[c][0] = __ldg(bp + (lane & 7));
            }
        }
    }
    long long my_cache_row = 0;                          // EPI_QKV: cache row of this lane's output row
    if (EPI == EPI_QKV && r < R) my_cache_row = (long long)g.pg.row(g.seq[r], g.pos[r]);
    float ld = CUDART_INF_F; int id = -1;                // EPI_STATS: pre-pass logit and id of the row's draft
    if (EPI == EPI_STATS && r < R) { if (g.ld) ld = g.ld[r]; if (g.ld_id) id = g.ld_id[r]; }
    const bool live = mbar_wait(bar_acc_full_addr, parity, abort_flag, err_word, 3);
    if (threadIdx.x == 64) tc_stamp(g.trace, 7 + 2 * (later_tile ? 1 : 0));
    tc_fence_after();
    const uint32_t trow = tmem_acc + ((uint32_t)(q * 32) << 16) + half * HALF;
    const bool warp_live = live && (m0 + q * 32 < R);    // warp-uniform: any live row in this quadrant
    float v[CW];
    if (warp_live && EPI == EPI_STATS) {
        // four interleaved running statistics shorten the dependent chain; merged in column order
        float mx[4]; int arg[4]; int cnt = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) { mx[u] = -CUDART_INF_F; arg[u] = 0x7fffffff; }
        // the next chunk's tensor-memory load runs under this chunk's comparisons (two register buffers)
        uint32_t vr[2][CW];
        tmem_ld_issue<CW>(trow, vr[0]);
#pragma unroll
        for (int c = 0; c < HALF / CW; ++c) {
            tmem_ld_done<CW>(vr[c & 1]);
            if (c + 1 < HALF / CW) tmem_ld_issue<CW>(trow + (c + 1) * CW, vr[(c + 1) & 1]);
            const int nb = n0 + c * CW;
            if (nb + CW <= g.N && (unsigned)(id - nb) >= (unsigned)CW) {
                // whole chunk inside the vocabulary and without the row's draft column: no per-element checks
#pragma unroll
                for (int j = 0; j < CW; ++j) {
                    const float x = __uint_as_float(vr[c & 1][j]);
                    if (x > mx[j & 3]) { mx[j & 3] = x; arg[j & 3] = nb + j; }
                    cnt += (x > ld) ? 1 : 0;
                }
            } else {
#pragma unroll
                for (int j = 0; j < CW; ++j) {
                    const int n = nb + j;
                    const float x = (n >= g.N) ? -CUDART_INF_F : ((n == id) ? ld : __uint_as_float(vr[c & 1][j]));   // draft column: pre-pass value
                    if (x > mx[j & 3]) { mx[j & 3] = x; arg[j & 3] = n; }
                    cnt += (x > ld) ? 1 : 0;
                }
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
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const int nb = n0 + c * CW;
            if (EPI == EPI_RESID && c >= 2 && vec_ok && nb + CW <= g.N) {      // chunks 0 and 1 were requested before the wait
#pragma unroll
                for (int ps = 0; ps < 8; ++ps) {
                    const int gr = rbase + ps * 4 + (lane >> 3);
                    xin[c & 1][ps] = gr < R ? *reinterpret_cast<const float4*>(g.resid + (size_t)gr * g.N + nb + (lane & 7) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            tmem_ld<CW>(trow + c * CW, v);
            if (CW == 32 && vec_ok && nb + CW <= g.N) {
                // Transpose through shared memory: a thread owns one output ROW in tensor memory, but global
                // memory wants neighbouring lanes on neighbouring addresses.  The 32 x 32 block is written row-wise
                // with its 16-byte chunks XOR-swizzled by the row, then read back 16 bytes of output per lane.
                float* srow = stg + lane * 32;
#pragma unroll
                for (int j4 = 0; j4 < 8; ++j4)
                    *reinterpret_cast<float4*>(srow + ((j4 ^ (lane & 7)) << 2)) = make_float4(v[j4 * 4], v[j4 * 4 + 1], v[j4 * 4 + 2], v[j4 * 4 + 3]);
                __syncwarp();
                if (!bf_out) {
                    // fp32 rows: 8 lanes per row (4 columns each), 4 rows per pass
                    const int l8 = lane & 7, rsub = lane >> 3;
                    const float4 bz = g.bias ? bzv[c][0] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int ps = 0; ps < 8; ++ps) {
                        const int rr = ps * 4 + rsub, gr = rbase + rr;
                        float4 a = *reinterpret_cast<const float4*>(stg + rr * 32 + ((l8 ^ (rr & 7)) << 2));
                        a.x += bz.x; a.y += bz.y; a.z += bz.z; a.w += bz.w;
                        if (EPI == EPI_RESID) { const float4 x = xin[c & 1][ps]; a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w; }
                        if (gr < R) *reinterpret_cast<float4*>(g.resid + (size_t)gr * g.N + nb + l8 * 4) = a;
                        if constexpr (LNF) {
                            ln_s1[ps] += (a.x + a.y) + (a.z + a.w);
                            ln_s2[ps] += (a.x * a.x + a.y * a.y) + (a.z * a.z + a.w * a.w);
                        }
                    }
                } else {
                    // bf16 rows: 4 lanes per row (8 columns = 16 bytes each), 8 rows per pass
                    const int c4 = lane & 3, rsub = lane >> 2;
                    float4 b0 = make_float4(0.f, 0.f, 0.f, 0.f), b1 = b0;
                    if (g.bias) { b0 = bzv[c][0]; b1 = bzv[c][1]; }
#pragma unroll
                    for (int ps = 0; ps < 4; ++ps) {
                        const int rr = ps * 8 + rsub, gr = rbase + rr;
                        const long long row_of = (EPI == EPI_QKV) ? __shfl_sync(0xffffffffu, my_cache_row, rr) : 0;
                        float4 a0 = *reinterpret_cast<const float4*>(stg + rr * 32 + (((2 * c4) ^ (rr & 7)) << 2));
                        float4 a1 = *reinterpret_cast<const float4*>(stg + rr * 32 + (((2 * c4 + 1) ^ (rr & 7)) << 2));
                        a0.x += b0.x; a0.y += b0.y; a0.z += b0.z; a0.w += b0.w;
                        a1.x += b1.x; a1.y += b1.y; a1.z += b1.z; a1.w += b1.w;
                        if (EPI == EPI_RELU) {
                            a0.x = fmaxf(a0.x, 0.f); a0.y = fmaxf(a0.y, 0.f); a0.z = fmaxf(a0.z, 0.f); a0.w = fmaxf(a0.w, 0.f);
                            a1.x = fmaxf(a1.x, 0.f); a1.y = fmaxf(a1.y, 0.f); a1.z = fmaxf(a1.z, 0.f); a1.w = fmaxf(a1.w, 0.f);
                        }
                        if (EPI == EPI_GELU) {
                            a0.x = ffn_act(a0.x, 1); a0.y = ffn_act(a0.y, 1); a0.z = ffn_act(a0.z, 1); a0.w = ffn_act(a0.w, 1);
                            a1.x = ffn_act(a1.x, 1); a1.y = ffn_act(a1.y, 1); a1.z = ffn_act(a1.z, 1); a1.w = ffn_act(a1.w, 1);
                        }
                        if (gr < R) {
                            bf16* o = g.out + (size_t)gr * g.ldo + nb;
                            if (EPI == EPI_QKV && nb >= g.kv_d) {          // K or V part: straight into the paged cache
                                const size_t row = (size_t)row_of;
                                o = (nb < 2 * g.kv_d ? g.kc + row * g.kv_d + (nb - g.kv_d) : g.vc + row * g.kv_d + (nb - 2 * g.kv_d));
                            }
                            __nv_bfloat162 p0 = __floats2bfloat162_rn(a0.x, a0.y), p1 = __floats2bfloat162_rn(a0.z, a0.w);
                            __nv_bfloat162 p2 = __floats2bfloat162_rn(a1.x, a1.y), p3 = __floats2bfloat162_rn(a1.z, a1.w);
                            uint4 pk;
                            pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                            pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
                            *reinterpret_cast<uint4*>(o + c4 * 8) = pk;
                        }
                    }
                }
                __syncwarp();
                continue;
            }
            // ragged or unaligned chunk: one row per thread, element by element
            if (g.bias) {
#pragma unroll
                for (int j = 0; j < CW; ++j) v[j] += (nb + j < g.N) ? __ldg(g.bias + nb + j) : 0.f;
            }
            if (EPI == EPI_RELU || EPI == EPI_GELU) {
#pragma unroll
                for (int j = 0; j < CW; ++j) v[j] = ffn_act(v[j], EPI == EPI_GELU ? 1 : 0);
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
    if constexpr (LNF) {                             // each row's partial statistics into every peer's table; every warp
        const uint32_t nct = tc_cluster_nctas();     // sends (rows past the end send what they have) so the byte count is fixed
#pragma unroll
        for (int ps = 0; ps < 8; ++ps) {
            float s1 = ln_s1[ps], s2 = ln_s2[ps];
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
            if ((lane & 7) == 0) {
                const int rr = ps * 4 + (lane >> 3);
                const uint32_t slot = smem_u32(ln_part + ((q * 32 + rr) * 16 + n_tile * 2 + half) * 2);
                for (uint32_t rk = 0; rk < nct; ++rk) tc_st_peer2(slot, ln_bar, rk, s1, s2);
            }
        }
    }
    tc_fence_before();
    __syncwarp();
}

// Persistent kernel: CTA c works on tiles c, c + gridDim.x, ... (row tile fastest, so CTAs running
// together share one weight tile).  The TMA ring and the two TMEM accumulators run across tiles, so the
// epilogue of tile i overlaps the loads and MMAs of tile i + 1.
//
// LNF (residual epilogue, N = the model width): the LayerNorm that consumes the new residual stream is applied in the
// same kernel.  The CTAs of one row tile form a cluster (N / BN of them, one tile each, column tile = cluster rank);
// each writes per-row sums and sums of squares of its columns into every peer's shared memory (distributed shared
// memory stores), and after one cluster barrier every CTA has the whole row's statistics locally and normalises the values it still holds in registers into
// g.ln_out (bf16).  Sums are added in a fixed order; the variance is E[x^2] - mean^2 in fp32.
template <int EPI, int BN, int AR = 128, bool LNF = false>
__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, GemmArgs<bf16> g,
          int* err_word) {
    using Cfg = TcCfg<BN, AR, EPI != EPI_STATS, LNF>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int A_BYTES = AR * TC_BK * 2;          // activation part of a stage
    if (threadIdx.x == 0) tc_stamp(g.trace, 0);
    // The kernel sets itself up (barriers, tensor memory) and lets its successors start before its predecessor has
    // finished (programmatic dependent launch).  With a row count known on the host, or rows that fit one row tile
    // whatever their count (one_m_tile), it also knows its first tile and starts streaming that tile's weights; a
    // device-side count is read after the wait.  (Requesting the first tile's weights before the wait for those
    // launches too -- tiles numbered column tile fastest, a drain path for CTAs left without a tile -- measured no gain.)
    const bool early = g.rows_static >= 0 || g.one_m_tile;
    int R = g.rows_static >= 0 ? g.rows_static : 0;
    int m_tiles = g.one_m_tile ? 1 : (R + TC_BM - 1) / TC_BM;
    const int n_tiles = (g.N + BN - 1) / BN;
    int total = m_tiles * n_tiles;
    if (g.rows_static >= 0 && (int)blockIdx.x >= total) return;   // (static count) whole CTA leaves before touching barriers or tensor memory

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[STAGES], bar_empty[STAGES], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ __align__(16) float ln_part_s[LNF ? TC_BM * 32 : 1];  // [row][2 * cluster rank + column half][sum, sum of squares]
    __shared__ float ln_mr_s[LNF ? TC_BM * 2 : 1];                   // [row][mean, 1 / std]
    __shared__ __align__(8) uint64_t bar_ln;                         // LNF: counts the peers' statistics as they arrive
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
        tc_stamp(g.trace, 12);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_s), Cfg::TMEM_COLS); if (lane == 0) tc_stamp(g.trace, 13); }
    if constexpr (LNF) {
        if (threadIdx.x == 0) {
            mbar_init(smem_u32(&bar_ln), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            mbar_expect_tx(smem_u32(&bar_ln), tc_cluster_nctas() * TC_BM * 2 * 8);   // 8 bytes per row and column half from every peer
        }
        tc_fence_before();
        tc_cluster_sync();                           // peers' barriers exist before anybody sends (all of this precedes the dependency wait)
    } else {
        tc_fence_before();
        __syncthreads();
    }
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0 && tmem_d != 0xffffffffu) tc_stamp(g.trace, 1);   // (the test pins the stamp behind the read)
    int pre = 0;                                       // stages whose weight half was requested before the wait
    if (early) {
        if (threadIdx.x == 0) {
            const int n0 = (LNF ? (int)blockIdx.x % n_tiles : (int)blockIdx.x / m_tiles) * BN;
            for (; pre < STAGES && pre < nkb; ++pre) {
                const uint32_t bar = smem_u32(&bar_full[pre]);
                mbar_expect_tx(bar, Cfg::STAGE_BYTES);
                tma_load_2d(tiles + pre * Cfg::STAGE_BYTES + A_BYTES, &tmW, pre * TC_BK, n0, bar);
            }
        }
    }
    pdl_launch_dependents();
    pdl_wait();                                        // activations, residual and outputs belong to the predecessors until here
    if (g.rows_static < 0) {
        R = *g.n_rows;
        if (!g.one_m_tile) m_tiles = (R + TC_BM - 1) / TC_BM;
        total = m_tiles * n_tiles;                     // a CTA without a tile walks through its empty loops to the common exit
    }

    if (warp == 0) {
        if (lane == 0) {
            int kbi = 0;                               // k-blocks issued so far, over all tiles
            // ring position kept incrementally and the abort flag read only when a wait gave up: this thread's own
            // instructions are part of every stage's turnaround (freed -> requested again)
            int ps = 0; uint32_t ppar = 0; bool wrapped = false, dead = false;
            for (int t = blockIdx.x; t < total && !dead && !*abort_flag; t += gridDim.x) {
                const int m0 = (LNF ? t / n_tiles : t % m_tiles) * TC_BM, n0 = (LNF ? t % n_tiles : t / m_tiles) * BN;
                for (int kb = 0; kb < nkb; ++kb, ++kbi) {
                    if (wrapped && !mbar_wait(smem_u32(&bar_empty[ps]), ppar, abort_flag, err_word, 1)) { dead = true; break; }
                    const uint32_t a_dst = tiles + ps * Cfg::STAGE_BYTES, w_dst = a_dst + A_BYTES;
                    const uint32_t bar = smem_u32(&bar_full[ps]);
                    if (kbi >= pre) {
                        mbar_expect_tx(bar, Cfg::STAGE_BYTES);
                        tma_load_2d(w_dst, &tmW, kb * TC_BK, n0, bar);
                    }
                    tma_load_2d(a_dst, &tmA, kb * TC_BK, m0, bar);
                    if (++ps == STAGES) { ps = 0; if (wrapped) ppar ^= 1u; wrapped = true; }
                }
            }
            tc_stamp(g.trace, 3);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(TC_BM, BN);
            int kbi = 0, i = 0;
            int s = 0; uint32_t par = 0;                     // ring position of k-block kbi: stage and phase parity, kept incrementally
            const bool stamps = g.trace != nullptr && blockIdx.x == 0;
            for (int t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++i) {
                const int ab = i & 1;
                if (i >= 2) mbar_wait(smem_u32(&bar_acc_empty[ab]), ((i >> 1) - 1) & 1, abort_flag, err_word, 4);
                tc_fence_after();
                const uint32_t acc = tmem_d + ab * BN;
                // The tensor pipe takes one MMA at a time from this thread and the thread stalls in each issue until the
                // pipe accepts it, so whatever the thread does BETWEEN two issues is free while whatever it does between
                // the last MMA of a k-block and the first of the next leaves the pipe idle (measured: ~300 clocks of
                // bookkeeping per MMA throttle the pipe to exactly that).  All bookkeeping for the next k-block -- its
                // ring position, descriptors and the test of its barrier -- therefore sits between this k-block's issues.
                bool ok = mbar_wait(smem_u32(&bar_full[s]), par, abort_flag, err_word, 2);
                if (stamps && kbi == 0) tc_stamp(g.trace, 4);
                for (int kb = 0; kb < nkb && ok; ++kb, ++kbi) {
                    const uint32_t a_src = tiles + s * Cfg::STAGE_BYTES, w_src = a_src + A_BYTES;
                    const uint64_t ad = umma_desc_k_sw128(a_src), wd = umma_desc_k_sw128(w_src);
                    umma_bf16(acc, ad, wd, idesc, kb ? 1u : 0u);
                    int sn = s + 1; uint32_t parn = par;
                    if (sn == STAGES) { sn = 0; parn ^= 1u; }
                    const uint32_t next_bar = smem_u32(&bar_full[sn]);
                    umma_bf16(acc, ad + 2, wd + 2, idesc, 1u);       // +32 bytes along K per instruction: 2 address units
                    const uint32_t early_ok = (kb + 1 < nkb) ? mbar_try_wait(next_bar, parn) : 1u;
                    umma_bf16(acc, ad + 4, wd + 4, idesc, 1u);
                    if (stamps && kbi < 16) tc_stamp(g.trace, 40 + kbi);          // landing cadence of the first k-blocks
                    umma_bf16(acc, ad + 6, wd + 6, idesc, 1u);
                    umma_commit(smem_u32(&bar_empty[s]));        // stage reusable once these MMAs have read it
                    if (!early_ok) ok = mbar_wait(next_bar, parn, abort_flag, err_word, 2);
                    s = sn; par = parn;
                }
                if (!ok) break;
                umma_commit(smem_u32(&bar_acc_full[ab]));        // accumulator of this tile complete
                if (stamps) tc_stamp(g.trace, 5 + (i > 0));
            }
        }
    } else {
        const int q = warp & 3;                                  // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;                        // which half of the tile's columns
        int i = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++i) {
            const int ab = i & 1;
            const int m0 = (LNF ? t / n_tiles : t % m_tiles) * TC_BM, n_tile = LNF ? t % n_tiles : t / m_tiles;
            tc_epilogue_tile<EPI, BN, LNF>(g, R, m0, n_tile, q, half, lane, tmem_d + ab * BN, stg, smem_u32(&bar_acc_full[ab]),
                                           (i >> 1) & 1, abort_flag, err_word, i > 0, ln_part_s, smem_u32(&bar_ln));
            // this warp is done with the accumulator: hand it back to the MMA warp
            if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty[ab]));
            if (threadIdx.x == 64) tc_stamp(g.trace, 8 + 2 * (i > 0));
        }
    }
    if constexpr (LNF) {
        if (warp >= 2 && (int)blockIdx.x < total) {  // (a cluster without a tile exchanged nothing)
            const int q = warp & 3, half = (warp - 2) >> 2;
            const int m0 = ((int)blockIdx.x / n_tiles) * TC_BM, n_tile = (int)blockIdx.x % n_tiles;
            if (half == 0) {                         // one thread per row: the whole row's statistics, slots in a fixed order
                mbar_wait(smem_u32(&bar_ln), 0, abort_flag, err_word, 7);   // every peer's partial sums have landed here
                const int row = q * 32 + lane;
                const float* pr = ln_part_s + row * 32;
                float s1 = 0.f, s2 = 0.f;
                for (int sl = 0; sl < 2 * n_tiles; ++sl) { s1 += pr[sl * 2]; s2 += pr[sl * 2 + 1]; }
                const float mu = s1 / g.N;
                const float var = fmaxf(s2 / g.N - mu * mu, 0.f);
                ln_mr_s[row * 2] = mu;
                ln_mr_s[row * 2 + 1] = 1.0f / sqrtf(var + g.ln_eps);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(TC_EPI_WARPS * 32) : "memory");     // the eight epilogue warps only
            constexpr int HALF = BN / 2, NCH = HALF / 32;
            const int l8 = lane & 7, rsub = lane >> 3, rbase = m0 + q * 32;
            if (rbase < R) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const int nb = n_tile * BN + half * HALF + c * 32;
                    const float4 gm = __ldg(reinterpret_cast<const float4*>(g.ln_g + nb) + l8);
                    const float4 bt = __ldg(reinterpret_cast<const float4*>(g.ln_b + nb) + l8);
#pragma unroll
                    for (int ps = 0; ps < 8; ++ps) {
                        const int rr = ps * 4 + rsub, gr = rbase + rr;
                        const float mu = ln_mr_s[(q * 32 + rr) * 2], rstd = ln_mr_s[(q * 32 + rr) * 2 + 1];
                        if (gr < R) {
                            const float4 a = *reinterpret_cast<const float4*>(g.resid + (size_t)gr * g.N + nb + l8 * 4);   // written by this thread above
                            __nv_bfloat162 p0 = __floats2bfloat162_rn((a.x - mu) * rstd * gm.x + bt.x, (a.y - mu) * rstd * gm.y + bt.y);
                            __nv_bfloat162 p1 = __floats2bfloat162_rn((a.z - mu) * rstd * gm.z + bt.z, (a.w - mu) * rstd * gm.w + bt.w);
                            uint2 pk; pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                            *reinterpret_cast<uint2*>(g.ln_out + (size_t)gr * g.N + nb + l8 * 4) = pk;
                        }
                    }
                }
            }
        }
        tc_fence_before();
        __syncthreads();                             // (peers only ever WROTE into this CTA, before the cluster barrier)
    } else {
        tc_fence_before();
        __syncthreads();
    }
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

template <int EPI, int BN, int AR = 128>
inline cudaError_t tc_set_smem() {
    return cudaFuncSetAttribute(k_gemm_tc<EPI, BN, AR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                TcCfg<BN, AR, EPI != EPI_STATS>::SMEM);
}
template <int EPI>
inline cudaError_t tc_set_smem_all() {
    cudaError_t e = tc_set_smem<EPI, 32>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 64>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 128>();
    if (e == cudaSuccess) e = tc_set_smem<EPI, 192>();
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
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_GELU>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_RESID>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_F32>();
    if (e == cudaSuccess) e = tc_set_smem_all<EPI_QKV>();
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc<EPI_RESID, 64, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<64, 128, true, true>::SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_tc<EPI_RESID, 128, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcCfg<128, 128, true, true>::SMEM);
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 128>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 224, 32>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 224, 64>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 224, 128>();
    if (e == cudaSuccess) e = tc_set_smem<EPI_STATS, 256>();
    if (e != cudaSuccess) { enc.err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e); return -1; }
    enc.err_word = err_word;
    enc.ready = true;
    enc.err.clear();
    return 0;
}

template <int EPI, int BN, int AR = 128>
inline int tc_launch_one(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, AR);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, BN);
    if (!ta || !tw) return -1;
    const long long tiles_ub = (long long)((g.N + BN - 1) / BN) * ((rows_ub + TC_BM - 1) / TC_BM);
    const int grid = (int)std::min<long long>(tiles_ub, enc.n_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = TcCfg<BN, AR, EPI != EPI_STATS>::SMEM; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemm_tc<EPI, BN, AR>, *ta, *tw, g, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("launch: ") + cudaGetErrorString(e); return -1; }
    return 0;
}

// Residual GEMM with the following LayerNorm fused (see k_gemm_tc, LNF): one cluster of N / BN CTAs per row tile.
inline bool tc_ln_fusable(int N, int K) { return N % 128 == 0 && N <= 1024 && K % TC_BK == 0 && K >= TC_BK; }
template <int BN>
inline int tc_launch_ln_one(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    const CUtensorMap* ta = enc.get(g.A, rows_ub, g.K, g.lda, TC_BM);
    const CUtensorMap* tw = enc.get(g.W, g.N, g.K, g.K, BN);
    if (!ta || !tw) return -1;
    const int n_tiles = g.N / BN, m_tiles = (rows_ub + TC_BM - 1) / TC_BM;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tiles * m_tiles); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = TcCfg<BN, 128, true, true>::SMEM; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = n_tiles; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = enc.pdl ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_gemm_tc<EPI_RESID, BN, 128, true>, *ta, *tw, g, enc.err_word);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { enc.err = std::string("launch (fused LayerNorm): ") + cudaGetErrorString(e); return -1; }
    return 0;
}
inline int gemm_tc_launch_ln(TmaEncoder& enc, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    if (!enc.ready) return -1;
    g.one_m_tile = 0;
    // 64-wide tiles (clusters of up to 8) while there are few row tiles, 128-wide otherwise and for wide models
    const bool narrow = rows_ub <= 2 * TC_BM && g.N <= 512;
    return narrow ? tc_launch_ln_one<64>(enc, g, rows_ub, st) : tc_launch_ln_one<128>(enc, g, rows_ub, st);
}

template <int EPI>
inline int tc_launch_bn(TmaEncoder& enc, int bn, GemmArgs<bf16>& g, int rows_ub, cudaStream_t st) {
    switch (bn) {
        case 256: return tc_launch_one<EPI, 256>(enc, g, rows_ub, st);
        case 192: return tc_launch_one<EPI, 192>(enc, g, rows_ub, st);
        case 128: return tc_launch_one<EPI, 128>(enc, g, rows_ub, st);
        case 64: return tc_launch_one<EPI, 64>(enc, g, rows_ub, st);
        default: return tc_launch_one<EPI, 32>(enc, g, rows_ub, st);
    }
}

// Tile width: a CTA ingests (128 + BN) * K * 2 bytes per tile and the SMs are ingest-bound long before
// they are math-bound, so pick the BN that minimises waves * (128 + BN); ties go to the narrower tile
// (more tiles per CTA, so more of the epilogue overlaps the next tile's loads).  32-wide tiles are for
// matrices narrower than 64 only: their 16-column epilogue halves cannot use the 16-byte store path, and a
// verify step over 78 rows measured 649 us with them against 399 us with 64-wide tiles.
inline int tc_pick_bn(int N, int rows_ub, int n_sm) {
    const int m_tiles = (rows_ub + TC_BM - 1) / TC_BM;
    if (N < 64) return 32;
    const int cand[4] = {256, 192, 128, 64};
    int best = 64; long long best_cost = -1;
    for (int i = 0; i < 4; ++i) {
        const int bn = cand[i];
        if (bn > N && bn != 64) continue;
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
        int bn = wide ? 256 : 128;
        // One row tile is pure weight streaming: when 128-wide tiles need a second, part-empty wave but 224-wide
        // ones fit in one, every SM streams one equal slice of the matrix (32768 columns = 147 tiles of 224).
        if (rows_ub <= TC_BM && (g.N + 127) / 128 > enc.n_sm && (g.N + 223) / 224 <= enc.n_sm) bn = 224;
        if (enc.force_bn == 128 || enc.force_bn == 256 || (enc.force_bn == 224 && rows_ub <= TC_BM)) bn = enc.force_bn;
        g.n_tiles = 2 * ((g.N + bn - 1) / bn);                   // two column halves per tile
        if (n_tiles_out) *n_tiles_out = g.n_tiles;
        g.one_m_tile = (bn == 224);
        if (bn == 224)      // one tile per CTA: the ring is as deep as shared memory allows, most of it requested up front
            return rows_ub <= 32 ? tc_launch_one<EPI_STATS, 224, 32>(enc, g, rows_ub, st)
                 : rows_ub <= 64 ? tc_launch_one<EPI_STATS, 224, 64>(enc, g, rows_ub, st)
                                 : tc_launch_one<EPI_STATS, 224, 128>(enc, g, rows_ub, st);
        return bn == 256 ? tc_launch_one<EPI_STATS, 256>(enc, g, rows_ub, st) : tc_launch_one<EPI_STATS, 128>(enc, g, rows_ub, st);
    }
    const int fb = enc.force_bn;
    const bool forced = (fb == 32 || fb == 64 || fb == 128 || fb == 192 || fb == 256) && fb <= g.N;
    const int bn = forced ? fb : tc_pick_bn(g.N, rows_ub, enc.n_sm);
    g.one_m_tile = rows_ub <= TC_BM;        // one row tile whatever the device-side count says: set up and prefetch before the wait
    switch (epi) {
        case EPI_STORE: return tc_launch_bn<EPI_STORE>(enc, bn, g, rows_ub, st);
        case EPI_RELU: return tc_launch_bn<EPI_RELU>(enc, bn, g, rows_ub, st);
        case EPI_GELU: return tc_launch_bn<EPI_GELU>(enc, bn, g, rows_ub, st);
        case EPI_RESID: return tc_launch_bn<EPI_RESID>(enc, bn, g, rows_ub, st);
        case EPI_QKV: return tc_launch_bn<EPI_QKV>(enc, bn, g, rows_ub, st);
        default: return tc_launch_bn<EPI_F32>(enc, bn, g, rows_ub, st);
    }
}

}  // namespace sd
