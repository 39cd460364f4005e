// The verifier's decoder stack for one sequence per thread-block cluster (small batches).
//
// At batch 1 a verify block has k+1 <= 32 rows and the step is a pass over 44 MB of layer weights.
// Run as ~50 separate kernels it is bounded by launch boundaries and dependent round trips, not by
// HBM.  Here the six layers run inside ONE kernel: a cluster of 8 CTAs (one per attention head) owns a
// sequence, the CTAs synchronise with the hardware cluster barrier between phases, and each CTA streams
// its eighth of every weight matrix as one contiguous run of 16 KB stages (the weights are re-packed at
// handle creation into exactly the order and fragment layout the warps consume) through a ring in
// shared memory with bulk async copies -- the stream runs ahead across phase boundaries, so the next
// phase's weights arrive while the cluster is still synchronising.
//
// Per layer (6 cluster barriers):
//   A  LN1(x) -> operand rows; Q,K,V of head c (bias, K/V into the paged cache); causal attention of head c
//   B  attention output -> operand rows; out-projection columns 64c..64c+63; x += (owner-exclusive columns)
//   C  LNc(x); cross-attention query of head c; attention over the cached encoder K/V
//   D  cross out-projection; x +=
//   E  LN2(x); FFN1 columns F/8 * c ..; ReLU -> hidden (bf16)
//   F  hidden -> operand rows (K = F); FFN2 columns 64c..; x +=
// Products run on warp-level MMAs (m16n8k16, fp32 accumulate) exactly as in the weight-streaming GEMM:
// a lane's 16 contiguous weight bytes are its B fragments under a fixed permutation of k.
// Activations exchanged between CTAs (x, attention output, hidden) live in global memory (L2) and are
// read with L1-bypassing loads after the cluster barrier.  Every mbarrier wait is bounded.
#pragma once
#include "attention_tc.cuh"
#include "gemm_tc.cuh"
#include "kernels.cuh"

namespace sd {

constexpr int CL_C = 8;              // CTAs per cluster = attention heads of the model
constexpr int CL_STAGE = 16384;      // bytes per weight stage: 8 warps x 4 super-steps x (8 rows x 32 k x 2 B)
constexpr int CL_NS = 5;             // stages in the ring
constexpr int CL_THREADS = 256;
constexpr int CL_M = 32;             // operand rows (k+1 padded)
constexpr int CL_MAX_LAYERS = 8;

struct ClLayer {
    const float *ln1_g, *ln1_b, *lnc_g, *lnc_b, *ln2_g, *ln2_b;
    const float *qkv_b, *o_b, *cq_b, *co_b, *b1, *b2;
    bf16 *kc, *vc;                   // paged self-attention cache of this layer
    const bf16* ckv;                 // cross K|V of the session [B*S_max, 2d]
};
struct ClArgs {
    const unsigned char* wstream;    // packed weights: CTA c reads wstream + c * cta_stride, stage after stage
    size_t cta_stride;
    ClLayer layer[CL_MAX_LAYERS];
    int n_layers;
    float* x;                        // residual rows [B*(k+1), d]
    bf16* att;                       // attention output rows [B*(k+1), d]
    bf16* hbuf;                      // FFN hidden rows [B*(k+1), F]
    const int* len;                  // committed tokens per sequence
    const int* src_len;
    Paged pg;
    int S_max, k1, d, F, max_keys;
    int* err_word;
    long long* trace;                // optional: CTA 0 of cluster 0 records %globaltimer after every phase
};

__host__ __device__ inline int cl_stages_per_layer(int d, int F) { return 3 * (d / 128) + 3 * (d / 128) + (F / (CL_C * 64)) * (d / 128) + F / 128; }
__host__ __device__ inline size_t cl_region_bytes(int F) { return (size_t)CL_M * (F + 32) * 2; }
inline size_t cl_smem_bytes(int F) { return (size_t)CL_NS * CL_STAGE + cl_region_bytes(F) + CL_M * 128 + 128; }
inline int cl_max_keys(int F) { return (int)((cl_region_bytes(F) - 512) / 384) & ~15; }

// ---- packing: wstream[c][layer][stage][warp w][super-step ss][lane (g,t)] = 16 bytes W[n][k .. k+7]
struct ClPackSrc { const bf16 *qkv_w, *o_w, *cq_w, *co_w, *w1, *w2; };
__global__ void k_cl_pack(ClPackSrc s, int layer, int d, int F, uint4* __restrict__ out, size_t cta_stride_u4, int spl) {
    const int KS = d / 128;                                  // k stages for K = d
    const int SA = 3 * KS, SB = KS, SE = (F / (CL_C * 64)) * KS, SF = F / 128;
    const long long per_cta = (long long)spl * 1024;
    for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < per_cta * CL_C; p += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(p / per_cta);
        const long long q = p % per_cta;
        int st = (int)(q / 1024);
        const int in = (int)(q % 1024), blk = in / 32, lane = in % 32, w = blk / 4, ss = blk % 4, g = lane / 4, t = lane % 4;
        const bf16* W; int K, n, kst;
        if (st < SA) { const int gs = st / KS; kst = st % KS; W = s.qkv_w; K = d; n = gs * d + c * 64 + w * 8 + g; }
        else if ((st -= SA) < SB) { kst = st; W = s.o_w; K = d; n = c * 64 + w * 8 + g; }
        else if ((st -= SB) < SB) { kst = st; W = s.cq_w; K = d; n = c * 64 + w * 8 + g; }
        else if ((st -= SB) < SB) { kst = st; W = s.co_w; K = d; n = c * 64 + w * 8 + g; }
        else if ((st -= SB) < SE) { const int gs = st / KS; kst = st % KS; W = s.w1; K = d; n = c * (F / CL_C) + gs * 64 + w * 8 + g; }
        else { st -= SE; kst = st % SF; W = s.w2; K = F; n = c * 64 + w * 8 + g; }
        const int k = kst * 128 + ss * 32 + t * 8;
        out[(size_t)c * cta_stride_u4 + (size_t)layer * spl * 1024 + q] = *reinterpret_cast<const uint4*>(W + (size_t)n * K + k);
    }
}

// ---- device helpers
__device__ __forceinline__ void cl_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void cl_cluster_sync() {
    __threadfence();
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cl_trace(const ClArgs& a, int& n) {
    if (a.trace && blockIdx.x == 0 && threadIdx.x == 0) {
        long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.trace[n] = t;
        a.trace[128 + n] = clock64();
    }
    ++n;
}
__device__ __forceinline__ uint32_t cl_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

struct ClCtx {
    uint32_t ring, full0, empty0;        // shared addresses: ring base, first full / empty barrier (8 bytes each)
    const unsigned char* ring_ptr;       // the ring as a generic pointer
    const unsigned char* stream;         // this CTA's weight stream
    int stage, total;                    // next stage to consume, number of stages
    volatile int* abort_flag;
    int* err_word;
    int warp, lane;
};

__device__ __forceinline__ void cl_issue(const ClCtx& c, int i) {
    const int slot = i % CL_NS;
    const uint32_t bar = c.full0 + slot * 8;
    mbar_expect_tx(bar, CL_STAGE);
    cl_bulk_load(c.ring + slot * CL_STAGE, c.stream + (size_t)i * CL_STAGE, CL_STAGE, bar);
}

// acc[mt][..] += A[32 x K] (shared, row pitch `pitch` elements) x W^T for this warp's 8 weight rows of set `gs`,
// over n_kst stages of 128 k.  Consumes n_kst stages of the ring.
__device__ __forceinline__ void cl_gemm_set(ClCtx& c, const bf16* As, int pitch, int n_kst, float (&acc)[2][4]) {
    const int g = c.lane >> 2, t4 = c.lane & 3;
    // four independent accumulator chains per 16-row tile (one per super-step of a stage) keep the
    // dependent-MMA chain short; they are summed once at the end, in a fixed order
    float part[4][2][4];
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int e = 0; e < 4; ++e) part[ch][mt][e] = 0.f;
    for (int kst = 0; kst < n_kst; ++kst) {
        const int i = c.stage++;
        const int slot = i % CL_NS;
        if (c.warp == 0 && c.lane == 0 && i >= 1) {          // refill the slot the previous stage just vacated
            const int nxt = i - 1 + CL_NS;
            if (nxt < c.total) {
                mbar_wait(c.empty0 + ((i - 1) % CL_NS) * 8, ((i - 1) / CL_NS) & 1, c.abort_flag, c.err_word, 11);
                if (!*c.abort_flag) cl_issue(c, nxt);
            }
        }
        __syncwarp();
        mbar_wait(c.full0 + slot * 8, (i / CL_NS) & 1, c.abort_flag, c.err_word, 12);
        const unsigned char* base = c.ring_ptr + (size_t)slot * CL_STAGE + c.warp * 2048 + c.lane * 16;
        uint4 w[4];
#pragma unroll
        for (int ss = 0; ss < 4; ++ss) w[ss] = *reinterpret_cast<const uint4*>(base + ss * 512);
#pragma unroll
        for (int ss = 0; ss < 4; ++ss) {
            const bf16* ap = As + (size_t)g * pitch + kst * 128 + ss * 32 + t4 * 8;
            const uint4 a0 = *reinterpret_cast<const uint4*>(ap);
            const uint4 a1 = *reinterpret_cast<const uint4*>(ap + (size_t)8 * pitch);
            const uint4 a2 = *reinterpret_cast<const uint4*>(ap + (size_t)16 * pitch);
            const uint4 a3 = *reinterpret_cast<const uint4*>(ap + (size_t)24 * pitch);
            { const uint32_t f0[4] = {a0.x, a1.x, a0.y, a1.y}; mma_bf16(part[ss][0], f0, w[ss].x, w[ss].y); }
            { const uint32_t f1[4] = {a2.x, a3.x, a2.y, a3.y}; mma_bf16(part[ss][1], f1, w[ss].x, w[ss].y); }
            { const uint32_t f0[4] = {a0.z, a1.z, a0.w, a1.w}; mma_bf16(part[ss][0], f0, w[ss].z, w[ss].w); }
            { const uint32_t f1[4] = {a2.z, a3.z, a2.w, a3.w}; mma_bf16(part[ss][1], f1, w[ss].z, w[ss].w); }
        }
        __syncwarp();
        if (c.lane == 0) mbar_arrive(c.empty0 + slot * 8);
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][e] = (part[0][mt][e] + part[1][mt][e]) + (part[2][mt][e] + part[3][mt][e]);
}

// LayerNorm of the sequence's rows (fp32, global, read past L1) into bf16 operand rows in shared memory.
__device__ __forceinline__ void cl_layernorm(const float* x, int M, int d, const float* gam, const float* bet,
                                             bf16* As, int pitch, int warp, int lane) {
    float4 xv[4][4];                                       // 4 rows per warp, 4 float4 per lane and row: d <= 512
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int m = warp + s * 8;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int e = lane * 4 + c * 128;
            xv[s][c] = (m < M && e < d) ? __ldcg(reinterpret_cast<const float4*>(x + (size_t)m * d + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int m = warp + s * 8;
        bf16* dst = As + (size_t)m * pitch;
        if (m < M) {
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) sum += xv[s][c].x + xv[s][c].y + xv[s][c].z + xv[s][c].w;
            const float mu = warp_sum(sum) / d;
            float q = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (lane * 4 + c * 128 < d) {
                    const float c0 = xv[s][c].x - mu, c1 = xv[s][c].y - mu, c2 = xv[s][c].z - mu, c3 = xv[s][c].w - mu;
                    q += c0 * c0 + c1 * c1 + c2 * c2 + c3 * c3;
                }
            const float rstd = 1.0f / sqrtf(warp_sum(q) / d + 1e-5f);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = lane * 4 + c * 128;
                if (e < d) {
                    const float4 v = xv[s][c];
                    const float4 gm = __ldg(reinterpret_cast<const float4*>(gam + e)), bt = __ldg(reinterpret_cast<const float4*>(bet + e));
                    __nv_bfloat162 p0, p1;
                    p0.x = __float2bfloat16_rn((v.x - mu) * rstd * gm.x + bt.x); p0.y = __float2bfloat16_rn((v.y - mu) * rstd * gm.y + bt.y);
                    p1.x = __float2bfloat16_rn((v.z - mu) * rstd * gm.z + bt.z); p1.y = __float2bfloat16_rn((v.w - mu) * rstd * gm.w + bt.w);
                    *reinterpret_cast<__nv_bfloat162*>(dst + e) = p0;
                    *reinterpret_cast<__nv_bfloat162*>(dst + e + 2) = p1;
                }
            }
        } else {
            for (int e = lane * 8; e < d; e += 256) *reinterpret_cast<uint4*>(dst + e) = make_uint4(0, 0, 0, 0);
        }
    }
}

// bf16 rows [M, K] from global (written by other CTAs of the cluster: cp.async.cg reads them at L2) into operand rows.
__device__ __forceinline__ void cl_load_rows(const bf16* src, int M, int K, bf16* As, int pitch, int tid) {
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(As);
    const int chunks = K / 8;
    for (int i = tid; i < CL_M * chunks; i += CL_THREADS) {
        const int m = i / chunks, c = i % chunks;
        if (m < M) cp_async16(base + (uint32_t)(m * pitch + c * 8) * 2, src + (size_t)m * K + c * 8);
        else *reinterpret_cast<uint4*>(As + (size_t)m * pitch + c * 8) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Attention of one head for the sequence's M query rows (Q tile already in shared memory, swizzled).
// Keys: paged cache rows 0..nk-1 (causal: row m sees j + m + 1 keys) or contiguous encoder K/V (all rows see nk_all).
template <bool PAGED>
__device__ __forceinline__ void cl_attention(unsigned char* region, uint32_t Qs, const bf16* kbase, const bf16* vbase, int kv_stride,
                                             size_t kv_row0, const Paged& pg, int b, int head, int M, int j, int nk_all,
                                             int max_keys, bf16* att_rows, int d, int tid) {
    __shared__ float s_sum[CL_M];
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int nkmax = min(PAGED ? j + M : nk_all, max_keys);
    const int nkp = max((nkmax + 15) & ~15, 16);
    unsigned char* Kp = region;
    unsigned char* Vp = region + (size_t)nkp * 128;
    float* Ss = reinterpret_cast<float*>(Vp + (size_t)nkp * 128);
    const uint32_t Ks = (uint32_t)__cvta_generic_to_shared(Kp), Vs = Ks + nkp * 128;
    const int sstr = nkp + 4, pstr = nkp + 8;
    const float scale = 0.125f;                                  // 1 / sqrt(64)
    for (int i = tid; i < nkp * 8; i += CL_THREADS) {
        const int t = i >> 3, c = i & 7;
        if (t < nkmax) {
            const size_t kr = PAGED ? pg.row(b, t) : kv_row0 + t;
            cp_async16(Ks + swz(t, c), kbase + kr * kv_stride + head * 64 + c * 8);
            cp_async16(Vs + swz(t, c), vbase + kr * kv_stride + head * 64 + c * 8);
        } else {
            *reinterpret_cast<uint4*>(Kp + swz(t, c)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(Vp + swz(t, c)) = make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    {   // S = scale * Q K^T, masked; the 8 warps stride over 8-key tiles
        uint32_t qf[2][4][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
                ldsm_x4(Qs + swz(r, c), qf[mt][ks][0], qf[mt][ks][1], qf[mt][ks][2], qf[mt][ks][3]);
            }
        for (int nt = warp; nt < nkp / 8; nt += 8) {
            uint32_t kf[2][4];
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                const int r = nt * 8 + (lane & 7), c = kk * 4 + (lane >> 3);
                ldsm_x4(Ks + swz(r, c), kf[kk][0], kf[kk][1], kf[kk][2], kf[kk][3]);
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) mma_bf16(acc, qf[mt][ks], kf[ks >> 1][(ks & 1) * 2], kf[ks >> 1][(ks & 1) * 2 + 1]);
                const int ra = mt * 16 + g, rb = ra + 8, col = nt * 8 + t4 * 2;
                const int na = ra < M ? (PAGED ? min(j + ra + 1, max_keys) : nkmax) : 0;
                const int nb = rb < M ? (PAGED ? min(j + rb + 1, max_keys) : nkmax) : 0;
                Ss[ra * sstr + col] = (col < na) ? acc[0] * scale : -CUDART_INF_F;
                Ss[ra * sstr + col + 1] = (col + 1 < na) ? acc[1] * scale : -CUDART_INF_F;
                Ss[rb * sstr + col] = (col < nb) ? acc[2] * scale : -CUDART_INF_F;
                Ss[rb * sstr + col + 1] = (col + 1 < nb) ? acc[3] * scale : -CUDART_INF_F;
            }
        }
    }
    __syncthreads();
    {   // softmax with the true row maximum: 8 threads per row; P (bf16, un-normalised) overwrites the K tile
        bf16* P = reinterpret_cast<bf16*>(Kp);
        const int r = tid >> 3, sub = tid & 7;
        const float* srow = Ss + r * sstr;
        float m = -CUDART_INF_F;
        for (int c = sub; c < nkp; c += 8) m = fmaxf(m, srow[c]);
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 4));
        float sum = 0.f;
        for (int c = sub; c < nkp; c += 8) {
            const float s = srow[c];
            const float e = (s == -CUDART_INF_F) ? 0.f : expf(s - m);
            sum += e;
            P[r * pstr + c] = __float2bfloat16_rn(e);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        sum += __shfl_xor_sync(0xffffffffu, sum, 4);
        if (sub == 0) s_sum[r] = sum;
    }
    __syncthreads();
    if (warp < 4) {   // O = P V; warp w owns head columns 16w .. 16w+15
        float acc[2][2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][jj][e] = 0.f;
        for (int kt = 0; kt < nkp / 16; ++kt) {
            uint32_t vf[4];
            {
                const int r = kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = warp * 2 + (lane >> 4);
                ldsm_x4_t(Vs + swz(r, c), vf[0], vf[1], vf[2], vf[3]);
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                uint32_t pf[4];
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = kt * 16 + (lane >> 4) * 8;
                ldsm_x4(Ks + (uint32_t)(r * pstr + c) * 2, pf[0], pf[1], pf[2], pf[3]);
                mma_bf16(acc[mt][0], pf, vf[0], vf[1]);
                mma_bf16(acc[mt][1], pf, vf[2], vf[3]);
            }
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int r = mt * 16 + g + half * 8;
                if (r < M) {
                    const float den = s_sum[r];
                    bf16* o = att_rows + (size_t)r * d + head * 64 + warp * 16 + t4 * 2;
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        __nv_bfloat162 v2;
                        v2.x = __float2bfloat16_rn(den > 0.f ? acc[mt][nt][half * 2] / den : 0.f);
                        v2.y = __float2bfloat16_rn(den > 0.f ? acc[mt][nt][half * 2 + 1] / den : 0.f);
                        *reinterpret_cast<__nv_bfloat162*>(o + nt * 8) = v2;
                    }
                }
            }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(CL_THREADS, 1) k_decoder_cluster(ClArgs a) {
    extern __shared__ __align__(128) unsigned char cl_sm[];
    __shared__ __align__(8) uint64_t bar_full[CL_NS], bar_empty[CL_NS];
    __shared__ int abort_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int c = (int)cl_cta_rank();                 // = attention head owned by this CTA
    const int b = blockIdx.x / CL_C;                  // sequence of this cluster
    const int d = a.d, F = a.F, M = a.k1, Fc = F / CL_C;
    const int KS = d / 128;
    unsigned char* ring_p = cl_sm;
    unsigned char* region = cl_sm + (size_t)CL_NS * CL_STAGE;
    unsigned char* q_p = region + cl_region_bytes(F);
    bf16* As = reinterpret_cast<bf16*>(region);
    const uint32_t Qs = (uint32_t)__cvta_generic_to_shared(q_p);

    ClCtx cx;
    cx.ring = (uint32_t)__cvta_generic_to_shared(ring_p); cx.ring_ptr = ring_p;
    cx.full0 = smem_u32(&bar_full[0]); cx.empty0 = smem_u32(&bar_empty[0]);
    cx.stream = a.wstream + (size_t)c * a.cta_stride;
    cx.stage = 0; cx.total = a.n_layers * cl_stages_per_layer(d, F);
    cx.abort_flag = &abort_s; cx.err_word = a.err_word; cx.warp = warp; cx.lane = lane;
    if (tid == 0) {
        abort_s = 0;
        for (int s = 0; s < CL_NS; ++s) { mbar_init(cx.full0 + s * 8, 1); mbar_init(cx.empty0 + s * 8, CL_THREADS / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0)
        for (int i = 0; i < CL_NS && i < cx.total; ++i) cl_issue(cx, i);      // weights only: may run before the predecessor ends
    pdl_launch_dependents();
    pdl_wait();

    int tn = 0;
    cl_trace(a, tn);
    const int j = a.len[b];
    const int sl = min(a.src_len[b], a.S_max);
    const size_t r0 = (size_t)b * M;
    float* xr = a.x + r0 * d;
    bf16* attr = a.att + r0 * d;
    bf16* hr = a.hbuf + r0 * F;
    const int pd = d + 32, pF = F + 32;                // operand row pitches (elements)
    float acc[2][4];

    for (int l = 0; l < a.n_layers; ++l) {
        const ClLayer& L = a.layer[l];
        // ---------------- A: LN1, Q/K/V of head c, causal attention
        cl_layernorm(xr, M, d, L.ln1_g, L.ln1_b, As, pd, warp, lane);
        __syncthreads();
        cl_trace(a, tn);                                   // LN1 done
        for (int gs = 0; gs < 3; ++gs) {
            cl_gemm_set(cx, As, pd, KS, acc);
            const int col = warp * 8 + t4 * 2;
            const float b0 = __ldg(L.qkv_b + gs * d + c * 64 + col), b1 = __ldg(L.qkv_b + gs * d + c * 64 + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    __nv_bfloat162 v2;
                    v2.x = __float2bfloat16_rn(acc[mt][half * 2] + b0);
                    v2.y = __float2bfloat16_rn(acc[mt][half * 2 + 1] + b1);
                    if (gs == 0) {
                        *reinterpret_cast<__nv_bfloat162*>(q_p + swz(r, warp) + t4 * 4) = v2;
                    } else if (r < M) {
                        bf16* dst = (gs == 1 ? L.kc : L.vc) + a.pg.row(b, j + r) * d + c * 64 + col;
                        *reinterpret_cast<__nv_bfloat162*>(dst) = v2;
                    }
                }
        }
        __threadfence();
        __syncthreads();
        cl_trace(a, tn);                                   // QKV done
        cl_attention<true>(region, Qs, L.kc, L.vc, d, 0, a.pg, b, c, M, j, 0, a.max_keys, attr, d, tid);
        cl_trace(a, tn);                                   // self-attention done
        cl_cluster_sync();
        cl_trace(a, tn);                                   // barrier A
        // ---------------- B: out-projection + residual
        cl_load_rows(attr, M, d, As, pd, tid);
        __syncthreads();
        cl_gemm_set(cx, As, pd, KS, acc);
        {
            const int col = c * 64 + warp * 8 + t4 * 2;
            const float b0 = __ldg(L.o_b + col), b1 = __ldg(L.o_b + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    if (r < M) {
                        float2* px = reinterpret_cast<float2*>(xr + (size_t)r * d + col);
                        float2 v = __ldcg(px);
                        v.x += acc[mt][half * 2] + b0; v.y += acc[mt][half * 2 + 1] + b1;
                        *px = v;
                    }
                }
        }
        cl_cluster_sync();
        cl_trace(a, tn);                                   // phase B + barrier
        // ---------------- C: LNc, cross query of head c, attention over the encoder K/V
        cl_layernorm(xr, M, d, L.lnc_g, L.lnc_b, As, pd, warp, lane);
        __syncthreads();
        cl_gemm_set(cx, As, pd, KS, acc);
        {
            const int col = warp * 8 + t4 * 2;
            const float b0 = __ldg(L.cq_b + c * 64 + col), b1 = __ldg(L.cq_b + c * 64 + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    __nv_bfloat162 v2;
                    v2.x = __float2bfloat16_rn(acc[mt][half * 2] + b0);
                    v2.y = __float2bfloat16_rn(acc[mt][half * 2 + 1] + b1);
                    *reinterpret_cast<__nv_bfloat162*>(q_p + swz(r, warp) + t4 * 4) = v2;
                }
        }
        __syncthreads();
        cl_attention<false>(region, Qs, L.ckv, L.ckv + d, 2 * d, (size_t)b * a.S_max, a.pg, b, c, M, j, sl, a.max_keys, attr, d, tid);
        cl_cluster_sync();
        cl_trace(a, tn);                                   // phase C + barrier
        // ---------------- D: cross out-projection + residual
        cl_load_rows(attr, M, d, As, pd, tid);
        __syncthreads();
        cl_gemm_set(cx, As, pd, KS, acc);
        {
            const int col = c * 64 + warp * 8 + t4 * 2;
            const float b0 = __ldg(L.co_b + col), b1 = __ldg(L.co_b + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    if (r < M) {
                        float2* px = reinterpret_cast<float2*>(xr + (size_t)r * d + col);
                        float2 v = __ldcg(px);
                        v.x += acc[mt][half * 2] + b0; v.y += acc[mt][half * 2 + 1] + b1;
                        *px = v;
                    }
                }
        }
        cl_cluster_sync();
        cl_trace(a, tn);                                   // phase D + barrier
        // ---------------- E: LN2, FFN1 columns of this CTA, ReLU
        cl_layernorm(xr, M, d, L.ln2_g, L.ln2_b, As, pd, warp, lane);
        __syncthreads();
        for (int gs = 0; gs < Fc / 64; ++gs) {
            cl_gemm_set(cx, As, pd, KS, acc);
            const int col = c * Fc + gs * 64 + warp * 8 + t4 * 2;
            const float b0 = __ldg(L.b1 + col), b1 = __ldg(L.b1 + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    if (r < M) {
                        __nv_bfloat162 v2;
                        v2.x = __float2bfloat16_rn(fmaxf(acc[mt][half * 2] + b0, 0.f));
                        v2.y = __float2bfloat16_rn(fmaxf(acc[mt][half * 2 + 1] + b1, 0.f));
                        *reinterpret_cast<__nv_bfloat162*>(hr + (size_t)r * F + col) = v2;
                    }
                }
        }
        cl_cluster_sync();
        cl_trace(a, tn);                                   // phase E + barrier
        // ---------------- F: FFN2 + residual
        cl_load_rows(hr, M, F, As, pF, tid);
        __syncthreads();
        cl_trace(a, tn);                                   // hidden rows loaded
        cl_gemm_set(cx, As, pF, F / 128, acc);
        {
            const int col = c * 64 + warp * 8 + t4 * 2;
            const float b0 = __ldg(L.b2 + col), b1 = __ldg(L.b2 + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    if (r < M) {
                        float2* px = reinterpret_cast<float2*>(xr + (size_t)r * d + col);
                        float2 v = __ldcg(px);
                        v.x += acc[mt][half * 2] + b0; v.y += acc[mt][half * 2 + 1] + b1;
                        *px = v;
                    }
                }
        }
        cl_cluster_sync();
        cl_trace(a, tn);                                   // phase F + barrier
    }
}

}  // namespace sd
