// Tile attention for bf16 operands and head size 64: one CTA per (32-query tile, head, sequence).
//
//   K and V of every visible key are staged once in shared memory (16-byte cp.async, 128-byte rows,
//   XOR-swizzled chunks), S = Q K^T runs on the tensor cores (mma.sync m16n8k16, fp32 accumulate),
//   the softmax is single pass with the true row maximum, the un-normalised probabilities are
//   rounded to bf16 for P V (second tensor-core contraction) and the result is divided by the fp32
//   sum of the unrounded exponentials -- the same arithmetic as the reference attention kernel.
//
// Used for the verifier's causal attention over the paged cache, both cross-attentions, the
// drafter's bidirectional attention and the encoders.  Work per CTA is 2 * 32 * keys * 64 * 2 flops:
// far too little to fill a 128-row tcgen05 tile, which is why this contraction uses warp-level MMA.
#pragma once
#include "kernels.cuh"

namespace sd {

struct AttnTcArgs {
    const bf16* q; int q_stride; const int* q_index;     // query row r reads q + (q_index ? q_index[r] : r) * q_stride
    const bf16* k; const bf16* v; int kv_stride;         // contiguous: key t of sequence b at row kv_off[b] + t
    const int* kv_off;
    Paged pg;                                             // paged: row pg.row(b, t)
    const int* q_off; const int* q_cnt;                   // per sequence: first query row, number of query rows
    const int* nkeys;                                     // per query row: visible keys (0..nkeys-1)
    const int* pre_keys;                                  // per sequence (or null): keys 0..pre-1 were written before this
                                                          // step began, so they may be fetched before the dependency wait
    bf16* out; int out_stride;
    int max_keys;                                         // capacity the shared memory was sized for
    float scale;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// byte offset of 16-byte chunk c (0..7) of row r in a tile of 128-byte rows
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

constexpr int ATT_Q = 32;
// NW warps per CTA: 8 when few CTAs are in flight (each CTA is one latency chain: more warps shorten it) or
// when shared memory leaves room for one or two CTAs per SM; 4 when the SMs are saturated with CTAs anyway
// (fewer duplicated fragment loads per CTA).
inline size_t attn_tc_smem(int max_keys) {
    const int nkp = (max_keys + 15) & ~15;
    return (size_t)ATT_Q * 128 + (size_t)nkp * 256 + (size_t)ATT_Q * (nkp + 4) * 4 + 16;
}
// RS ("register scores"): with at most ATT_RS_TILES 8-key tiles per warp the scores stay in the MMA accumulators
// through the softmax, so shared memory holds Q, K and V only (a third less at 96 keys: more CTAs per SM).
constexpr int ATT_RS_TILES = 6;
inline int attn_tc_rs_max_keys(int warps) { return warps * ATT_RS_TILES * 8; }
inline size_t attn_tc_smem_rs(int max_keys) {
    const int nkp = (max_keys + 15) & ~15;
    return (size_t)ATT_Q * 128 + (size_t)nkp * 256 + 16;
}

template <bool PAGED, int NW, bool RS = false>
__global__ void __launch_bounds__(NW * 32) k_attn_tc(AttnTcArgs a) {
    constexpr int ATT_THREADS = NW * 32;
    __shared__ float s_wmax[RS ? NW * ATT_Q : 1], s_wsum[RS ? NW * ATT_Q : 1];   // RS: per-warp row maxima and sums
    extern __shared__ __align__(128) unsigned char sm[];
    __shared__ int s_nk[ATT_Q];
    __shared__ float s_sum[ATT_Q];
    __shared__ int s_nkmax;
    const int b = blockIdx.z, h = blockIdx.y, qt = blockIdx.x;
    // Row metadata, page table and sequence lengths are written at the start of the step, before the first
    // kernel of the programmatic-launch chain can begin, so they may be read before the dependency wait.
    const int cnt = a.q_cnt[b];
    if (qt * ATT_Q >= cnt) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r0 = a.q_off[b] + qt * ATT_Q, nq = min(ATT_Q, cnt - qt * ATT_Q);

    if (tid < 32) {
        int nk = (tid < nq) ? min(a.nkeys[r0 + tid], a.max_keys) : 0;
        s_nk[tid] = nk;
        int m = nk;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (tid == 0) s_nkmax = m;
    }
    __syncthreads();
    const int nkmax = s_nkmax;
    const int nkp = max((nkmax + 15) & ~15, 16);
    const uint32_t Qs = (uint32_t)__cvta_generic_to_shared(sm), Ks = Qs + ATT_Q * 128, Vs = Ks + nkp * 128;
    unsigned char* Qp = sm;
    unsigned char* Kp = sm + ATT_Q * 128;
    unsigned char* Vp = Kp + nkp * 128;
    float* Ss = reinterpret_cast<float*>(Vp + nkp * 128);
    const int sstr = nkp + 4;                    // fp32 row pitch of S
    const int pstr = nkp + 8;                    // bf16 row pitch of P (lives where K was)

    // ---- stage K, V of the keys that predate this step (cached prefix, encoder memory) before the wait ...
    const int npre = a.pre_keys ? min(a.pre_keys[b], nkmax) : 0;
    // a thread keeps its 16-byte chunk of the 128-byte head slice and walks the keys: one row lookup per request pair
    const int c8 = tid & 7, t0 = tid >> 3;
    constexpr int TSTEP = ATT_THREADS / 8;
    const bf16* kcol = a.k + h * 64 + c8 * 8;
    const bf16* vcol = a.v + h * 64 + c8 * 8;
    for (int t = t0; t < npre; t += TSTEP) {
        const size_t off = (PAGED ? a.pg.row(b, t) : (size_t)(a.kv_off[b] + t)) * a.kv_stride;
        cp_async16(Ks + swz(t, c8), kcol + off);
        cp_async16(Vs + swz(t, c8), vcol + off);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    pdl_launch_dependents();
    pdl_wait();                                   // ... and everything the predecessor kernels wrote after it
    for (int r = t0; r < ATT_Q; r += TSTEP) {
        if (r < nq) {
            const size_t qr = a.q_index ? (size_t)a.q_index[r0 + r] : (size_t)(r0 + r);
            cp_async16(Qs + swz(r, c8), a.q + qr * a.q_stride + h * 64 + c8 * 8);
        } else {
            *reinterpret_cast<uint4*>(Qp + swz(r, c8)) = make_uint4(0, 0, 0, 0);
        }
    }
    for (int t = t0; t < nkp; t += TSTEP) {
        if (t < npre) continue;
        if (t < nkmax) {
            const size_t off = (PAGED ? a.pg.row(b, t) : (size_t)(a.kv_off[b] + t)) * a.kv_stride;
            cp_async16(Ks + swz(t, c8), kcol + off);
            cp_async16(Vs + swz(t, c8), vcol + off);
        } else {
            *reinterpret_cast<uint4*>(Kp + swz(t, c8)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(Vp + swz(t, c8)) = make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    const int g = lane >> 2, t4 = lane & 3;
    if constexpr (RS) {
        // ---- S = scale * Q K^T in registers: warp w takes key tiles w, w + NW, ...
        uint32_t qf[2][4][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
                ldsm_x4(Qs + swz(r, c), qf[mt][ks][0], qf[mt][ks][1], qf[mt][ks][2], qf[mt][ks][3]);
            }
        float sc[2][ATT_RS_TILES][4];
        float rmax[2][2] = {{-CUDART_INF_F, -CUDART_INF_F}, {-CUDART_INF_F, -CUDART_INF_F}};   // [mt][row g / row g + 8]
        int nkr[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) { nkr[mt][0] = s_nk[mt * 16 + g]; nkr[mt][1] = s_nk[mt * 16 + g + 8]; }
#pragma unroll
        for (int j = 0; j < ATT_RS_TILES; ++j) {
            const int nt = warp + j * NW;
            if (nt < nkp / 8) {
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
                    const int col = nt * 8 + t4 * 2;
                    sc[mt][j][0] = (col < nkr[mt][0]) ? acc[0] * a.scale : -CUDART_INF_F;
                    sc[mt][j][1] = (col + 1 < nkr[mt][0]) ? acc[1] * a.scale : -CUDART_INF_F;
                    sc[mt][j][2] = (col < nkr[mt][1]) ? acc[2] * a.scale : -CUDART_INF_F;
                    sc[mt][j][3] = (col + 1 < nkr[mt][1]) ? acc[3] * a.scale : -CUDART_INF_F;
                    rmax[mt][0] = fmaxf(rmax[mt][0], fmaxf(sc[mt][j][0], sc[mt][j][1]));
                    rmax[mt][1] = fmaxf(rmax[mt][1], fmaxf(sc[mt][j][2], sc[mt][j][3]));
                }
            } else {
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) sc[mt][j][e] = -CUDART_INF_F;
            }
        }
        // row maximum: across the four lanes that share a row, then across warps through shared memory
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                float m = rmax[mt][hb];
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
                if (t4 == 0) s_wmax[warp * ATT_Q + mt * 16 + hb * 8 + g] = m;
            }
        __syncthreads();                              // every warp is also done reading K: P may overwrite it
        bf16* P = reinterpret_cast<bf16*>(Kp);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                const int row = mt * 16 + hb * 8 + g;
                float m = -CUDART_INF_F;
#pragma unroll
                for (int w = 0; w < NW; ++w) m = fmaxf(m, s_wmax[w * ATT_Q + row]);
                const float mb = (m == -CUDART_INF_F) ? 0.f : m * 1.4426950408889634f;     // masked scores (-inf) give 0
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < ATT_RS_TILES; ++j) {
                    const int nt = warp + j * NW;
                    if (nt < nkp / 8) {
                        const float s0 = sc[mt][j][hb * 2], s1 = sc[mt][j][hb * 2 + 1];
                        const float e0 = exp2f(fmaf(s0, 1.4426950408889634f, -mb)), e1 = exp2f(fmaf(s1, 1.4426950408889634f, -mb));
                        sum += e0 + e1;
                        *reinterpret_cast<__nv_bfloat162*>(P + row * pstr + nt * 8 + t4 * 2) = __floats2bfloat162_rn(e0, e1);
                    }
                }
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                if (t4 == 0) s_wsum[warp * ATT_Q + row] = sum;
            }
        __syncthreads();
        if (tid < ATT_Q) {                            // normaliser of a row: the warps' sums in a fixed order
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) t += s_wsum[w * ATT_Q + tid];
            s_sum[tid] = t;
        }
        __syncthreads();
    } else {
    // ---- S = scale * Q K^T, masked
    {
        uint32_t qf[2][4][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
                ldsm_x4(Qs + swz(r, c), qf[mt][ks][0], qf[mt][ks][1], qf[mt][ks][2], qf[mt][ks][3]);
            }
        int nkr[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) { nkr[mt][0] = s_nk[mt * 16 + g]; nkr[mt][1] = s_nk[mt * 16 + g + 8]; }
        for (int nt = warp; nt < nkp / 8; nt += ATT_THREADS / 32) {
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
                const int na = nkr[mt][0], nb = nkr[mt][1];
                *reinterpret_cast<float2*>(Ss + ra * sstr + col) =
                    make_float2((col < na) ? acc[0] * a.scale : -CUDART_INF_F, (col + 1 < na) ? acc[1] * a.scale : -CUDART_INF_F);
                *reinterpret_cast<float2*>(Ss + rb * sstr + col) =
                    make_float2((col < nb) ? acc[2] * a.scale : -CUDART_INF_F, (col + 1 < nb) ? acc[3] * a.scale : -CUDART_INF_F);
            }
        }
    }
    __syncthreads();
    // ---- softmax: NW threads per row, four scores at a time; P (bf16, un-normalised) overwrites the K tile
    {
        bf16* P = reinterpret_cast<bf16*>(Kp);
        const int r = tid / NW, sub = tid % NW;
        const float4* srow = reinterpret_cast<const float4*>(Ss + r * sstr);
        float m = -CUDART_INF_F;
        for (int c = sub; c < nkp / 4; c += NW) {
            const float4 s4 = srow[c];
            m = fmaxf(m, fmaxf(fmaxf(s4.x, s4.y), fmaxf(s4.z, s4.w)));
        }
#pragma unroll
        for (int o = 1; o < NW; o <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        // exp(s - m) as 2^((s - m) log2 e); a masked score is -inf and gives 0, a row without keys keeps sum 0
        const float mb = (m == -CUDART_INF_F) ? 0.f : m * 1.4426950408889634f;
        float sum = 0.f;
        for (int c = sub; c < nkp / 4; c += NW) {
            const float4 s4 = srow[c];
            const float e0 = exp2f(fmaf(s4.x, 1.4426950408889634f, -mb)), e1 = exp2f(fmaf(s4.y, 1.4426950408889634f, -mb));
            const float e2 = exp2f(fmaf(s4.z, 1.4426950408889634f, -mb)), e3 = exp2f(fmaf(s4.w, 1.4426950408889634f, -mb));
            sum += (e0 + e1) + (e2 + e3);
            __nv_bfloat162 p01 = __floats2bfloat162_rn(e0, e1), p23 = __floats2bfloat162_rn(e2, e3);
            *reinterpret_cast<uint2*>(P + r * pstr + c * 4) = make_uint2(*reinterpret_cast<uint32_t*>(&p01), *reinterpret_cast<uint32_t*>(&p23));
        }
#pragma unroll
        for (int o = 1; o < NW; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (sub == 0) s_sum[r] = sum;
    }
    __syncthreads();
    }
    // ---- O = P V ; warp w owns query rows 16 (w / (NW / 2)) .. and 128 / NW head columns
    {
        constexpr int WPM = NW / 2;                  // warps per 16-row query tile
        constexpr int NV = 64 / WPM / 16;            // 16-column groups per warp
        const int mt = warp / WPM, wq = warp % WPM;
        float acc[2 * NV][4];
#pragma unroll
        for (int j = 0; j < 2 * NV; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
        for (int kt = 0; kt < nkp / 16; ++kt) {
            uint32_t pf[4];
            {
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = kt * 16 + (lane >> 4) * 8;
                ldsm_x4(Ks + (uint32_t)(r * pstr + c) * 2, pf[0], pf[1], pf[2], pf[3]);
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                uint32_t vf[4];
                const int r = kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = (wq * NV + v) * 2 + (lane >> 4);
                ldsm_x4_t(Vs + swz(r, c), vf[0], vf[1], vf[2], vf[3]);
                mma_bf16(acc[2 * v], pf, vf[0], vf[1]);
                mma_bf16(acc[2 * v + 1], pf, vf[2], vf[3]);
            }
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = mt * 16 + g + half * 8;
            if (r < nq) {
                const float den = s_sum[r], inv = den > 0.f ? 1.0f / den : 0.f;
                bf16* o = a.out + (size_t)(r0 + r) * a.out_stride + h * 64 + wq * (NV * 16) + t4 * 2;
#pragma unroll
                for (int nt = 0; nt < 2 * NV; ++nt)
                    *reinterpret_cast<__nv_bfloat162*>(o + nt * 8) = __floats2bfloat162_rn(acc[nt][half * 2] * inv, acc[nt][half * 2 + 1] * inv);
            }
        }
    }
}

}  // namespace sd
