// Attention and its output projection in one kernel, for blocks of at most 32 query rows per sequence
// (the verify block, the drafter's mask rows) and models with 8 heads of 64.
//
// A cluster of 8 CTAs owns one sequence, CTA h one head.  Each CTA runs the tile attention of its head
// (the same arithmetic as k_attn_tc), then writes its 32 x 64 slice of the attention output into the
// operand buffer of ALL eight CTAs through distributed shared memory.  After one hardware cluster
// barrier every CTA holds the full 32 x 512 attention output and computes 64 columns of the output
// projection (warp-level MMA, weights streamed from global memory with the k permutation of the
// weight-streaming GEMM), adds bias and accumulates into the fp32 residual stream.
// This removes a kernel boundary, the round trip of the attention output through global memory and the
// separate projection kernel; the projection weights are read once per sequence.
#pragma once
#include "attention_tc.cuh"
#include "kernels.cuh"

namespace sd {

struct AttnProjArgs {
    AttnTcArgs at;          // attention part (out / out_stride unused)
    const bf16* wo;         // [d, d] output projection, row-major [out, in]
    const float* bo;        // [d]
    float* x;               // residual rows [rows, d]: x[r, n] += proj
    int d;                  // model width = 8 * 64
};

constexpr int AP_HEADS = 8;
inline size_t attn_proj_smem(int max_keys, int d) { return attn_tc_smem(max_keys) + (size_t)ATT_Q * (d + 32) * 2 + 128; }

__device__ __forceinline__ uint32_t ap_map_remote(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void ap_st_remote_b32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

template <bool PAGED>
__global__ void __launch_bounds__(128) k_attn_proj(AttnProjArgs p) {
    extern __shared__ __align__(128) unsigned char sm[];
    __shared__ int s_nk[ATT_Q];
    __shared__ float s_sum[ATT_Q];
    __shared__ int s_nkmax;
    const AttnTcArgs& a = p.at;
    const int h = blockIdx.x, b = blockIdx.y;           // cluster rank = head
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int d = p.d, apitch = d + 32;                 // operand row pitch (elements)
    // first barrier phase: a CTA may only be written through distributed shared memory once it has started;
    // arrive now, wait right before the remote stores
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    pdl_launch_dependents();
    pdl_wait();
    const int cnt = min(a.q_cnt[b], ATT_Q);             // uniform over the cluster: every CTA reaches the barriers
    const int r0 = a.q_off[b], nq = cnt;

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
    // layout: [operand rows 32 x (d+32) bf16][Q 32 x 128 B][K nkp x 128 B][V nkp x 128 B][S 32 x (nkp+4) fp32]
    unsigned char* Ap = sm;
    unsigned char* Qp = sm + (((size_t)ATT_Q * apitch * 2 + 127) & ~size_t(127));
    unsigned char* Kp = Qp + ATT_Q * 128;
    unsigned char* Vp = Kp + nkp * 128;
    float* Ss = reinterpret_cast<float*>(Vp + nkp * 128);
    const uint32_t As = (uint32_t)__cvta_generic_to_shared(Ap);
    const uint32_t Qs = (uint32_t)__cvta_generic_to_shared(Qp), Ks = Qs + ATT_Q * 128, Vs = Ks + nkp * 128;
    const int sstr = nkp + 4, pstr = nkp + 8;

    if (nq == 0) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
    if (nq > 0) {
        for (int i = tid; i < ATT_Q * 8; i += 128) {
            const int r = i >> 3, c = i & 7;
            if (r < nq) {
                const size_t qr = a.q_index ? (size_t)a.q_index[r0 + r] : (size_t)(r0 + r);
                cp_async16(Qs + swz(r, c), a.q + qr * a.q_stride + h * 64 + c * 8);
            } else {
                *reinterpret_cast<uint4*>(Qp + swz(r, c)) = make_uint4(0, 0, 0, 0);
            }
        }
        for (int i = tid; i < nkp * 8; i += 128) {
            const int t = i >> 3, c = i & 7;
            if (t < nkmax) {
                const size_t kr = PAGED ? a.pg.row(b, t) : (size_t)(a.kv_off[b] + t);
                cp_async16(Ks + swz(t, c), a.k + kr * a.kv_stride + h * 64 + c * 8);
                cp_async16(Vs + swz(t, c), a.v + kr * a.kv_stride + h * 64 + c * 8);
            } else {
                *reinterpret_cast<uint4*>(Kp + swz(t, c)) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(Vp + swz(t, c)) = make_uint4(0, 0, 0, 0);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        {   // S = scale * Q K^T, masked
            uint32_t qf[2][4][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
                    ldsm_x4(Qs + swz(r, c), qf[mt][ks][0], qf[mt][ks][1], qf[mt][ks][2], qf[mt][ks][3]);
                }
            for (int nt = warp; nt < nkp / 8; nt += 4) {
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
                    const int na = s_nk[ra], nb = s_nk[rb];
                    Ss[ra * sstr + col] = (col < na) ? acc[0] * a.scale : -CUDART_INF_F;
                    Ss[ra * sstr + col + 1] = (col + 1 < na) ? acc[1] * a.scale : -CUDART_INF_F;
                    Ss[rb * sstr + col] = (col < nb) ? acc[2] * a.scale : -CUDART_INF_F;
                    Ss[rb * sstr + col + 1] = (col + 1 < nb) ? acc[3] * a.scale : -CUDART_INF_F;
                }
            }
        }
        __syncthreads();
        {   // softmax with the true row maximum; P (bf16, un-normalised) overwrites the K tile
            bf16* P = reinterpret_cast<bf16*>(Kp);
            const int r = tid >> 2, sub = tid & 3;
            const float* srow = Ss + r * sstr;
            float m = -CUDART_INF_F;
            for (int c = sub; c < nkp; c += 4) m = fmaxf(m, srow[c]);
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            float sum = 0.f;
            for (int c = sub; c < nkp; c += 4) {
                const float s = srow[c];
                const float e = (s == -CUDART_INF_F) ? 0.f : expf(s - m);
                sum += e;
                P[r * pstr + c] = __float2bfloat16_rn(e);
            }
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            if (sub == 0) s_sum[r] = sum;
        }
        __syncthreads();
        {   // O = P V ; warp w owns head columns 16w .. 16w+15; the result goes to every CTA of the cluster
            float acc[2][2][4];
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;
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
            asm volatile("barrier.cluster.wait.aligned;" ::: "memory");      // all eight CTAs are running
            uint32_t remote[AP_HEADS];
#pragma unroll
            for (int c = 0; c < AP_HEADS; ++c) remote[c] = ap_map_remote(As, (uint32_t)c);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    const float den = s_sum[r];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        __nv_bfloat162 v2;
                        v2.x = __float2bfloat16_rn((r < nq && den > 0.f) ? acc[mt][nt][half * 2] / den : 0.f);
                        v2.y = __float2bfloat16_rn((r < nq && den > 0.f) ? acc[mt][nt][half * 2 + 1] / den : 0.f);
                        const uint32_t off = (uint32_t)(r * apitch + h * 64 + warp * 16 + nt * 8 + t4 * 2) * 2;
                        const uint32_t bits = *reinterpret_cast<const uint32_t*>(&v2);
#pragma unroll
                        for (int c = 0; c < AP_HEADS; ++c) ap_st_remote_b32(remote[c] + off, bits);
                    }
                }
        }
    }
    // every CTA's slice has landed in every operand buffer after this barrier
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (nq == 0) return;

    // ---- output projection: columns h*64 + warp*16 + {0..15} (two 8-row weight groups per warp), K = d
    {
        const bf16* A = reinterpret_cast<const bf16*>(Ap);
        float acc[2][2][4];                                  // [group][16-row tile][..]
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;
        const int nbase = h * 64 + warp * 16;
        const bf16* w0 = p.wo + (size_t)(nbase + g) * d + t4 * 8;
        const bf16* w1 = w0 + (size_t)8 * d;
        for (int k0 = 0; k0 < d; k0 += 128) {                // 4 super-steps of 32 k in flight per group
            uint4 wa[4], wb[4];
#pragma unroll
            for (int ss = 0; ss < 4; ++ss) {
                wa[ss] = __ldg(reinterpret_cast<const uint4*>(w0 + k0 + ss * 32));
                wb[ss] = __ldg(reinterpret_cast<const uint4*>(w1 + k0 + ss * 32));
            }
#pragma unroll
            for (int ss = 0; ss < 4; ++ss) {
                const bf16* ap = A + (size_t)g * apitch + k0 + ss * 32 + t4 * 8;
                const uint4 a0 = *reinterpret_cast<const uint4*>(ap);
                const uint4 a1 = *reinterpret_cast<const uint4*>(ap + (size_t)8 * apitch);
                const uint4 a2 = *reinterpret_cast<const uint4*>(ap + (size_t)16 * apitch);
                const uint4 a3 = *reinterpret_cast<const uint4*>(ap + (size_t)24 * apitch);
                const uint32_t f00[4] = {a0.x, a1.x, a0.y, a1.y}, f01[4] = {a2.x, a3.x, a2.y, a3.y};
                const uint32_t f10[4] = {a0.z, a1.z, a0.w, a1.w}, f11[4] = {a2.z, a3.z, a2.w, a3.w};
                mma_bf16(acc[0][0], f00, wa[ss].x, wa[ss].y); mma_bf16(acc[0][1], f01, wa[ss].x, wa[ss].y);
                mma_bf16(acc[0][0], f10, wa[ss].z, wa[ss].w); mma_bf16(acc[0][1], f11, wa[ss].z, wa[ss].w);
                mma_bf16(acc[1][0], f00, wb[ss].x, wb[ss].y); mma_bf16(acc[1][1], f01, wb[ss].x, wb[ss].y);
                mma_bf16(acc[1][0], f10, wb[ss].z, wb[ss].w); mma_bf16(acc[1][1], f11, wb[ss].z, wb[ss].w);
            }
        }
#pragma unroll
        for (int grp = 0; grp < 2; ++grp) {
            const int col = nbase + grp * 8 + t4 * 2;
            const float b0 = __ldg(p.bo + col), b1 = __ldg(p.bo + col + 1);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = mt * 16 + g + half * 8;
                    if (r < nq) {
                        float2* px = reinterpret_cast<float2*>(p.x + (size_t)(r0 + r) * d + col);
                        float2 v = *px;
                        v.x += acc[grp][mt][half * 2] + b0; v.y += acc[grp][mt][half * 2 + 1] + b1;
                        *px = v;
                    }
                }
        }
    }
}

}  // namespace sd
