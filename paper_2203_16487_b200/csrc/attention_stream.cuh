// Streaming tile attention for long key ranges (bf16 operands, head size 64): one CTA of four warps per
// (32-query tile, head, sequence) walks the keys in blocks of 64 through a ring of NS cp.async stages (2 when the
// SMs are full of CTAs anyway, 4 when a CTA's own chain of round trips is what counts), so its shared memory
// (36 / 68 KB) does not grow with the number of keys -- the one-shot tile kernel stages every key at
// once, which caps it near 590 keys and leaves one or two CTAs per SM long before that.
//
//   per block and warp: S = Q K^T for 16 query rows x 32 keys (mma.sync m16n8k16), running row maximum and
//   sum in registers, the accumulator of O rescaled when the maximum moves, P (bf16, relative to the running
//   maximum) fed to the second contraction straight from the score registers.  The two warps that share a
//   query tile (one per half of every key block) merge their (maximum, sum, O) through shared memory at the end;
//   the result is divided by the fp32 sum of the unrounded exponentials, as in the one-shot kernel.
//
// Softmax over the visible keys of scaled dot-product attention (Vaswani et al.; the paper's Transformer
// blocks, Section 3.1 / 3.2): mathematically the same quantity, summed in a different order and with P rounded
// relative to a running instead of the final maximum -- a difference of a few bf16 ulps of single terms.
#pragma once
#include "attention_tc.cuh"

namespace sd {

constexpr int ATS_KB = 64;                                   // keys per block
constexpr int ATS_STAGE = ATS_KB * 128 * 2;                  // K and V of a block: 16 KB
constexpr int ats_smem(int ns) { return ATT_Q * 128 + ns * ATS_STAGE + 16; }   // Q + the stages
static_assert(2 * ATS_STAGE >= 2 * 16 * 64 * 4 + 2 * 2 * 16 * 4, "the merge buffers reuse the stages");

__device__ __forceinline__ void ats_wait_pending(int n) {       // cp.async.wait_group takes an immediate
    if (n <= 0) asm volatile("cp.async.wait_group 0;" ::: "memory");
    else if (n == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else if (n == 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else asm volatile("cp.async.wait_group 3;" ::: "memory");
}

template <bool PAGED, int NS>
__global__ void __launch_bounds__(128) k_attn_stream(AttnTcArgs a) {
    static_assert(NS >= 2 && NS <= 4, "ring depth");
    extern __shared__ __align__(128) unsigned char sm[];
    __shared__ int s_nk[ATT_Q];
    __shared__ int s_nkmax;
    const int b = blockIdx.z, h = blockIdx.y, qt = blockIdx.x;
    const int cnt = a.q_cnt[b];                  // row metadata predates the step's kernel chain: readable before the wait
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
    const int nblk = max((nkmax + ATS_KB - 1) / ATS_KB, 1);
    const uint32_t Qs = (uint32_t)__cvta_generic_to_shared(sm), St = Qs + ATT_Q * 128;
    unsigned char* Qp = sm;
    unsigned char* Sp = sm + ATT_Q * 128;

    auto load_block = [&](int blk) {            // keys blk * 64 .. + 63 into stage blk % NS; rows past the last key are zeroed
        const uint32_t Ks = St + (blk % NS) * ATS_STAGE, Vs = Ks + ATS_KB * 128;
        unsigned char* Kp = Sp + (blk % NS) * ATS_STAGE;
        unsigned char* Vp = Kp + ATS_KB * 128;
        for (int i = tid; i < ATS_KB * 8; i += 128) {
            const int t = i >> 3, c = i & 7, key = blk * ATS_KB + t;
            if (key < nkmax) {
                const size_t kr = PAGED ? a.pg.row(b, key) : (size_t)(a.kv_off[b] + key);
                cp_async16(Ks + swz(t, c), a.k + kr * a.kv_stride + h * 64 + c * 8);
                cp_async16(Vs + swz(t, c), a.v + kr * a.kv_stride + h * 64 + c * 8);
            } else {
                *reinterpret_cast<uint4*>(Kp + swz(t, c)) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(Vp + swz(t, c)) = make_uint4(0, 0, 0, 0);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // blocks made only of keys that predate this step (cached prefix, encoder memory) may be requested before the wait
    const int npre = a.pre_keys ? min(a.pre_keys[b], nkmax) : 0;
    int issued = 0;
    while (issued < NS && issued < nblk && (issued + 1) * ATS_KB <= npre) { load_block(issued); ++issued; }
    const int pre_issued = issued;
    pdl_launch_dependents();
    pdl_wait();
    for (int i = tid; i < ATT_Q * 8; i += 128) {
        const int r = i >> 3, c = i & 7;
        if (r < nq) {
            const size_t qr = a.q_index ? (size_t)a.q_index[r0 + r] : (size_t)(r0 + r);
            cp_async16(Qs + swz(r, c), a.q + qr * a.q_stride + h * 64 + c * 8);
        } else {
            *reinterpret_cast<uint4*>(Qp + swz(r, c)) = make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");

    const int g = lane >> 2, t4 = lane & 3;
    const int mt = warp & 1, kh = warp >> 1;     // query rows 16 mt .. + 15, keys 32 kh .. + 31 of every block
    const int nk0 = s_nk[mt * 16 + g], nk1 = s_nk[mt * 16 + g + 8];
    uint32_t qf[4][4];
    float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};   // rows g, g + 8 (sums: this lane's share)
    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;

    for (int blk = 0; blk < nblk; ++blk) {
        while (issued < min(blk + NS, nblk)) { load_block(issued); ++issued; }
        // commit order: blocks requested before the wait, Q, the other blocks.  Block blk and Q must have landed;
        // the groups committed after both may stay in flight
        ats_wait_pending(blk == 0 ? (pre_issued > 0 ? issued - pre_issued : issued - 1) : issued - blk - 1);
        __syncthreads();
        if (blk == 0) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
                ldsm_x4(Qs + swz(r, c), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
            }
        }
        const uint32_t Ks = St + (blk % NS) * ATS_STAGE, Vs = Ks + ATS_KB * 128;
        const int kbase = blk * ATS_KB + kh * 32;
        if (kbase < nkmax) {                       // warp-uniform: this half of the block holds a visible key
            float sc[4][4];
            float bm0 = -CUDART_INF_F, bm1 = -CUDART_INF_F;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                uint32_t kf[2][4];
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int r = kh * 32 + nt * 8 + (lane & 7), c = kk * 4 + (lane >> 3);
                    ldsm_x4(Ks + swz(r, c), kf[kk][0], kf[kk][1], kf[kk][2], kf[kk][3]);
                }
                float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) mma_bf16(s4, qf[ks], kf[ks >> 1][(ks & 1) * 2], kf[ks >> 1][(ks & 1) * 2 + 1]);
                const int col = kbase + nt * 8 + t4 * 2;
                sc[nt][0] = (col < nk0) ? s4[0] * a.scale : -CUDART_INF_F;
                sc[nt][1] = (col + 1 < nk0) ? s4[1] * a.scale : -CUDART_INF_F;
                sc[nt][2] = (col < nk1) ? s4[2] * a.scale : -CUDART_INF_F;
                sc[nt][3] = (col + 1 < nk1) ? s4[3] * a.scale : -CUDART_INF_F;
                bm0 = fmaxf(bm0, fmaxf(sc[nt][0], sc[nt][1]));
                bm1 = fmaxf(bm1, fmaxf(sc[nt][2], sc[nt][3]));
            }
            bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1)); bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
            bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1)); bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
            const float mn0 = fmaxf(m_run[0], bm0), mn1 = fmaxf(m_run[1], bm1);
            // a row with no visible key so far keeps maximum -inf: its factor is 1 and its terms are 0
            const float al0 = (m_run[0] == -CUDART_INF_F) ? 1.f : expf(m_run[0] - mn0);
            const float al1 = (m_run[1] == -CUDART_INF_F) ? 1.f : expf(m_run[1] - mn1);
            m_run[0] = mn0; m_run[1] = mn1;
            l_run[0] *= al0; l_run[1] *= al1;
#pragma unroll
            for (int j = 0; j < 8; ++j) { acc[j][0] *= al0; acc[j][1] *= al0; acc[j][2] *= al1; acc[j][3] *= al1; }
            constexpr float L2E = 1.4426950408889634f;
            const float mb0 = (mn0 == -CUDART_INF_F) ? 0.f : mn0 * L2E, mb1 = (mn1 == -CUDART_INF_F) ? 0.f : mn1 * L2E;
            uint32_t pf[2][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const float e0 = exp2f(fmaf(sc[nt][0], L2E, -mb0)), e1 = exp2f(fmaf(sc[nt][1], L2E, -mb0));   // -inf scores give 0
                const float e2 = exp2f(fmaf(sc[nt][2], L2E, -mb1)), e3 = exp2f(fmaf(sc[nt][3], L2E, -mb1));
                l_run[0] += e0 + e1; l_run[1] += e2 + e3;
                __nv_bfloat162 p01 = __floats2bfloat162_rn(e0, e1), p23 = __floats2bfloat162_rn(e2, e3);
                // accumulator layout of an 8-key tile = half of the A fragment of a 16-key step
                pf[nt >> 1][(nt & 1) * 2] = *reinterpret_cast<uint32_t*>(&p01);
                pf[nt >> 1][(nt & 1) * 2 + 1] = *reinterpret_cast<uint32_t*>(&p23);
            }
#pragma unroll
            for (int kt = 0; kt < 2; ++kt)
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint32_t vf[4];
                    const int r = kh * 32 + kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = v * 2 + (lane >> 4);
                    ldsm_x4_t(Vs + swz(r, c), vf[0], vf[1], vf[2], vf[3]);
                    mma_bf16(acc[2 * v], pf[kt], vf[0], vf[1]);
                    mma_bf16(acc[2 * v + 1], pf[kt], vf[2], vf[3]);
                }
        }
        __syncthreads();                           // the stage may be overwritten by the load of block blk + NS
    }

    // ---- merge the two key halves of each query tile, normalise, store
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1); l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1); l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    float* mO = reinterpret_cast<float*>(Sp) + mt * (16 * 64);            // [16 rows][64 columns] per query tile
    float* mML = reinterpret_cast<float*>(Sp) + 2 * 16 * 64 + mt * 32;    // [16 rows][maximum, sum]
    if (kh == 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            *reinterpret_cast<float2*>(mO + g * 64 + j * 8 + t4 * 2) = make_float2(acc[j][0], acc[j][1]);
            *reinterpret_cast<float2*>(mO + (g + 8) * 64 + j * 8 + t4 * 2) = make_float2(acc[j][2], acc[j][3]);
        }
        if (t4 == 0) {
            mML[g * 2] = m_run[0]; mML[g * 2 + 1] = l_run[0];
            mML[(g + 8) * 2] = m_run[1]; mML[(g + 8) * 2 + 1] = l_run[1];
        }
    }
    __syncthreads();
    if (kh == 0) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int rr = g + half * 8, r = mt * 16 + rr;
            const float m1 = mML[rr * 2], l1 = mML[rr * 2 + 1], m0 = m_run[half], l0 = l_run[half];
            const float m = fmaxf(m0, m1);
            const float f0 = (m0 == -CUDART_INF_F) ? 0.f : expf(m0 - m), f1 = (m1 == -CUDART_INF_F) ? 0.f : expf(m1 - m);
            const float den = l0 * f0 + l1 * f1, inv = den > 0.f ? 1.0f / den : 0.f;
            if (r < nq) {
                bf16* o = a.out + (size_t)(r0 + r) * a.out_stride + h * 64 + t4 * 2;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float2 o1 = *reinterpret_cast<const float2*>(mO + rr * 64 + j * 8 + t4 * 2);
                    const float x = acc[j][half * 2] * f0 + o1.x * f1, y = acc[j][half * 2 + 1] * f0 + o1.y * f1;
                    *reinterpret_cast<__nv_bfloat162*>(o + j * 8) = __floats2bfloat162_rn(x * inv, y * inv);
                }
            }
        }
    }
}

}  // namespace sd
