// Weight-streaming GEMM for a handful of activation rows (the library uses it for M <= 32):  C[r, n] = sum_k A[r, k] W[n, k].
//
// At batch 1 a verify block has k+1 = 26 rows, so every layer GEMM is a pass over its weight matrix
// bounded by HBM, not by math.  This kernel is shaped for that: one CTA per 8 weight rows, so a
// 512 x 512 projection already spreads over 64 SMs; the eight warps of a CTA split K, each lane
// streams 16-byte pieces of its weight rows straight from global memory into registers (all loads are
// issued before anything else happens), the activation rows sit in shared memory, and the products
// run on warp-level tensor-core MMAs (m16n8k16, fp32 accumulate) with the k index permuted so that a
// lane's 16 contiguous weight bytes are exactly its B fragments.  The K-split partial sums are added
// in a fixed order, so results do not depend on timing.
//
// Optionally the activation rows are produced in the prologue as LayerNorm(x) (fp32 residual rows in,
// bf16 operand rows into shared memory), which removes the separate normalisation launch and its
// round trip through HBM.  Epilogues: bias + store / ReLU / residual add / QKV with K,V scattered into
// the paged cache.
#pragma once
#include "attention_tc.cuh"
#include "gemm_tc.cuh"
#include "kernels.cuh"

namespace sd {

struct SkinnyArgs {
    GemmArgs<bf16> g;            // A (bf16 rows) unless ln_x is set; W, bias, N, K, n_rows and the epilogue fields
    const float* ln_x;           // LayerNorm prologue: fp32 rows [rows, K] ...
    const float* ln_g; const float* ln_b; float ln_eps;
    bf16* ln_out;                // ... optionally also written out as bf16 rows [rows, K] (by CTA 0)
    long long* trace;            // optional: CTA 0 records %globaltimer at a few points (debugging aid)
    int* err_word;               // raised when a bounded wait gives up
};

__device__ __forceinline__ void sk_stamp(long long* trace, int slot) {
    if (trace && blockIdx.x == 0 && threadIdx.x == 0) { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); trace[slot] = t; }
}

constexpr int SK_NB = 8;         // weight rows per 8-row group
constexpr int SK_WARPS = 8;
// G groups of 8 weight rows per CTA; the 8 warps are G groups x (8 / G) K-splits
// Row pitch of the activation tile in shared memory: K + 32 bf16, i.e. 16 words past a multiple of 32.  A quarter warp
// (rows g, g + 1 x the four 16-byte pieces of a super-step) then reads all 32 banks once per 16-byte load; with the
// earlier K + 8 and 8-byte loads every load was a 4-way bank conflict (the MMA phase of FFN2 took 2.6 us).
constexpr int SK_PAD = 32;
inline size_t skinny_smem(int MT, int K) { return (size_t)MT * 16 * (K + SK_PAD) * 2 + (size_t)SK_WARPS * MT * 16 * SK_NB * 4; }

// CL (with LN, clusters of 8 CTAs along the weight rows): every CTA of the grid needs the same normalised rows, and
// 200 CTAs each reading the same 26 x 2 KB at the same moment queue up on the same L2 lines.  With CL each CTA of a
// cluster normalises only the rows r, r + 8, ... (r = its cluster rank) and sends them to its seven peers'
// shared memory (st.async, counted on the receiver's mbarrier): one eighth of the L2 requests, and no CTA
// repeats another's arithmetic.
__device__ __forceinline__ void sk_st_peer(uint32_t local_addr, uint32_t local_bar, uint32_t rank, uint32_t lo, uint32_t hi) {
    uint32_t ra, rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];"
                 ::"r"(ra), "r"(lo), "r"(hi), "r"(rb) : "memory");
}

__device__ __forceinline__ void sk_st_peer16(uint32_t local_addr, uint32_t local_bar, uint32_t rank, uint4 v) {
    uint32_t ra, rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(ra), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(rb) : "memory");
}

template <int EPI, int MT, bool LN, int G, bool CL = false>
__global__ void __launch_bounds__(SK_WARPS * 32) k_skinny(SkinnyArgs a) {
    extern __shared__ __align__(16) unsigned char sk_sm[];
    const GemmArgs<bf16>& g = a.g;
    const int K = g.K, N = g.N;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t4 = lane & 3;
    sk_stamp(a.trace, 0);
    constexpr int SPL = SK_WARPS / G;                          // K-splits per group
    const int grp = warp % G, spl = warp / G;
    const int n0 = blockIdx.x * (SK_NB * G);                  // first weight row of this CTA
    const int pitch = K + SK_PAD;                             // bf16 elements per activation row in shared memory
    bf16* As = reinterpret_cast<bf16*>(sk_sm);
    float* red = reinterpret_cast<float*>(sk_sm + (size_t)MT * 16 * pitch * 2);

    // K split: warp s takes k in [s * ks, (s + 1) * ks), in super-steps of 32
    const int nsplit = min(SPL, K / 32);
    const int ks = (K / 32 + nsplit - 1) / nsplit * 32;
    const int k_begin = spl * ks, k_end = min(K, k_begin + ks);
    constexpr int MAX_SS = 8;                                 // super-steps whose weights are preloaded in registers
    uint4 wreg[MAX_SS];
    const bool w_ok = (n0 + grp * SK_NB + gq) < N;
    const bf16* wrow = g.W + (size_t)(n0 + grp * SK_NB + gq) * K + t4 * 8;
#pragma unroll
    for (int ss = 0; ss < MAX_SS; ++ss) {
        const int k0 = k_begin + ss * 32;
        wreg[ss] = (w_ok && spl < nsplit && k0 < k_end) ? ldg_pinned(reinterpret_cast<const uint4*>(wrow + k0)) : make_uint4(0, 0, 0, 0);
    }

    // bias and LayerNorm parameters are weights too: fetch them before waiting for the predecessor
    const float bias_v = (g.bias && n0 + (tid % (SK_NB * G)) < N) ? __ldg(g.bias + n0 + (tid % (SK_NB * G))) : 0.f;
    float4 lgam[4], lbet[4];
    if (LN) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int e = lane * 4 + c * 128;
            lgam[c] = e < K ? __ldg(reinterpret_cast<const float4*>(a.ln_g + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
            lbet[c] = e < K ? __ldg(reinterpret_cast<const float4*>(a.ln_b + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    __shared__ __align__(8) uint64_t row_bar;                 // CL: counts the peers' rows as they arrive
    __shared__ int row_abort;
    if constexpr (CL) {
        if (tid == 0) {
            row_abort = 0;
            mbar_init(smem_u32(&row_bar), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        tc_cluster_sync();                                    // every peer's barrier exists before anybody sends
    }
    // everything above touched only weights; from here on the predecessor's output is read
    sk_stamp(a.trace, 1);
    pdl_launch_dependents();
    pdl_wait();
    sk_stamp(a.trace, 2);
    const int R = min(g.rows_static >= 0 ? g.rows_static : *g.n_rows, MT * 16);   // a device-side count is itself written earlier in the step
    // residual epilogue with one output per thread: its old value is requested now, not after the products
    constexpr bool ONE_OUT = (MT * 16 * SK_NB * G == SK_WARPS * 32);
    float x_old = 0.f;
    if (EPI == EPI_RESID && ONE_OUT) {
        const int r = tid / (SK_NB * G), n = n0 + (tid % (SK_NB * G));
        if (r < R && n < N) x_old = g.resid[(size_t)r * N + n];
    }
    // ---- activation rows into shared memory
    if (LN && CL) {
        uint32_t rank;
        asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
        const int own = (R > (int)rank) ? (R - 1 - (int)rank) / 8 + 1 : 0;      // rows rank, rank + 8, ... below R
        if (tid == 0) mbar_expect_tx(smem_u32(&row_bar), (uint32_t)(R - own) * K * 2);
        const int m = (int)rank + 8 * warp;                   // warps 0..3: one row each (MT * 16 = 32 rows at most)
        if (warp < MT * 2 && m < R) {
            float4 xv[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = lane * 4 + c * 128;
                xv[c] = e < K ? *reinterpret_cast<const float4*>(a.ln_x + (size_t)m * K + e) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) sum += xv[c].x + xv[c].y + xv[c].z + xv[c].w;
            const float mu = warp_sum(sum) / K;
            float q = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (lane * 4 + c * 128 < K) {
                    const float c0 = xv[c].x - mu, c1 = xv[c].y - mu, c2 = xv[c].z - mu, c3 = xv[c].w - mu;
                    q += c0 * c0 + c1 * c1 + c2 * c2 + c3 * c3;
                }
            const float rstd = 1.0f / sqrtf(warp_sum(q) / K + a.ln_eps);
            bf16* dst = As + (size_t)m * pitch;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = lane * 4 + c * 128;
                if (e < K) {
                    const float4 v = xv[c];
                    const float4 gm = lgam[c], bt = lbet[c];
                    __nv_bfloat162 p0, p1;
                    p0.x = __float2bfloat16_rn((v.x - mu) * rstd * gm.x + bt.x); p0.y = __float2bfloat16_rn((v.y - mu) * rstd * gm.y + bt.y);
                    p1.x = __float2bfloat16_rn((v.z - mu) * rstd * gm.z + bt.z); p1.y = __float2bfloat16_rn((v.w - mu) * rstd * gm.w + bt.w);
                    const uint32_t lo = *reinterpret_cast<uint32_t*>(&p0), hi = *reinterpret_cast<uint32_t*>(&p1);
                    *reinterpret_cast<uint2*>(dst + e) = make_uint2(lo, hi);
                    const uint32_t la = smem_u32(dst + e);
#pragma unroll
                    for (uint32_t rk = 0; rk < 8; ++rk)
                        if (rk != rank) sk_st_peer(la, smem_u32(&row_bar), rk, lo, hi);
                }
            }
        }
        // rows past the end are zeroed locally by the idle warps
        for (int mm = R + warp; mm < MT * 16; mm += SK_WARPS)
            for (int c = lane; c < K / 8; c += 32) *reinterpret_cast<uint4*>(As + (size_t)mm * pitch + c * 8) = make_uint4(0, 0, 0, 0);
        mbar_wait(smem_u32(&row_bar), 0, &row_abort, a.err_word, 8);             // the peers' rows have landed
    } else if (LN) {
        // each warp normalises rows warp, warp + 8, ...; all of its rows are fetched first (one round trip)
        constexpr int RS = (MT * 16 + SK_WARPS - 1) / SK_WARPS;      // row slots per warp
        constexpr int CH = 4;                                        // float4 chunks per lane and row: K <= 512
        float4 xv[RS][CH];
#pragma unroll
        for (int s = 0; s < RS; ++s) {
            const int m = warp + s * SK_WARPS;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int e = lane * 4 + c * 128;
                xv[s][c] = (m < R && e < K) ? *reinterpret_cast<const float4*>(a.ln_x + (size_t)m * K + e) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int s = 0; s < RS; ++s) {
            const int m = warp + s * SK_WARPS;
            if (m >= MT * 16) continue;
            bf16* dst = As + (size_t)m * pitch;
            if (m < R) {
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < CH; ++c) sum += xv[s][c].x + xv[s][c].y + xv[s][c].z + xv[s][c].w;   // chunks past K are zero
                const float mu = warp_sum(sum) / K;
                float q = 0.f;
#pragma unroll
                for (int c = 0; c < CH; ++c)
                    if (lane * 4 + c * 128 < K) {
                        const float c0 = xv[s][c].x - mu, c1 = xv[s][c].y - mu, c2 = xv[s][c].z - mu, c3 = xv[s][c].w - mu;
                        q += c0 * c0 + c1 * c1 + c2 * c2 + c3 * c3;
                    }
                const float rstd = 1.0f / sqrtf(warp_sum(q) / K + a.ln_eps);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int e = lane * 4 + c * 128;
                    if (e < K) {
                        const float4 v = xv[s][c];
                        const float4 gm = lgam[c], bt = lbet[c];
                        __nv_bfloat162 p0, p1;
                        p0.x = __float2bfloat16_rn((v.x - mu) * rstd * gm.x + bt.x); p0.y = __float2bfloat16_rn((v.y - mu) * rstd * gm.y + bt.y);
                        p1.x = __float2bfloat16_rn((v.z - mu) * rstd * gm.z + bt.z); p1.y = __float2bfloat16_rn((v.w - mu) * rstd * gm.w + bt.w);
                        *reinterpret_cast<__nv_bfloat162*>(dst + e) = p0;
                        *reinterpret_cast<__nv_bfloat162*>(dst + e + 2) = p1;
                        if (a.ln_out && blockIdx.x == 0) {
                            *reinterpret_cast<__nv_bfloat162*>(a.ln_out + (size_t)m * K + e) = p0;
                            *reinterpret_cast<__nv_bfloat162*>(a.ln_out + (size_t)m * K + e + 2) = p1;
                        }
                    }
                }
            } else {
                for (int e = lane * 8; e < K; e += 256) *reinterpret_cast<uint4*>(dst + e) = make_uint4(0, 0, 0, 0);
            }
        }
    } else if (CL) {
        // plain rows, shared the same way: this CTA fetches rows rank, rank + 8, ... and sends them to its peers
        uint32_t rank;
        asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
        const int own = (R > (int)rank) ? (R - 1 - (int)rank) / 8 + 1 : 0;
        if (tid == 0) mbar_expect_tx(smem_u32(&row_bar), (uint32_t)(R - own) * K * 2);
        const int m = (int)rank + 8 * (warp >> 1), hf = warp & 1;     // two warps per row: halves of its 16-byte pieces
        if ((warp >> 1) < MT * 2 && m < R) {
            const int pieces = K / 8;                                 // 16-byte pieces per row
            for (int p0 = hf * 32 + lane; p0 < pieces; p0 += 64) {
                const uint4 v = *reinterpret_cast<const uint4*>(g.A + (size_t)m * g.lda + p0 * 8);
                bf16* dst = As + (size_t)m * pitch + p0 * 8;
                *reinterpret_cast<uint4*>(dst) = v;
                const uint32_t la = smem_u32(dst);
#pragma unroll
                for (uint32_t rk = 0; rk < 8; ++rk)
                    if (rk != rank) sk_st_peer16(la, smem_u32(&row_bar), rk, v);
            }
        }
        for (int mm = R + warp; mm < MT * 16; mm += SK_WARPS)
            for (int c = lane; c < K / 8; c += 32) *reinterpret_cast<uint4*>(As + (size_t)mm * pitch + c * 8) = make_uint4(0, 0, 0, 0);
        mbar_wait(smem_u32(&row_bar), 0, &row_abort, a.err_word, 8);
    } else {
        const uint32_t as_base = (uint32_t)__cvta_generic_to_shared(As);
        const int chunks = K / 8;
        // (row, 16-byte piece) of request i without an integer division where K / 8 is a power of two (it is for the
        // usual widths; up to 32 requests per thread when K = 2048)
        const bool p2 = (chunks & (chunks - 1)) == 0;
        const int sh = 31 - __clz(chunks);
        for (int i = tid; i < MT * 16 * chunks; i += SK_WARPS * 32) {
            const int m = p2 ? (i >> sh) : i / chunks, c = p2 ? (i & (chunks - 1)) : i % chunks;
            if (m < R) cp_async16(as_base + (uint32_t)(m * pitch + c * 8) * 2, g.A + (size_t)m * g.lda + c * 8);
            else *reinterpret_cast<uint4*>(As + (size_t)m * pitch + c * 8) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    sk_stamp(a.trace, 3);

    // ---- products: per super-step of 32 k, two MMAs per 16-row tile
    // four accumulator chains per 16-row tile (the two MMAs of a super-step x even / odd super-steps): an mma.sync takes
    // on the order of 100 clocks to return here, and one chain of 2 K / 32 / 8 dependent MMAs was most of this phase
    float acc4[MT][4][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc4[mt][c][e] = 0.f;
    if (spl < nsplit) {
        auto step = [&](const uint4& w, int k0, int par) {
            const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                // the lane's 8 consecutive k of rows g and g + 8: both MMAs of the super-step from one 16-byte load each
                const uint4 lo = *reinterpret_cast<const uint4*>(As + (size_t)(mt * 16 + gq) * pitch + k0 + t4 * 8);
                const uint4 hi = *reinterpret_cast<const uint4*>(As + (size_t)(mt * 16 + gq + 8) * pitch + k0 + t4 * 8);
                const uint32_t a0[4] = {lo.x, hi.x, lo.y, hi.y}, a1[4] = {lo.z, hi.z, lo.w, hi.w};
                mma_bf16(acc4[mt][par * 2], a0, wv[0], wv[1]);
                mma_bf16(acc4[mt][par * 2 + 1], a1, wv[2], wv[3]);
            }
        };
        // chunks of MAX_SS super-steps: the next chunk's weights are in flight while this one is multiplied
        for (int cb = k_begin; cb < k_end; cb += MAX_SS * 32) {
            uint4 wnext[MAX_SS];
            const int nb = cb + MAX_SS * 32;
#pragma unroll
            for (int ss = 0; ss < MAX_SS; ++ss) {
                const int k0 = nb + ss * 32;
                wnext[ss] = (w_ok && k0 < k_end) ? __ldg(reinterpret_cast<const uint4*>(wrow + k0)) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int ss = 0; ss < MAX_SS; ++ss) {
                const int k0 = cb + ss * 32;
                if (k0 < k_end) step(wreg[ss], k0, ss & 1);
            }
#pragma unroll
            for (int ss = 0; ss < MAX_SS; ++ss) wreg[ss] = wnext[ss];
        }
    }
    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][e] = (acc4[mt][0][e] + acc4[mt][1][e]) + (acc4[mt][2][e] + acc4[mt][3][e]);
    sk_stamp(a.trace, 4);
    // ---- fixed-order sum over the K split, then the epilogue
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        float* r0 = red + ((size_t)spl * MT * 16 + mt * 16 + gq) * (SK_NB * G) + grp * SK_NB + t4 * 2;
        r0[0] = acc[mt][0]; r0[1] = acc[mt][1];
        r0[8 * SK_NB * G] = acc[mt][2]; r0[8 * SK_NB * G + 1] = acc[mt][3];
    }
    __syncthreads();
    for (int o = tid; o < MT * 16 * SK_NB * G; o += SK_WARPS * 32) {
        const int r = o / (SK_NB * G), n = n0 + (o % (SK_NB * G));
        if (r >= R || n >= N) continue;
        float v = 0.f;
        for (int s = 0; s < nsplit; ++s) v += red[(size_t)s * MT * 16 * SK_NB * G + o];
        v += bias_v;
        if (EPI == EPI_STORE) g.out[(size_t)r * g.ldo + n] = __float2bfloat16_rn(v);
        if (EPI == EPI_RELU) g.out[(size_t)r * g.ldo + n] = __float2bfloat16_rn(fmaxf(v, 0.f));
        if (EPI == EPI_GELU) g.out[(size_t)r * g.ldo + n] = __float2bfloat16_rn(ffn_act(v, 1));
        if (EPI == EPI_RESID) { if (ONE_OUT) g.resid[(size_t)r * N + n] = x_old + v; else g.resid[(size_t)r * N + n] += v; }
        if (EPI == EPI_QKV) {
            if (n < g.kv_d) g.out[(size_t)r * g.ldo + n] = __float2bfloat16_rn(v);
            else {
                const size_t row = g.pg.row(g.seq[r], g.pos[r]);
                if (n < 2 * g.kv_d) g.kc[row * g.kv_d + (n - g.kv_d)] = __float2bfloat16_rn(v);
                else g.vc[row * g.kv_d + (n - 2 * g.kv_d)] = __float2bfloat16_rn(v);
            }
        }
    }
    sk_stamp(a.trace, 5);
}

}  // namespace sd
