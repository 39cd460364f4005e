// Kernels of the SpecDec draft/verify path other than the tensor-core GEMM:
// row preparation, embedding, layer norm, attention, the SIMT reference GEMM with
// the shared epilogues, vocabulary row statistics, the acceptance scan and commit.
// Every kernel takes its live row count from device memory and exits early past
// it, so the host can launch worst-case grids without knowing per-sequence lengths.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <math_constants.h>
#include <type_traits>

namespace sd {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }
// value as the operand type would hold it, back in fp32
template <typename T> __device__ __forceinline__ float round_as(float v) { return to_f(from_f<T>(v)); }

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start
// while its predecessor is still running.  pdl_wait() blocks until the predecessor grids have completed
// and their writes are visible; everything a kernel does before it must not depend on them (weights and
// constants only) and must not write global memory.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Read-only loads that must be ISSUED where they are written: a plain __ldg is a pure load the compiler may sink to its
// first use, i.e. past griddepcontrol.wait, which turns a prefetch issued under the predecessor's tail into a miss on the
// critical path.  A volatile asm keeps its place among the other volatile asms (the wait is one).
__device__ __forceinline__ uint4 ldg_pinned(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ldg_pinned(const float4* p) {
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float ldg_pinned(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One link of a chain of dependent launches (diagnostics: what one kernel boundary costs inside a step): waits for its
// predecessor, reads the word it wrote, and the first thread writes it back incremented.
__global__ void k_link(int* word) {
    pdl_launch_dependents();
    pdl_wait();
    const int v = *reinterpret_cast<volatile int*>(word);
    if (blockIdx.x == 0 && threadIdx.x == 0) *word = v + 1;
}

// Device-resident session state shared by the kernels of one handle.
struct Session {
    int* len;          // [B] committed target tokens j_b
    int* finished;     // [B]
    int* max_tgt;      // [B]
    int* src_len;      // [B]
    int* out;          // [B, out_stride] committed ids
    int out_stride;
    int* counters;     // [8]: 0 rows of the drafter's full pass, 1 rows of its mask-only pass,
                       //      2 verify rows, 3 encoder rows, 4 unfinished sequences
    unsigned long long* stats;  // [4]: seq_iterations, drafted, accepted, emitted
    int* dlen;         // [B] prefix-causal drafter: positions of [BOS, committed...] whose K/V its cache already holds
    int* dticket;      // [1] block ticket of the drafter's row preparation
};
enum { CNT_DRAFT_ALL = 0, CNT_DRAFT_MASK = 1, CNT_VERIFY = 2, CNT_ENC = 3, CNT_ACTIVE = 4, CNT_TICKET = 5, CNT_SEQ = 6 };

// Per-row metadata of the pass being run.
struct Rows {
    int* tok;       // token id fed at the row
    int* pos;       // position of the row
    int* seq;       // sequence the row belongs to
    int* nk_self;   // keys visible to the row in self-attention
    int* nk_cross;  // keys visible in cross-attention (source length)
    int* kv_off;    // [B] first K/V row of the sequence in a contiguous K/V buffer
    int* kv_off_cross;  // [B]
    int* src_row;   // mask-only pass: the row of the full pass this row continues
    int* slot;      // mask-only pass: index into the [B,k] draft array
    int* q_off;     // [B] first row of the sequence in this pass
    int* q_cnt;     // [B] rows of the sequence in this pass (0: none)
};

// ------------------------------------------------------------------ row preparation
// Encoder: rows are the padded [B,S_max] grid.
__global__ void k_enc_prep(const int* __restrict__ src, const int* __restrict__ src_len, int B, int S_max,
                           Rows r, int* counters) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) counters[CNT_ENC] = B * S_max;
    if (i < B) { r.kv_off[i] = i * S_max; r.kv_off_cross[i] = i * S_max; r.q_off[i] = i * S_max; r.q_cnt[i] = src_len[i]; }
    if (i >= B * S_max) return;
    int b = i / S_max, t = i % S_max;
    r.tok[i] = src[i];
    r.pos[i] = t;
    r.seq[i] = b;
    r.nk_self[i] = src_len[b];
    r.nk_cross[i] = src_len[b];
}

// Verify block: row b*(k+1)+i holds [last committed token (BOS if none), drafts] at positions j..j+k.
__global__ void k_verify_prep(Session s, const int* __restrict__ draft, int B, int k, int S_max, int bos,
                              Rows r) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) s.counters[CNT_VERIFY] = B * (k + 1);
    if (i < B) { r.kv_off_cross[i] = i * S_max; r.q_off[i] = i * (k + 1); r.q_cnt[i] = k + 1; }
    if (i >= B * (k + 1)) return;
    int b = i / (k + 1), c = i % (k + 1);
    int j = s.len[b];
    r.tok[i] = (c == 0) ? (j == 0 ? bos : s.out[(size_t)b * s.out_stride + j - 1]) : draft[b * k + c - 1];
    r.pos[i] = j + c;
    r.seq[i] = b;
    r.nk_self[i] = j + c + 1;     // causal: positions 0..j+c
    r.nk_cross[i] = s.src_len[b];
}

// The same, together with the embedding of the block's rows (x = sqrt(d) E[tok] + P[pos]): one block per row.  The row
// metadata is complete before the block lets its successors start, because kernels further down the chain read it
// ahead of their own dependency waits.
template <typename T>
__global__ void k_verify_prep_embed(Session s, const int* __restrict__ draft, int B, int k, int S_max, int bos, Rows r,
                                    const T* __restrict__ E, const float* __restrict__ P, float* __restrict__ x, int d,
                                    float scale, int vocab, int max_pos) {
    const int i = blockIdx.x;                      // row b * (k + 1) + c
    pdl_wait();                                    // session state comes from the previous step's commit
    const int b = i / (k + 1), c = i % (k + 1);
    const int j = s.len[b];
    const int tok = (c == 0) ? (j == 0 ? bos : s.out[(size_t)b * s.out_stride + j - 1]) : draft[b * k + c - 1];
    if (threadIdx.x == 0) {
        if (i == 0) s.counters[CNT_VERIFY] = B * (k + 1);
        if (c == 0) { r.kv_off_cross[b] = b * S_max; r.q_off[b] = b * (k + 1); r.q_cnt[b] = k + 1; }
        r.tok[i] = tok;
        r.pos[i] = j + c;
        r.seq[i] = b;
        r.nk_self[i] = j + c + 1;     // causal: positions 0..j+c
        r.nk_cross[i] = s.src_len[b];
        __threadfence();
    }
    __syncthreads();
    pdl_launch_dependents();
    const int t = min(max(tok, 0), vocab - 1), p = min(max(j + c, 0), max_pos - 1);
    for (int e = threadIdx.x; e < d; e += blockDim.x)
        x[(size_t)i * d + e] = scale * to_f(E[(size_t)t * d + e]) + P[(size_t)p * d + e];
}

// Embedding of the rows [r0, r0 + n) of the draft pass by the block that prepared them.
template <typename T>
__device__ __forceinline__ void embed_rows(const Rows& all, int r0, int n, const T* __restrict__ E, const float* __restrict__ P,
                                           float* __restrict__ x, int d, float scale, int vocab, int max_pos) {
    const int per_row = d / 4;                     // float4 pieces per row (d is a multiple of 16)
    for (int i = threadIdx.x; i < n * per_row; i += blockDim.x) {
        const int row = r0 + i / per_row, e = (i % per_row) * 4;
        const int t = min(max(all.tok[row], 0), vocab - 1), p = min(max(all.pos[row], 0), max_pos - 1);
        const T* ep = E + (size_t)t * d + e;
        const float4 pv = *reinterpret_cast<const float4*>(P + (size_t)p * d + e);
        float4 o;
        o.x = scale * to_f(ep[0]) + pv.x; o.y = scale * to_f(ep[1]) + pv.y; o.z = scale * to_f(ep[2]) + pv.z; o.w = scale * to_f(ep[3]) + pv.w;
        *reinterpret_cast<float4*>(x + (size_t)row * d + e) = o;
    }
}

// Drafter: packed rows [BOS, committed, MASK x k] of every unfinished sequence.
// `all` describes the full pass, `msk` the mask-only continuation of the last layer.
// gridDim.y blocks per sequence: each sums the row counts of the sequences before its own (B loads spread over its
// threads: the one-block version walked the batch serially, 106 us at 128 sequences), then fills an equal slice of the
// sequence's rows and embeds that slice (x = sqrt(d) E[tok] + P[pos]; one block per sequence made the embedding of a
// 90-row pass a 26 us serial walk).  Every block completes its metadata before it lets the successors start, because
// kernels further down the chain read it ahead of their dependency waits.
template <typename T>
__global__ void k_draft_prep(Session s, int B, int k, int S_max, int bos, int mask, Rows all, Rows msk,
                             const T* __restrict__ E, const float* __restrict__ P, float* __restrict__ x, int d, float scale,
                             int vocab, int max_pos) {
    __shared__ int red_a[32], red_m[32], tot_a[32], tot_l[32];
    const int b = blockIdx.x, part = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    pdl_wait();                                    // session state comes from the previous step's commit
    int a = 0, m = 0, ta = 0, tl = 0;               // rows / mask rows of the sequences before b; rows / live sequences of the batch
    for (int o = tid; o < B; o += blockDim.x) {
        const int n = s.finished[o] ? 0 : s.len[o] + 1 + k;
        ta += n; tl += n ? 1 : 0;
        if (o < b) { a += n; m += n ? k : 0; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o); m += __shfl_xor_sync(0xffffffffu, m, o);
        ta += __shfl_xor_sync(0xffffffffu, ta, o); tl += __shfl_xor_sync(0xffffffffu, tl, o);
    }
    if (lane == 0) { red_a[warp] = a; red_m[warp] = m; tot_a[warp] = ta; tot_l[warp] = tl; }
    __syncthreads();
    int off = 0, moff = 0, total = 0, live = 0;
    for (int w = 0; w < nw; ++w) { off += red_a[w]; moff += red_m[w]; total += tot_a[w]; live += tot_l[w]; }
    const bool fin = s.finished[b] != 0;
    const int j = s.len[b], n = fin ? 0 : j + 1 + k, sl = s.src_len[b];
    const int chunk = (n + (int)gridDim.y - 1) / (int)gridDim.y, t0 = min(n, part * chunk), t1 = min(n, t0 + chunk);
    if (tid == 0 && part == 0) {
        all.kv_off[b] = off; all.kv_off_cross[b] = b * S_max;
        msk.kv_off[b] = off; msk.kv_off_cross[b] = b * S_max;
        all.q_off[b] = off; all.q_cnt[b] = n;
        msk.q_off[b] = moff; msk.q_cnt[b] = fin ? 0 : k;
        if (b == 0) {
            s.counters[CNT_DRAFT_ALL] = total;
            s.counters[CNT_DRAFT_MASK] = live * k;  // k mask rows per unfinished sequence
        }
    }
    for (int t = t0 + tid; t < t1; t += blockDim.x) {
        const int row = off + t;
        all.tok[row] = (t == 0) ? bos : (t <= j ? s.out[(size_t)b * s.out_stride + t - 1] : mask);
        all.pos[row] = t;
        all.seq[row] = b;
        all.nk_self[row] = n;            // no causal mask: every valid position
        all.nk_cross[row] = sl;
    }
    for (int i = tid; i < ((fin || part) ? 0 : k); i += blockDim.x) {
        const int row = moff + i;
        msk.seq[row] = b;
        msk.nk_self[row] = n;
        msk.nk_cross[row] = sl;
        msk.src_row[row] = off + j + 1 + i;
        msk.slot[row] = b * k + i;
    }
    __threadfence();
    __syncthreads();
    pdl_launch_dependents();
    embed_rows<T>(all, off + t0, t1 - t0, E, P, x, d, scale, vocab, max_pos);
}

// Drafter, prefix-causal reading (the committed tokens attend causally among themselves and never see the [MASK]
// block, so their keys and values are cached like an autoregressive decoder's; Section 3.1.2: the drafter's decoder runs
// every iteration, so its work should not grow with the prefix).  Rows of sequence b: the positions the cache does not
// hold yet, c..j of [BOS, committed...], then k [MASK] rows at positions j+1..j+k.  Position p sees keys 0..p when it is
// a prefix row and every key 0..j+k when it is a [MASK] row.  The last block to finish records the new cache length.
template <typename T>
__global__ void k_draft_prep_pc(Session s, int B, int k, int S_max, int bos, int mask, Rows all, Rows msk,
                                const T* __restrict__ E, const float* __restrict__ P, float* __restrict__ x, int d, float scale,
                                int vocab, int max_pos) {
    __shared__ int red_a[32], red_m[32], tot_a[32], tot_l[32];
    __shared__ int last_s;
    const int b = blockIdx.x, part = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    pdl_wait();                                    // session state comes from the previous step's commit
    int a = 0, m = 0, ta = 0, tl = 0;
    for (int o = tid; o < B; o += blockDim.x) {
        const int n = s.finished[o] ? 0 : (s.len[o] + 1 - min(s.dlen[o], s.len[o] + 1)) + k;
        ta += n; tl += n ? 1 : 0;
        if (o < b) { a += n; m += n ? k : 0; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o); m += __shfl_xor_sync(0xffffffffu, m, o);
        ta += __shfl_xor_sync(0xffffffffu, ta, o); tl += __shfl_xor_sync(0xffffffffu, tl, o);
    }
    if (lane == 0) { red_a[warp] = a; red_m[warp] = m; tot_a[warp] = ta; tot_l[warp] = tl; }
    __syncthreads();
    int off = 0, moff = 0, total = 0, live = 0;
    for (int w = 0; w < nw; ++w) { off += red_a[w]; moff += red_m[w]; total += tot_a[w]; live += tot_l[w]; }
    const bool fin = s.finished[b] != 0;
    const int j = s.len[b], c = min(s.dlen[b], j + 1), n_new = j + 1 - c, n = fin ? 0 : n_new + k, sl = s.src_len[b];
    const int chunk = (n + (int)gridDim.y - 1) / (int)gridDim.y, t0 = min(n, part * chunk), t1 = min(n, t0 + chunk);
    if (tid == 0 && part == 0) {
        all.kv_off[b] = off; all.kv_off_cross[b] = b * S_max;
        msk.kv_off[b] = off; msk.kv_off_cross[b] = b * S_max;
        all.q_off[b] = off; all.q_cnt[b] = n;
        msk.q_off[b] = moff; msk.q_cnt[b] = fin ? 0 : k;
        if (b == 0) {
            s.counters[CNT_DRAFT_ALL] = total;
            s.counters[CNT_DRAFT_MASK] = live * k;
        }
    }
    if (!fin) {
        for (int t = t0 + tid; t < t1; t += blockDim.x) {
            const int row = off + t, p = c + t;
            all.tok[row] = (t >= n_new) ? mask : (p == 0 ? bos : s.out[(size_t)b * s.out_stride + p - 1]);
            all.pos[row] = p;
            all.seq[row] = b;
            all.nk_self[row] = (t >= n_new) ? j + 1 + k : p + 1;
            all.nk_cross[row] = sl;
        }
        for (int i = tid; i < (part ? 0 : k); i += blockDim.x) {
            const int row = moff + i;
            msk.seq[row] = b;
            msk.nk_self[row] = j + 1 + k;
            msk.nk_cross[row] = sl;
            msk.src_row[row] = off + n_new + i;
            msk.slot[row] = b * k + i;
        }
    }
    // every block has read the old cache lengths before any is overwritten
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        last_s = (atomicAdd(s.dticket, 1) == (int)(gridDim.x * gridDim.y) - 1) ? 1 : 0;
    }
    __syncthreads();
    if (last_s) {
        for (int o = tid; o < B; o += blockDim.x)
            if (!s.finished[o]) s.dlen[o] = s.len[o] + 1;
        if (tid == 0) *s.dticket = 0;
    }
    __threadfence();
    __syncthreads();
    pdl_launch_dependents();
    embed_rows<T>(all, off + t0, t1 - t0, E, P, x, d, scale, vocab, max_pos);
}

// ------------------------------------------------------------------ embedding, gather, layer norm
// x[row] = sqrt(d) * E[tok] + P[pos]
template <typename T>
__global__ void k_embed(const int* __restrict__ tok, const int* __restrict__ pos, const int* __restrict__ n_rows,
                        const T* __restrict__ E, const float* __restrict__ P, float* __restrict__ x, int d,
                        float scale, int vocab, int max_pos) {
    int row = blockIdx.x;
    pdl_launch_dependents();                       // writes x only, which every successor reads after its own wait
    pdl_wait();
    if (row >= *n_rows) return;
    int t = min(max(tok[row], 0), vocab - 1), p = min(max(pos[row], 0), max_pos - 1);
    for (int e = threadIdx.x; e < d; e += blockDim.x)
        x[(size_t)row * d + e] = scale * to_f(E[(size_t)t * d + e]) + P[(size_t)p * d + e];
}

__global__ void k_gather_rows(const float* __restrict__ x, const int* __restrict__ src_row,
                              const int* __restrict__ n_rows, float* __restrict__ out, int d) {
    int row = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    if (row >= *n_rows) return;
    const float* s = x + (size_t)src_row[row] * d;
    for (int e = threadIdx.x; e < d; e += blockDim.x) out[(size_t)row * d + e] = s[e];
}

// Register-resident row of up to NC * 128 elements (one warp per row).  gm / bt = this lane's gain and bias columns,
// fetched by the caller before the dependency wait (they are weights).
template <typename T, int NC>
__device__ __forceinline__ void ln_row_regs(const float* __restrict__ xr, const float4* gm, const float4* bt,
                                            T* __restrict__ y, int row, int d, float eps, int lane, bool store = true) {
    float4 v[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int e = lane * 4 + c * 128;
        v[c] = e < d ? *reinterpret_cast<const float4*>(xr + e) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) s += v[c].x + v[c].y + v[c].z + v[c].w;
    const float mu = warp_sum(s) / d;
    float q = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c)
        if (lane * 4 + c * 128 < d) {
            const float c0 = v[c].x - mu, c1 = v[c].y - mu, c2 = v[c].z - mu, c3 = v[c].w - mu;
            q += c0 * c0 + c1 * c1 + c2 * c2 + c3 * c3;
        }
    const float rstd = 1.0f / sqrtf(warp_sum(q) / d + eps);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int e = lane * 4 + c * 128;
        if (e < d && store) {
            T* o = y + (size_t)row * d + e;
            const float r0 = (v[c].x - mu) * rstd * gm[c].x + bt[c].x, r1 = (v[c].y - mu) * rstd * gm[c].y + bt[c].y;
            const float r2 = (v[c].z - mu) * rstd * gm[c].z + bt[c].z, r3 = (v[c].w - mu) * rstd * gm[c].w + bt[c].w;
            if constexpr (sizeof(T) == 2) {          // bf16: one 8-byte store per lane and chunk
                __nv_bfloat162 p0 = __floats2bfloat162_rn(r0, r1), p1 = __floats2bfloat162_rn(r2, r3);
                *reinterpret_cast<uint2*>(o) = make_uint2(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1));
            } else {
                *reinterpret_cast<float4*>(o) = make_float4(r0, r1, r2, r3);
            }
        }
    }
}

// One warp per row; biased variance, eps inside the square root.  Rows of up to 1024 elements
// (a multiple of 128) are held in registers, so the row is read from memory once.
template <typename T>
__global__ void k_layernorm(const float* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b,
                            const int* __restrict__ n_rows, T* __restrict__ y, int d, float eps, int rows_static) {
    // rows_static >= 0: the row count is known on the host (saves the dependent load of n_rows in front of the row's own)
    int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    const bool regs4 = d % 128 == 0 && d <= 512, regs8 = d % 128 == 0 && d <= 1024;
    float4 gm[8], bt[8];                             // gain and bias are weights: fetched before the dependency wait
    if (regs8) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int e = lane * 4 + c * 128;
            if (c < 4 || !regs4) {
                gm[c] = e < d ? __ldg(reinterpret_cast<const float4*>(g + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
                bt[c] = e < d ? __ldg(reinterpret_cast<const float4*>(b + e)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
    pdl_launch_dependents();
    pdl_wait();
    if (row >= (rows_static >= 0 ? rows_static : *n_rows)) return;
    const float* xr = x + (size_t)row * d;
    if (regs4) { ln_row_regs<T, 4>(xr, gm, bt, y, row, d, eps, lane); return; }
    if (regs8) { ln_row_regs<T, 8>(xr, gm, bt, y, row, d, eps, lane); return; }
    float s = 0.f;
    for (int e = lane; e < d; e += 32) s += xr[e];
    float mu = warp_sum(s) / d;
    float v = 0.f;
    for (int e = lane; e < d; e += 32) { float c = xr[e] - mu; v += c * c; }
    float rstd = 1.0f / sqrtf(warp_sum(v) / d + eps);
    for (int e = lane; e < d; e += 32) y[(size_t)row * d + e] = from_f<T>((xr[e] - mu) * rstd * g[e] + b[e]);
}

// Final LayerNorm of the verify rows together with the pre-pass logit of each row's draft (the dot product of the
// normalised, operand-rounded row with the draft's embedding row): one warp per row, rows of d = 128 NC elements in registers.
template <typename T, int NC>
__global__ void k_layernorm_ld(const float* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b,
                               T* __restrict__ y, int d, float eps, const T* __restrict__ E, const int* __restrict__ draft,
                               int B, int k, int vocab, float* __restrict__ ld, int* __restrict__ ld_id) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    float4 gm[NC], bt[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int e = lane * 4 + c * 128;
        gm[c] = __ldg(reinterpret_cast<const float4*>(g + e));
        bt[c] = __ldg(reinterpret_cast<const float4*>(b + e));
    }
    const bool in_range = row < B * (k + 1);
    const int bs = in_range ? row / (k + 1) : 0, c0 = in_range ? row % (k + 1) : k;
    const int tok = (in_range && c0 < k) ? draft[bs * k + c0] : -1;       // drafts predate the step's kernel chain
    const bool ok = tok >= 0 && tok < vocab;
    pdl_launch_dependents();
    pdl_wait();
    if (!in_range) return;
    const float* xr = x + (size_t)row * d;
    float4 v[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) v[c] = *reinterpret_cast<const float4*>(xr + lane * 4 + c * 128);
    float sm = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) sm += v[c].x + v[c].y + v[c].z + v[c].w;
    const float mu = warp_sum(sm) / d;
    float q = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const float a0 = v[c].x - mu, a1 = v[c].y - mu, a2 = v[c].z - mu, a3 = v[c].w - mu;
        q += a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3;
    }
    const float rstd = 1.0f / sqrtf(warp_sum(q) / d + eps);
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int e = lane * 4 + c * 128;
        T o[4];
        o[0] = from_f<T>((v[c].x - mu) * rstd * gm[c].x + bt[c].x);
        o[1] = from_f<T>((v[c].y - mu) * rstd * gm[c].y + bt[c].y);
        o[2] = from_f<T>((v[c].z - mu) * rstd * gm[c].z + bt[c].z);
        o[3] = from_f<T>((v[c].w - mu) * rstd * gm[c].w + bt[c].w);
        T* yo = y + (size_t)row * d + e;
        yo[0] = o[0]; yo[1] = o[1]; yo[2] = o[2]; yo[3] = o[3];
        if (ok) {
            const T* ep = E + (size_t)tok * d + e;
#pragma unroll
            for (int i = 0; i < 4; ++i) dot = fmaf(to_f(o[i]), to_f(ep[i]), dot);
        }
    }
    dot = warp_sum(dot);
    if (lane == 0) {
        if (c0 == k) { ld[row] = CUDART_INF_F; ld_id[row] = -1; }
        else { ld[row] = ok ? dot : -CUDART_INF_F; ld_id[row] = ok ? tok : -2; }
    }
}

// ------------------------------------------------------------------ paged KV cache
struct Paged {
    const int* table;   // [B, max_pages] page ids
    int page_tokens, max_pages;
    // page_tokens is a power of two (checked when the handle is created): shift and mask, no integer division
    __device__ __forceinline__ size_t row(int b, int t) const {
        const int sh = 31 - __clz(page_tokens);
        return ((size_t)table[b * max_pages + (t >> sh)] << sh) + (size_t)(t & (page_tokens - 1));
    }
};

// Writes the K and V parts of the verify block's QKV rows to their cache positions.
template <typename T>
__global__ void k_kv_scatter(const T* __restrict__ qkv, const int* __restrict__ seq, const int* __restrict__ pos,
                             const int* __restrict__ n_rows, Paged pg, T* __restrict__ kc, T* __restrict__ vc, int d) {
    int row = blockIdx.x;
    if (row >= *n_rows) return;
    size_t dst = pg.row(seq[row], pos[row]) * d;
    const T* s = qkv + (size_t)row * 3 * d;
    for (int e = threadIdx.x; e < d; e += blockDim.x) { kc[dst + e] = s[d + e]; vc[dst + e] = s[2 * d + e]; }
}

// ------------------------------------------------------------------ attention
// One warp per (row, head).  Scores of all visible keys are held in shared memory, so the
// softmax uses the true row maximum; the un-normalised probabilities are rounded to the
// operand type before the weighted sum and normalised by the sum of the unrounded ones.
template <typename T>
struct AttnArgs {
    const T* q; int q_stride; const int* q_index;       // row r reads q + (q_index ? q_index[r] : r) * q_stride
    const T* k; const T* v; int kv_stride;              // contiguous: key t of seq b at (kv_off[b] + t) * kv_stride
    const int* kv_off;
    Paged pg;                                            // paged: row pg.row(b, t) * kv_stride
    const int* seq; const int* nkeys; const int* n_rows;
    T* out; int out_stride;
    int n_heads, d_head, max_keys;
    float scale;
};

template <typename T, bool PAGED>
__global__ void k_attention(AttnArgs<T> a) {
    extern __shared__ float sm_att[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, wpb = blockDim.x >> 5;
    long long gw = (long long)blockIdx.x * wpb + warp;
    int r = (int)(gw / a.n_heads), h = (int)(gw % a.n_heads);
    if (r >= *a.n_rows) return;
    const int dh = a.d_head;
    float* sc = sm_att + (size_t)warp * (a.max_keys + dh);
    float* qs = sc + a.max_keys;
    const int b = a.seq[r];
    const int nk = min(a.nkeys[r], a.max_keys);
    const T* qp = a.q + (size_t)(a.q_index ? a.q_index[r] : r) * a.q_stride + h * dh;
    for (int e = lane; e < dh; e += 32) qs[e] = to_f(qp[e]);
    __syncwarp();
    float mx = -CUDART_INF_F;
    for (int t = lane; t < nk; t += 32) {
        size_t kr = PAGED ? a.pg.row(b, t) : (size_t)(a.kv_off[b] + t);
        const T* kp = a.k + kr * a.kv_stride + h * dh;
        float s = 0.f;
        for (int e = 0; e < dh; ++e) s = fmaf(qs[e], to_f(kp[e]), s);
        s *= a.scale;
        sc[t] = s;
        mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int t = lane; t < nk; t += 32) {
        float e = expf(sc[t] - mx);
        sum += e;
        sc[t] = round_as<T>(e);
    }
    sum = warp_sum(sum);
    __syncwarp();
    T* op = a.out + (size_t)r * a.out_stride + h * dh;
    for (int e = lane; e < dh; e += 32) {
        float acc = 0.f;
        for (int t = 0; t < nk; ++t) {
            size_t vr = PAGED ? a.pg.row(b, t) : (size_t)(a.kv_off[b] + t);
            acc = fmaf(sc[t], to_f(a.v[vr * a.kv_stride + h * dh + e]), acc);
        }
        op[e] = from_f<T>(nk > 0 ? acc / sum : 0.f);
    }
}

// ------------------------------------------------------------------ GEMM epilogues
// C[r, n] = sum_k A[r, k] * W[n, k]  (+ bias[n])
enum { EPI_STORE = 0, EPI_RELU = 1, EPI_RESID = 2, EPI_STATS = 3, EPI_F32 = 4, EPI_QKV = 5, EPI_GELU = 6 };   // EPI_RELU / EPI_GELU = the feed-forward activation (separate kernels: erff costs registers)

// Feed-forward activation of EPI_RELU: ReLU (act = 0) or the exact GELU x * Phi(x) (act = 1).
__device__ __forceinline__ float ffn_act(float x, int act) {
    return act ? 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)) : fmaxf(x, 0.f);
}

// Partial statistics of one verifier (or drafter) row over one tile of vocabulary columns.
struct __align__(16) RowPart { float mx; int arg; float sum; int cnt; };

template <typename T>
struct GemmArgs {
    const T* A; int lda;
    const T* W;                 // [N, K]
    const float* bias;          // [N] or null
    int N, K;
    const int* n_rows;          // device row count
    int rows_static;            // >= 0: the row count is known on the host (saves a dependent load); else read n_rows
    int one_m_tile;             // tensor-core path: the rows fit one 128-row tile whatever n_rows says
    T* out; int ldo;            // EPI_STORE / EPI_RELU
    int act;                    // EPI_RELU: 0 ReLU, 1 exact GELU
    // EPI_RESID on the tensor-core path, optional: also write LayerNorm(new residual rows) as bf16 [rows, N]
    const float* ln_g; const float* ln_b; float ln_eps; T* ln_out;
    float* resid;               // EPI_RESID: resid[r, n] += value ; EPI_F32: resid[r, n] = value (ld = N)
    // EPI_STATS
    RowPart* part; int n_tiles; // part[r * n_tiles + tile]
    const float* ld;            // [rows] logit of the row's draft from the pre-pass (+inf: none)
    const int* ld_id;           // [rows] the draft's id (-1: none)
    int want_sum;               // also accumulate sum exp(l - max) (only needed to report log-probabilities)
    // EPI_QKV: columns [0, kv_d) are stored like EPI_STORE, [kv_d, 2 kv_d) go to the K cache and
    // [2 kv_d, 3 kv_d) to the V cache at the row's (sequence, position)
    const int* seq; const int* pos; Paged pg; T* kc; T* vc; int kv_d;
    long long* trace;           // optional: CTA 0 records %globaltimer at a few points (debugging aid)
};

// Merge of (max, argmax, count) only: used on the hot path, where the sum is not needed.
__device__ __forceinline__ void part_merge_nosum(RowPart& a, const RowPart& b) {
    if (b.mx > a.mx || (b.mx == a.mx && b.arg < a.arg)) { a.mx = b.mx; a.arg = b.arg; }
    a.cnt += b.cnt;
}

// Merge order of row statistics: larger maximum wins, equal maxima keep the lower id.
__device__ __forceinline__ void part_merge(RowPart& a, const RowPart& b) {
    float m = fmaxf(a.mx, b.mx);
    float sa = (a.mx == -CUDART_INF_F) ? 0.f : a.sum * expf(a.mx - m);
    float sb = (b.mx == -CUDART_INF_F) ? 0.f : b.sum * expf(b.mx - m);
    if (b.mx > a.mx || (b.mx == a.mx && b.arg < a.arg)) a.arg = b.arg;
    a.mx = m;
    a.sum = sa + sb;
    a.cnt += b.cnt;
}

// ------------------------------------------------------------------ SIMT reference GEMM
// 64x64x16 tiles, 256 threads, 4x4 outputs per thread; used by the fp32 path and as the
// on-device cross-check of the tensor-core GEMM.
template <typename T, int EPI>
__global__ void __launch_bounds__(256) k_gemm_simt(GemmArgs<T> g) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    __shared__ float Ct[(EPI == EPI_STATS) ? BM : 1][(EPI == EPI_STATS) ? BN + 1 : 1];
    const int R = *g.n_rows;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (m0 >= R) return;
    const int tid = threadIdx.x;
    const int lr = tid >> 2, lk = (tid & 3) * 4;       // loader: row lr, k offset lk..lk+3
    const int ty = tid >> 4, tx = tid & 15;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const bool a_ok = (m0 + lr) < R, w_ok = (n0 + lr) < g.N;
    const T* ap = g.A + (size_t)(m0 + lr) * g.lda + lk;
    const T* wp = g.W + (size_t)(n0 + lr) * g.K + lk;
    for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            As[lk + e][lr] = a_ok ? to_f(ap[k0 + e]) : 0.f;
            Ws[lk + e][lr] = w_ok ? to_f(wp[k0 + e]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; wv[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = m0 + ty * 4 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            float v = acc[i][j] + ((g.bias && n < g.N) ? g.bias[n] : 0.f);
            if (EPI == EPI_STATS) {
                Ct[ty * 4 + i][tx * 4 + j] = v;
            } else if (r < R && n < g.N) {
                if (EPI == EPI_STORE) g.out[(size_t)r * g.ldo + n] = from_f<T>(v);
                if (EPI == EPI_RELU) g.out[(size_t)r * g.ldo + n] = from_f<T>(ffn_act(v, g.act));
                if (EPI == EPI_RESID) g.resid[(size_t)r * g.N + n] += v;
                if (EPI == EPI_F32) g.resid[(size_t)r * g.N + n] = v;
            }
        }
    }
    if (EPI == EPI_STATS) {
        __syncthreads();
        if (tid < BM && m0 + tid < R) {
            const int r = m0 + tid;
            const float ld = g.ld ? g.ld[r] : CUDART_INF_F;
            const int id = g.ld_id ? g.ld_id[r] : -1;
            RowPart p; p.mx = -CUDART_INF_F; p.arg = 0x7fffffff; p.sum = 0.f; p.cnt = 0;
            const int nn = min(BN, g.N - n0);
            for (int j = 0; j < nn; ++j) {
                float v = Ct[tid][j];
                if (n0 + j == id) v = ld;             // the draft's column takes the pre-pass value
                if (v > p.mx) { p.mx = v; p.arg = n0 + j; }
                p.cnt += (v > ld) ? 1 : 0;
            }
            if (g.want_sum)
                for (int j = 0; j < nn; ++j) {
                    float v = (n0 + j == id) ? ld : Ct[tid][j];
                    p.sum += expf(v - p.mx);
                }
            g.part[(size_t)r * g.n_tiles + blockIdx.x] = p;
        }
    }
}

// ------------------------------------------------------------------ verify: draft logit pre-pass
// Row c < k of a sequence checks draft c+1: its logit is the dot product of the row's
// normalised hidden state with the draft's embedding row.  Row k (bonus) has no draft.
template <typename T>
__global__ void k_draft_logit(const T* __restrict__ y, const T* __restrict__ E, const int* __restrict__ draft,
                              int B, int k, int d, int vocab, float* __restrict__ ld, int* __restrict__ ld_id) {
    int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    // The draft ids were written before this step's kernel chain began and the embedding table is a weight: with bf16
    // rows of at most 512 columns a lane fetches its 16 columns of the draft's embedding row before the dependency wait.
    const bool vec = std::is_same<T, bf16>::value && d % 16 == 0 && d <= 512;
    const bool in_range = row < B * (k + 1);
    const int b = in_range ? row / (k + 1) : 0, c = in_range ? row % (k + 1) : k;
    const int tok = (in_range && c < k) ? draft[b * k + c] : -1;
    const bool ok = tok >= 0 && tok < vocab;
    uint4 ev[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
    if (vec && ok && lane * 16 < d) {
        const uint4* ep = reinterpret_cast<const uint4*>(E + (size_t)tok * d + lane * 16);
        ev[0] = __ldg(ep); ev[1] = __ldg(ep + 1);
    }
    pdl_launch_dependents();
    pdl_wait();
    if (!in_range) return;
    if (c == k) { if (lane == 0) { ld[row] = CUDART_INF_F; ld_id[row] = -1; } return; }
    float s = 0.f;
    if (vec) {
        if (ok && lane * 16 < d) {
            const uint4* yp = reinterpret_cast<const uint4*>(y + (size_t)row * d + lane * 16);
            const uint4 yv[2] = {yp[0], yp[1]};
            const __nv_bfloat162* e2 = reinterpret_cast<const __nv_bfloat162*>(ev);
            const __nv_bfloat162* y2 = reinterpret_cast<const __nv_bfloat162*>(yv);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float2 a = __bfloat1622float2(y2[i]), w = __bfloat1622float2(e2[i]);
                s = fmaf(a.x, w.x, s); s = fmaf(a.y, w.y, s);
            }
        }
    } else if (ok) {
        for (int e = lane; e < d; e += 32) s = fmaf(to_f(y[(size_t)row * d + e]), to_f(E[(size_t)tok * d + e]), s);
    }
    s = warp_sum(s);
    if (lane == 0) { ld[row] = ok ? s : -CUDART_INF_F; ld_id[row] = ok ? tok : -2; }
}

// ------------------------------------------------------------------ commit / rollback (Eq. 3)
// Appends drafts[0..keep) and the next token to sequence b, cuts after the first EOS and at max_tgt.
// Cache rows beyond the new length are simply dead: the next block overwrites them.
__device__ __forceinline__ void commit_sequence(const Session& s, int b, const int* __restrict__ draft, int keep, int next,
                                                int k, int eos) {
    if (s.finished[b]) return;
    int j = s.len[b];
    const int mt = s.max_tgt[b];
    const int a = min(max(keep, 0), k);
    bool fin = false;
    const int n0 = j;
    for (int c = 0; c <= a && !fin; ++c) {
        if (j >= mt) { fin = true; break; }
        const int tok = (c < a) ? draft[b * k + c] : next;
        s.out[(size_t)b * s.out_stride + j] = tok;
        ++j;
        if (tok == eos) fin = true;
    }
    if (j >= mt) fin = true;
    s.len[b] = j;
    atomicAdd(&s.stats[0], 1ull);
    atomicAdd(&s.stats[1], (unsigned long long)k);
    atomicAdd(&s.stats[2], (unsigned long long)a);
    atomicAdd(&s.stats[3], (unsigned long long)(j - n0));
    if (fin) { s.finished[b] = 1; atomicSub(&s.counters[CNT_ACTIVE], 1); }
}
// The last block of the grid to get here posts (commits of this handle so far) << 32 | (sequences still decoding) to the
// host-mapped word the generation loop polls: no copy, no event between the iterations.  Call after __syncthreads().
__device__ __forceinline__ void commit_post(const Session& s, unsigned long long* post) {
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&s.counters[CNT_TICKET], 1) == (int)gridDim.x - 1) {
            s.counters[CNT_TICKET] = 0;
            const int seq = ++s.counters[CNT_SEQ];
            const int active = atomicAdd(&s.counters[CNT_ACTIVE], 0);
            *reinterpret_cast<volatile unsigned long long*>(post) = ((unsigned long long)(unsigned)seq << 32) | (unsigned)active;
            __threadfence_system();
        }
    }
}
// What the acceptance scan needs to commit its own decision (the generation loop): on = 0 leaves the commit to k_commit.
struct FusedCommit { Session s; const int* draft; int eos; unsigned long long* post; int on; };

// ------------------------------------------------------------------ acceptance scan (Eq. 7-9)
// One block per sequence: warps merge the per-tile statistics of the k+1 rows, thread 0
// finds the first rejected draft.  row_stats (optional) receives 6 floats per row.
__global__ void k_accept(const RowPart* __restrict__ part, int n_tiles, const float* __restrict__ ld,
                         const int* __restrict__ ld_id, int k, int beta, float tau, int* __restrict__ accepted,
                         int* __restrict__ bif, float* __restrict__ row_stats, int want_sum, FusedCommit fc) {
    extern __shared__ unsigned char sm_acc[];
    RowPart* rs = reinterpret_cast<RowPart*>(sm_acc);       // [k+1]
    __shared__ unsigned char ok_s[256];                     // row c passes both tests (k <= 255 rows take this path)
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    pdl_launch_dependents();
    pdl_wait();
    for (int c = warp; c <= k; c += nw) {
        const RowPart* p = part + ((size_t)b * (k + 1) + c) * n_tiles;
        // the draft's logit of this row is requested with the first partials, not by the serial scan afterwards
        const float l = (lane == 0 && c < k) ? ld[b * (k + 1) + c] : 0.f;
        RowPart m; m.mx = -CUDART_INF_F; m.arg = 0x7fffffff; m.sum = 0.f; m.cnt = 0;
        if (want_sum) {
            for (int t = lane; t < n_tiles; t += 32) part_merge(m, p[t]);
        } else {
            int t = lane;
            for (; t + 224 < n_tiles; t += 256) {           // eight independent loads in flight
                RowPart q[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) q[i] = p[t + 32 * i];
#pragma unroll
                for (int i = 0; i < 8; ++i) part_merge_nosum(m, q[i]);
            }
            for (; t + 96 < n_tiles; t += 128) {
                const RowPart q0 = p[t], q1 = p[t + 32], q2 = p[t + 64], q3 = p[t + 96];
                part_merge_nosum(m, q0); part_merge_nosum(m, q1); part_merge_nosum(m, q2); part_merge_nosum(m, q3);
            }
            for (; t < n_tiles; t += 32) part_merge_nosum(m, p[t]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            RowPart q;
            q.mx = __shfl_xor_sync(0xffffffffu, m.mx, o);
            q.arg = __shfl_xor_sync(0xffffffffu, m.arg, o);
            q.sum = __shfl_xor_sync(0xffffffffu, m.sum, o);
            q.cnt = __shfl_xor_sync(0xffffffffu, m.cnt, o);
            if (want_sum) part_merge(m, q); else part_merge_nosum(m, q);
        }
        if (lane == 0) {
            rs[c] = m;
            if (c < 256) ok_s[c] = (c < k && (m.cnt <= beta - 1) && ((m.mx - l) <= tau)) ? 1 : 0;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int a = 0;
        for (int c = 0; c < k; ++c) {
            bool ok;
            if (c < 256) ok = ok_s[c] != 0;
            else { const float l = ld[b * (k + 1) + c]; ok = (rs[c].cnt <= beta - 1) && ((rs[c].mx - l) <= tau); }
            if (!ok) break;
            ++a;
        }
        accepted[b] = a;
        bif[b] = rs[a].arg;
        if (fc.on) commit_sequence(fc.s, b, fc.draft, a, rs[a].arg, k, fc.eos);
    }
    if (row_stats)
        for (int c = threadIdx.x; c <= k; c += blockDim.x) {
            float* o = row_stats + ((size_t)b * (k + 1) + c) * 6;
            o[0] = rs[c].mx; o[1] = (float)rs[c].arg; o[2] = want_sum ? rs[c].mx + logf(rs[c].sum) : 0.f;
            o[3] = (float)rs[c].cnt; o[4] = ld[b * (k + 1) + c]; o[5] = (float)ld_id[b * (k + 1) + c];
        }
    if (fc.on) { __syncthreads(); commit_post(fc.s, fc.post); }
}

// The same rule on caller-provided logits [B, k+1, V]: one block per sequence walks the rows
// in order and stops at the first rejected draft, so it needs no scratch memory.
__global__ void k_accept_logits(const float* __restrict__ logits, const int* __restrict__ draft, int k, int V,
                                int beta, float tau, int* __restrict__ accepted, int* __restrict__ bif) {
    __shared__ RowPart wsm[32];
    __shared__ int stop;
    const int b = blockIdx.x;
    for (int c = 0; c <= k; ++c) {
        const float* l = logits + ((size_t)b * (k + 1) + c) * V;
        const int tok = (c < k) ? draft[b * k + c] : -1;
        const float ld = (c == k) ? CUDART_INF_F : ((tok >= 0 && tok < V) ? l[tok] : -CUDART_INF_F);
        RowPart m; m.mx = -CUDART_INF_F; m.arg = 0x7fffffff; m.sum = 0.f; m.cnt = 0;
        for (int v = threadIdx.x; v < V; v += blockDim.x) {
            RowPart q; q.mx = l[v]; q.arg = v; q.sum = 1.f; q.cnt = (l[v] > ld) ? 1 : 0;
            part_merge(m, q);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            RowPart q;
            q.mx = __shfl_xor_sync(0xffffffffu, m.mx, o);
            q.arg = __shfl_xor_sync(0xffffffffu, m.arg, o);
            q.sum = __shfl_xor_sync(0xffffffffu, m.sum, o);
            q.cnt = __shfl_xor_sync(0xffffffffu, m.cnt, o);
            part_merge(m, q);
        }
        if ((threadIdx.x & 31) == 0) wsm[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < (int)(blockDim.x >> 5); ++w) part_merge(m, wsm[w]);
            const bool ok = (c < k) && (m.cnt <= beta - 1) && ((m.mx - ld) <= tau);
            stop = ok ? 0 : 1;
            if (!ok) { accepted[b] = c; bif[b] = m.arg; }
        }
        __syncthreads();
        if (stop) return;
    }
}

// Per (row, tile of `tile` columns) statistics of caller-provided logits [rows, V]: the first stage of the
// two-stage acceptance scan whose partials live in the library's static scratch array.
__global__ void k_logit_tile_stats(const float* __restrict__ logits, const int* __restrict__ draft, int k, int V,
                                   int tile, int n_tiles, RowPart* __restrict__ part, float* __restrict__ ld_out,
                                   int* __restrict__ id_out) {
    __shared__ RowPart wsm[32];
    const int row = blockIdx.y, t = blockIdx.x, b = row / (k + 1), c = row % (k + 1);
    const float* l = logits + (size_t)row * V;
    const int tok = (c < k) ? draft[b * k + c] : -1;
    const bool ok = tok >= 0 && tok < V;
    const float ld = (c == k) ? CUDART_INF_F : (ok ? l[tok] : -CUDART_INF_F);
    RowPart m; m.mx = -CUDART_INF_F; m.arg = 0x7fffffff; m.sum = 0.f; m.cnt = 0;
    const int v1 = min(V, (t + 1) * tile);
    for (int v = t * tile + threadIdx.x; v < v1; v += blockDim.x) {
        RowPart q; q.mx = l[v]; q.arg = v; q.sum = 1.f; q.cnt = (l[v] > ld) ? 1 : 0;
        part_merge(m, q);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        RowPart q;
        q.mx = __shfl_xor_sync(0xffffffffu, m.mx, o);
        q.arg = __shfl_xor_sync(0xffffffffu, m.arg, o);
        q.sum = __shfl_xor_sync(0xffffffffu, m.sum, o);
        q.cnt = __shfl_xor_sync(0xffffffffu, m.cnt, o);
        part_merge(m, q);
    }
    if ((threadIdx.x & 31) == 0) wsm[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) part_merge(m, wsm[w]);
        part[(size_t)row * n_tiles + t] = m;
        if (t == 0) { ld_out[row] = ld; id_out[row] = (c == k) ? -1 : (ok ? tok : -2); }
    }
}

// ------------------------------------------------------------------ drafter argmax
// script (optional; benchmark / test hook): draft i of a sequence with j committed tokens is replaced by
// script[b * stride + j + i] wherever that entry is >= 0 (len = the committed lengths, k = drafts per sequence).
__global__ void k_draft_argmax(const RowPart* __restrict__ part, int n_tiles, const int* __restrict__ n_rows,
                               const int* __restrict__ slot, int* __restrict__ draft, const int* __restrict__ script,
                               int stride, const int* __restrict__ len, int k) {
    int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();
    if (row >= *n_rows) return;
    const RowPart* p = part + (size_t)row * n_tiles;
    float mx = -CUDART_INF_F; int arg = 0x7fffffff;
    const int slot_of_row = slot[row];              // written before the step's kernel chain; requested with the partials
    int t = lane;
    for (; t + 224 < n_tiles; t += 256) {           // eight independent loads in flight (merge order unchanged)
        RowPart q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = p[t + 32 * i];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (q[i].mx > mx || (q[i].mx == mx && q[i].arg < arg)) { mx = q[i].mx; arg = q[i].arg; }
    }
    for (; t < n_tiles; t += 32) {
        RowPart q = p[t];
        if (q.mx > mx || (q.mx == mx && q.arg < arg)) { mx = q.mx; arg = q.arg; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float om = __shfl_xor_sync(0xffffffffu, mx, o);
        int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
    }
    if (lane == 0) {
        if (script) {
            const int b = slot_of_row / k, pos = len[b] + slot_of_row % k;
            if (pos < stride) { const int t2 = script[(size_t)b * stride + pos]; if (t2 >= 0) arg = t2; }
        }
        draft[slot_of_row] = arg;
    }
}

// Scripted drafts (benchmark / test hook): draft i of a sequence with j committed tokens is
// replaced by script[b, j + i] where that entry is >= 0.  The drafter pass has already run.
__global__ void k_apply_script(Session s, const int* __restrict__ script, int stride, int B, int k,
                               int* __restrict__ draft) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();
    if (i >= B * k) return;
    int b = i / k, c = i % k;
    if (s.finished[b]) return;
    int p = s.len[b] + c;
    if (p < stride) { int t = script[(size_t)b * stride + p]; if (t >= 0) draft[i] = t; }
}

// Commit as a kernel of its own (specdec_commit; explicit keep / next).
__global__ void k_commit(Session s, const int* __restrict__ draft, const int* __restrict__ keep,
                         const int* __restrict__ next, int B, int k, int eos, unsigned long long* post) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();                                    // no early trigger: the lengths written here are read by later kernels BEFORE their waits
    if (b < B) commit_sequence(s, b, draft, keep[b], next[b], k, eos);
    __syncthreads();
    commit_post(s, post);
}

__global__ void k_session_init(Session s, const int* __restrict__ src_len, const int* __restrict__ max_tgt, int B,
                               int max_tgt_cap, int S_max) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) {
        for (int i = 0; i < 4; ++i) s.stats[i] = 0ull;
    }
    if (b >= B) return;
    int mt = max_tgt ? min(max(max_tgt[b], 0), max_tgt_cap) : max_tgt_cap;
    s.len[b] = 0;
    s.dlen[b] = 0;
    if (b == 0) *s.dticket = 0;
    s.max_tgt[b] = mt;
    s.finished[b] = (mt <= 0) ? 1 : 0;
    s.src_len[b] = min(max(src_len[b], 1), S_max);
}

__global__ void k_count_active(Session s, int B) {      // one warp
    int n = 0;
    for (int b = threadIdx.x; b < B; b += 32) n += s.finished[b] ? 0 : 1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        s.counters[CNT_ACTIVE] = n;
        s.counters[CNT_TICKET] = 0;
    }
}

__global__ void k_copy_out(Session s, int B, int* __restrict__ out, int out_stride, int* __restrict__ out_len,
                           int* __restrict__ fin) {
    int b = blockIdx.x;
    if (b >= B) return;
    int n = s.len[b];
    if (out) for (int t = threadIdx.x; t < min(n, out_stride); t += blockDim.x)
        out[(size_t)b * out_stride + t] = s.out[(size_t)b * s.out_stride + t];
    if (threadIdx.x == 0) { if (out_len) out_len[b] = n; if (fin) fin[b] = s.finished[b]; }
}

// ------------------------------------------------------------------ integrity checks (debugging aid)
// Every arena allocation is followed by a 256-byte red zone holding a fixed pattern; a kernel that writes past the end
// of its buffer damages one.  One warp per zone: report[0] += damaged zones, report[1] = lowest damaged zone index.
constexpr unsigned long long RED_PATTERN = 0xC5A5C5A5C5A5C5A5ull;
__global__ void k_red_fill(unsigned char* base, const unsigned long long* __restrict__ zone_off, int n_zones) {
    const int z = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (z < n_zones) reinterpret_cast<unsigned long long*>(base + zone_off[z])[lane] = RED_PATTERN;
}
__global__ void k_red_check(const unsigned char* base, const unsigned long long* __restrict__ zone_off, int n_zones,
                            unsigned long long* report) {
    const int z = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (z >= n_zones) return;
    const bool bad = reinterpret_cast<const unsigned long long*>(base + zone_off[z])[lane] != RED_PATTERN;
    if (__any_sync(0xffffffffu, bad) && lane == 0) {
        atomicAdd(report, 1ull);
        atomicMin(report + 1, (unsigned long long)z);
    }
}
// Non-finite values (NaN, +-Inf) in activation buffers and caches: blockIdx.y = buffer, blockIdx.x strides over its
// 16-byte pieces.  report[2] += count, report[3] = lowest buffer index holding one.
struct ScanBuf { const void* p; unsigned long long n16; int f32; int pad; };   // n16 = whole 16-byte pieces
__global__ void k_nonfinite_scan(const ScanBuf* __restrict__ bufs, unsigned long long* report) {
    const ScanBuf b = bufs[blockIdx.y];
    const uint4* p = reinterpret_cast<const uint4*>(b.p);
    int cnt = 0;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < b.n16; i += (unsigned long long)gridDim.x * blockDim.x) {
        const uint4 v = p[i];
        const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (b.f32) cnt += ((w[j] & 0x7F800000u) == 0x7F800000u) ? 1 : 0;
            else cnt += (((w[j] & 0x7F80u) == 0x7F80u) ? 1 : 0) + (((w[j] & 0x7F800000u) == 0x7F800000u) ? 1 : 0);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if ((threadIdx.x & 31) == 0 && cnt) {
        atomicAdd(report + 2, (unsigned long long)cnt);
        atomicMin(report + 3, (unsigned long long)blockIdx.y);
    }
}

// ------------------------------------------------------------------ weight repacking
template <typename T>
__global__ void k_convert(const float* __restrict__ in, T* __restrict__ out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t st = (size_t)gridDim.x * blockDim.x;
    for (; i < n; i += st) out[i] = from_f<T>(in[i]);
}

}  // namespace sd
