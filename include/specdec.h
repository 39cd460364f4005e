/*
 * specdec.h -- C ABI of the B200 (sm_100a) SpecDec draft -> verify -> commit library.
 *
 * The library implements the hot path of Speculative Decoding for seq2seq
 * generation: the Spec-Drafter's parallel pass over k [MASK] queries
 * (Section 3.1.3, inference equation), the verification pass in which the
 * autoregressive encoder-decoder Transformer scores all k drafts of every
 * sequence at once (Section 2, Eq. 1-3), the Spec-Verification acceptance rule
 * (Section 3.2, Eq. 7-9) and the loop that repeats draft -> verify -> commit
 * until [EOS] (Section 2, last sentence; Appendix "Case Study").
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller
 *     owns every buffer it passes; the library owns its arena (repacked weights,
 *     paged KV cache, workspaces) from specdec_create to specdec_destroy.
 *   - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on it
 *     unless stated otherwise; buffers must stay valid until the stream reaches
 *     the end of the call.
 *   - Every function returns SPECDEC_OK (0) or a negative error code; a message
 *     is kept in the handle (specdec_last_error).  Nothing throws, exits or prints.
 *   - One decoding session per handle at a time: specdec_encode starts it.
 *   - Token ids are int32.  Row-major everywhere.
 *   - There is no CPU fallback: without a CUDA device every compute call fails
 *     with SPECDEC_ERR_CUDA.
 */
#ifndef SPECDEC_H
#define SPECDEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECDEC_OK                 0
#define SPECDEC_ERR_INVALID_ARG   -1
#define SPECDEC_ERR_SHAPE         -2   /* weight manifest does not match the dims        */
#define SPECDEC_ERR_CAPACITY      -3   /* B / S / k / max_tgt beyond create-time limits  */
#define SPECDEC_ERR_NOT_ENCODED   -4
#define SPECDEC_ERR_CUDA          -5
#define SPECDEC_ERR_TIMEOUT       -6   /* a bounded device-side wait gave up.  specdec_generate reports it itself;
                                          the asynchronous step calls report it one call late: specdec_commit and
                                          specdec_get_output fetch the device's error word, and the next call on the
                                          handle that finds it set returns this code and clears it.  The handle stays
                                          usable: start over with specdec_encode                                      */
#define SPECDEC_ERR_UNSUPPORTED   -7
#define SPECDEC_ERR_CORRUPT       -8   /* an integrity check (option "debug_checks") found a damaged red zone behind an
                                          arena block or a non-finite activation; specdec_last_error names it        */

#define SPECDEC_DTYPE_F32   0
#define SPECDEC_DTYPE_BF16  1

#define SPECDEC_ACT_RELU    0
#define SPECDEC_ACT_GELU    1

typedef struct specdec_handle specdec_handle;

/* One encoder-decoder Transformer (pre-LN, shared embedding table; position tables are weights, so
 * sinusoidal and learned positions are both just data). */
typedef struct {
    int d_model, n_heads, d_ffn, vocab;
    int enc_layers, dec_layers;
    int max_pos;                       /* rows of the position tables */
} specdec_model_dims;

typedef struct {
    specdec_model_dims verifier, drafter;
    int k_max;                         /* largest draft block                                  */
    int max_batch, max_src, max_tgt;   /* capacity limits of a session                         */
    int page_tokens;                   /* tokens per KV-cache page (power of two)              */
    int pad_id, bos_id, eos_id, mask_id;
    int compute_dtype;                 /* SPECDEC_DTYPE_F32: fp32 operands (SIMT kernels);
                                          SPECDEC_DTYPE_BF16: bf16 operands, fp32 accumulation
                                          (tcgen05 tensor-core GEMMs)                          */
    int ffn_activation;                /* SPECDEC_ACT_RELU (Transformer-base, Section 4.1) or SPECDEC_ACT_GELU:
                                          the exact GELU x * Phi(x), for the BART-base-shaped pair of the
                                          summarisation experiment (Section 5.2); both models use it    */
} specdec_config;

/* One named weight.  `d_ptr` is a DEVICE pointer to fp32 data, row-major.
 * Names, per model prefix "verifier." / "drafter." (y = x W^T + b, W is [out,in]):
 *   embed [V,d]   pos_enc, pos_dec [max_pos,d]
 *   enc.{l}.ln1.{g,b}  enc.{l}.self.{q,k,v,o}.{w,b}  enc.{l}.ln2.{g,b}
 *   enc.{l}.ffn.{w1,b1,w2,b2}   enc.ln_f.{g,b}
 *   dec.{l}.ln1  dec.{l}.self.*  dec.{l}.ln_cross.{g,b}  dec.{l}.cross.{q,k,v,o}.{w,b}
 *   dec.{l}.ln2  dec.{l}.ffn.*   dec.ln_f.{g,b}                                        */
typedef struct {
    const char* name;
    const void* d_ptr;
    int         dtype;                 /* SPECDEC_DTYPE_F32 only */
    int         ndim;
    long long   shape[4];
} specdec_tensor;

/* Counters of specdec_generate.  Tok. of the paper's latency model (Eq. 4) is
 * accepted / seq_iterations (or emitted / seq_iterations counting the
 * bifurcation token); t_d, t_v are ms_draft, ms_verify per iteration. */
typedef struct {
    long long iterations;              /* draft->verify->commit rounds that ran               */
    long long seq_iterations;          /* sum over rounds of sequences still decoding         */
    long long drafted, accepted, emitted;
    double    ms_encode, ms_draft, ms_verify, ms_commit, ms_total;   /* draft / verify / commit: option "stats_timing" only */
    int       status;
} specdec_stats;

/* Builds a handle: validates the manifest against the dims, allocates the arena
 * (the only device allocation the library makes), copies and repacks the weights
 * (bf16 for SPECDEC_DTYPE_BF16).  Synchronises `stream` before returning, so the
 * caller may free its weight buffers afterwards.  *out is NULL on failure; the
 * reason is then available from specdec_last_error(NULL). */
int specdec_create(const specdec_config* cfg, const specdec_tensor* weights, int n_weights,
                   void* stream, specdec_handle** out);
int specdec_destroy(specdec_handle* h);

/* Starts a session: runs both encoders over the right-padded sources and caches
 * the per-decoder-layer cross-attention K/V of both models ("the encoder is
 * forwarded only once", Section 3.1.2).  All sequences start with no committed
 * target token.  d_src [B,S_max] int32, d_src_len [B] (1..S_max), d_max_tgt [B]
 * (0..max_tgt; NULL = max_tgt for all). */
int specdec_encode(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len,
                   const int32_t* d_max_tgt, int B, int S_max, void* stream);

/* Spec-Drafter pass (Section 3.1.3): for every unfinished sequence, the decoder
 * runs without a causal mask over [BOS, committed tokens, MASK x k] and the
 * argmax (lowest id on ties) at each mask row becomes a draft.
 * d_draft [B,k] int32 out; rows of finished sequences are left untouched. */
int specdec_draft(specdec_handle* h, int k, int32_t* d_draft, void* stream);

/* Verification pass (Section 2 Eq. 1-3, Section 3.2 Eq. 7-9): the verifier
 * decoder scores the block [last committed token, k drafts] causally over the
 * paged KV cache; draft i is accepted iff all earlier ones are, fewer than
 * `beta` vocabulary entries score strictly higher (Eq. 7) and top-1 score minus
 * its score <= tau (Eq. 8).  d_accepted [B] receives the accepted length in
 * [0,k]; d_bif [B] the verifier's top-1 token on the row after the accepted
 * prefix (the replacement at the bifurcation, or the bonus token when a = k).
 * Does not commit.  beta >= 1, tau >= 0, 0 <= k <= k_max (k = 0: one row, the next greedy token). */
int specdec_verify(specdec_handle* h, const int32_t* d_draft, int k, int beta, float tau,
                   int32_t* d_accepted, int32_t* d_bif, void* stream);

/* Commit / rollback (Eq. 3): appends drafts[0..keep) and `next` to each
 * unfinished sequence, cuts after the first [EOS] and at the sequence's max
 * target length, marks finished sequences, and keeps only the KV-cache rows of
 * the kept prefix.  d_keep / d_next [B] may be NULL: the results of the last
 * specdec_verify are used.  Must follow a specdec_verify (it reuses its block). */
int specdec_commit(specdec_handle* h, const int32_t* d_keep, const int32_t* d_next, void* stream);

/* encode + (draft -> verify -> commit) until every sequence is finished.
 * d_out [B,out_stride] int32 receives the generated ids (without BOS),
 * d_out_len [B] their count.  h_stats may be NULL.  Synchronises `stream`.
 * k = 0 is plain greedy autoregressive decoding with the verifier alone (no drafter pass, one-row
 * verify blocks): the baseline SpecDec is compared with. */
int specdec_generate(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len,
                     const int32_t* d_max_tgt, int B, int S_max, int k, int beta, float tau,
                     int32_t* d_out, int out_stride, int32_t* d_out_len,
                     specdec_stats* h_stats, void* stream);

/* Same, with HOST buffers: the copies host->device (sources) and device->host
 * (ids, lengths) are part of the call.  Pinned host memory avoids a staging copy. */
int specdec_generate_host(specdec_handle* h, const int32_t* h_src, const int32_t* h_src_len,
                          const int32_t* h_max_tgt, int B, int S_max, int k, int beta, float tau,
                          int32_t* h_out, int out_stride, int32_t* h_out_len,
                          specdec_stats* h_stats, void* stream);

/* Current session state: committed ids [B,out_stride], lengths [B], finished flags [B]
 * (any pointer may be NULL). */
int specdec_get_output(specdec_handle* h, int32_t* d_out, int out_stride, int32_t* d_out_len,
                       int32_t* d_finished, void* stream);

/* The acceptance rule alone (Eq. 7-9) on caller-provided fp32 logits
 * d_logits [B,k+1,V]: same outputs as specdec_verify.  No handle, no workspace. */
int specdec_accept_scan(const float* d_logits, const int32_t* d_draft, int B, int k, int V,
                        int beta, float tau, int32_t* d_accepted, int32_t* d_bif, void* stream);

/* The same acceptance rule for callers that must not allocate device memory -- the paper has no
 * counterpart; this exists for embedding the rule in programs where the device allocator is off
 * limits: a serving process whose memory pool already owns all of HBM (so a later cudaMalloc
 * fails), or a latency-critical loop that cannot afford the device-wide synchronisation an
 * allocation or free implies.  Inputs and outputs are the caller's, exactly as for
 * specdec_accept_scan (d_logits [B,k+1,V] fp32, d_draft [B,k]; d_accepted, d_bif [B]); the
 * intermediate per-row partial statistics live in a fixed array compiled into the library
 * (about 4.2 MB of device memory on every GPU that loads the library, held until the process
 * exits).  Limits: B*(k+1) <= 4096, V <= 65536 and k+1 <= 2048; beyond them the call returns
 * SPECDEC_ERR_CAPACITY and launches nothing.  The call makes no cudaMalloc / cudaFree and uses
 * no allocating library routine.  The first call on each device looks up the array's device
 * address (cudaGetSymbolAddress, with the caller's current device); make that first call
 * before starting any stream capture.  All calls share the one array, which keeps whatever
 * the previous call left in it; every entry a call reads is rewritten by that call first, so
 * nothing needs clearing, but two calls whose kernels overlap on the GPU (different streams,
 * or different host threads) race on it: serialise them. */
int specdec_accept_scan_static(const float* d_logits, const int32_t* d_draft, int B, int k, int V,
                               int beta, float tau, int32_t* d_accepted, int32_t* d_bif, void* stream);

/* Debug / parity helpers (not on the hot path).
 * specdec_debug_logits: re-runs the vocabulary projection of the last verify
 *   (which = 0, rows [B*(k+1)]) or draft (which = 1, rows [n_active*k]) pass
 *   unfused and stores fp32 logits [rows,V].
 * specdec_debug_row_stats: per verify row of the last specdec_verify, 6 floats:
 *   max logit, argmax id, log-sum-exp, count of entries above the draft's logit,
 *   the draft's logit (+inf on the bonus row), draft id (-1 on the bonus row). */
int specdec_debug_logits(specdec_handle* h, int which, float* d_logits, void* stream);
int specdec_debug_row_stats(specdec_handle* h, float* d_stats, void* stream);
/* With option "trace" != 0 the first CTA of some kernels records nanosecond time stamps of its phases into a
 * 256-entry device array; this copies the first n (<= 256) entries to the host.  Synchronises the device. */
int specdec_debug_trace(specdec_handle* h, long long* h_out, int n);

/* Integrity check (debugging aid; the paper has no counterpart).  The handle's device arena places a 256-byte red
 * zone with a fixed pattern behind every block it hands out (weights, activations, caches, row metadata, session
 * state), so a kernel that writes past the end of its buffer damages one.  This call checks every red zone and scans
 * the activation buffers, the encoder memories and the K/V caches for NaN / Inf, on `stream`, and synchronises it.
 * It returns SPECDEC_OK whenever the check itself ran; the findings are in *out (first_* are -1 when the count is 0;
 * buffers are numbered in the order: residual rows, mask rows, normalised rows, QKV rows, attention output, cross
 * query rows, feed-forward rows, encoder memory, the second encoder's six buffers, K caches, V caches, the drafter's
 * caches, cross K/V of the verifier and of the drafter).  With option "debug_checks" = 1 every encode / draft / verify /
 * commit / generate call runs it before returning and fails with SPECDEC_ERR_CORRUPT on a finding. */
typedef struct specdec_integrity {
    int32_t zones;                   /* red zones checked                                  */
    int32_t damaged_zones;
    int32_t first_damaged_zone;      /* index (allocation order) of the first damaged one  */
    int32_t first_nonfinite_buffer;
    int64_t nonfinite;               /* NaN / Inf values found                             */
} specdec_integrity;
int specdec_debug_integrity(specdec_handle* h, specdec_integrity* out, void* stream);

/* Diagnostics: the cost of one kernel boundary inside a step.  Replays (from a CUDA graph, on the handle's own stream)
 * a chain of n_links launches of `grid` CTAs, each of which waits for its predecessor (programmatic dependent
 * launch, as between the kernels of a step), reads the word it wrote and writes it back; returns the best of ten
 * replays divided by n_links, in microseconds.  Synchronises. */
int specdec_debug_link_cost(specdec_handle* h, int n_links, int grid, double* h_us_per_link);

/* Diagnostics: nanoseconds per exchange round between the CTAs of one thread-block cluster (8 or 16 CTAs of 256
 * threads) through distributed shared memory: every CTA stores bytes_per_peer (0 .. 8192, a multiple of 16) bytes into each
 * peer's shared memory, arrives on every peer's barrier and waits for all arrivals; `rounds` rounds back to back.
 * What a fused cluster kernel pays where separate kernels pay a kernel boundary.  Synchronises. */
int specdec_debug_cluster_round(specdec_handle* h, int cluster_size, int bytes_per_peer, int rounds, double* h_ns_per_round);

/* Diagnostics: clocks per tcgen05.mma (M = 128 x N = bn x K = 16, bf16) when the operands already sit in shared memory:
 * one CTA per SM issues n_mma of them back to back with no loads in the loop.  two_sm = 1: the cta_group::2 form
 * (M = 256 over two SMs).  *h_issue_clocks = clocks until the issuing thread is done, *h_done_clocks = until the last
 * MMA has completed, both per MMA.  Tells a main loop that waits for operands from one the tensor pipe limits.
 * bf16 handles only.  Synchronises. */
int specdec_debug_mma_rate(specdec_handle* h, int bn, int two_sm, int n_mma, double* h_issue_clocks, double* h_done_clocks);
/* The same with what a real main loop adds.  bg_stages (0..6): while the MMAs are issued, another thread of every CTA
 * keeps that many bulk copies of 16 KB in flight from global memory (the verifier's embedding table, at least 8 MB) into
 * a separate region of the CTA's shared memory, as a TMA producer would; *h_bg_bytes_per_clock = bytes it landed per SM
 * clock and CTA.  commit_every (0 = never, else): a tcgen05.commit after every k-block of four MMAs to a barrier nobody
 * waits on (the multicast form for two-SM tiles), as a main loop issues one.  Tells whether the producer's writes or
 * the commits slow the tensor pipe down.  Synchronises. */
int specdec_debug_mma_rate_bg(specdec_handle* h, int bn, int two_sm, int n_mma, int bg_stages, int commit_every,
                              double* h_issue_clocks, double* h_done_clocks, double* h_bg_bytes_per_clock);

/* Scripted drafts, a benchmark / test hook with no counterpart in the paper: random-init
 * models almost never agree, so a workload's acceptance pattern is imposed instead.  After the
 * drafter pass has run, draft i of a sequence with j committed tokens is replaced by
 * d_script[b*stride + j + i] wherever that entry is >= 0.  d_script = NULL turns it off. */
int specdec_set_draft_script(specdec_handle* h, const int32_t* d_script, int B, int stride, void* stream);

/* With option "profile" = 1, every vocabulary-projection launch of the verify step (B*(k+1) rows)
 * inside specdec_generate is bracketed by CUDA events; this returns their summed duration and
 * count since the option was set. */
int specdec_profile_read(specdec_handle* h, double* h_ms, long long* h_launches);

/* Options (experiments and on-device cross-checks; every combination computes the same result):
 * "drafter_prefix_causal" 0 (default) / 1: the second reading of the Spec-Drafter's decoder mask.  0: no self-attention
 *                mask at all (every row of [BOS, committed, MASK x k] sees every row: "mask-predict manner", Section 3.1);
 *                the whole input is recomputed every iteration.  1: the committed tokens attend causally among
 *                themselves and only the [MASK] rows see everything; the drafter's decoder then keeps a K/V cache of the
 *                committed positions and a draft pass computes only the newly committed tokens and the k [MASK] rows
 *                (Section 3.1.2: the decoder runs every iteration, so its cost should not grow with the prefix).  A
 *                different function of the same weights: drafts differ, the verified output under beta = 1, tau = 0
 *                does not.  Takes effect at the next specdec_encode.
 * "gemm"         0 SIMT reference GEMM / 1 tcgen05 tensor-core GEMM (bf16 handles; default 1)
 * "attn"         0 warp-per-row reference attention / 1 tensor-core tile attention (bf16, 64-wide heads; default 1)
 * "skinny"       0/1 weight-streaming GEMM with fused LayerNorm for passes of at most 32 rows (default 1)
 * "sk_cluster"   0 off / 1 (default): those GEMMs run in clusters of 8 CTAs that share the normalised input rows
 *                through distributed shared memory; 2 / 3 also the GEMMs without a LayerNorm (K <= 512 / all)
 * "pair"         0/1 two-SM tensor-core tiles (cta_group::2) for GEMMs with >= 1024 rows and columns (default 0)
 * "enc_skinny"   0 / 1 (default) / 2: the weight-streaming GEMM also serves neither / the drafter's / both encoders when a
 *                source has at most 32 positions
 * "ln_fuse"      0/1 the LayerNorm that reads the residual stream next runs inside the residual GEMM (default 0)
 * "splitk"       0/1 residual GEMMs with K >= 1024 over few row tiles split K across a cluster (default 1)
 * "attn_rs"      0 never / 1 by rule (default) / 2 whenever the keys allow: scores stay in the MMA accumulators
 * "attn_stream"  0 never / 1 by rule (default) / 2 always / 3 always, two-stage ring: attention walks the keys in
 *                blocks of 64 with a running maximum; "attn_stream_keys" (default 320) is the rule's threshold
 * "attn_warps"   0 choose per launch (default), 4 or 8 warps per tile-attention CTA
 * "tc_bn"        0 choose (default), else the column width of the tensor-core tiles (64 / 128 / 256)
 * "pdl"          0/1 programmatic dependent launch between the kernels of a step (default 1)
 * "graphs"       0/1 replay steps from CUDA graphs (default 1)
 * "gate"         0 never / 1 above batch 4 (default) / 2 always: each iteration of specdec_generate is one graph
 *                behind a device-side IF node, so the host can queue iterations ahead of the counter it reads
 * "poll_flag"    0/1 specdec_generate learns of each commit from a word in pinned host memory (default 1)
 * "poll_lag"     n: specdec_generate reads the unfinished-sequences counter n iterations late (default: by batch)
 * "stats_timing" 0/1 fill ms_draft / ms_verify / ms_commit of specdec_stats (default 0; turns the gate off)
 * "profile"      0/1 see specdec_profile_read
 * "row_lse"      0/1 also accumulate the log-sum-exp of every verifier row (reported by specdec_debug_row_stats)
 * "diag_repeat"  bit mask: launch every attention (1), LayerNorm (2), non-residual GEMM (4), vocabulary kernel (8)
 *                twice in a row (same result), so the step time rises by that class's cost inside the pipeline
 * "trace"        see specdec_debug_trace
 * "debug_checks" 0/1 see specdec_debug_integrity (default 0: the check synchronises)
 * "poke_zone" i / "heal_zones" / "poke_nan" 0|1: test hooks for that check -- damage red zone i from the host, restore
 *                every red zone, put a NaN (or a zero) into the last element of the attention-output buffer
 * "inject_error" code: test hook -- the next specdec_verify / specdec_generate finds this code in the device error
 *                word, as if a bounded device-side wait had given up (no kernel waits, nothing faults) */
int specdec_set_option(specdec_handle* h, const char* name, int value);

/* Number of kernels the library has launched on this handle since create. */
long long specdec_launch_count(const specdec_handle* h);

const char* specdec_last_error(const specdec_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* SPECDEC_H */
