// Host runtime and C ABI of the SpecDec draft -> verify -> commit library (see include/specdec.h).
// The arena is the only device allocation; every step of the path runs in the kernels of
// kernels.cuh and gemm_tc.cuh.  There is no CPU fallback.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <chrono>
#include <map>
#include <string>
#include <type_traits>
#include <unordered_map>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/specdec.h"
#include "attention_stream.cuh"
#include "attention_tc.cuh"
#include "cluster_round.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc_pair.cuh"
#include "gemm_tc_splitk.cuh"
#include "kernels.cuh"
#include "mma_rate.cuh"
#include "skinny_gemm.cuh"

using namespace sd;

namespace {

thread_local std::string g_create_error;

struct LayerW {
    void *qkv_w, *o_w, *cq_w, *ckv_w, *co_w, *w1, *w2;
    float *qkv_b, *o_b, *cq_b, *ckv_b, *co_b, *b1, *b2;
    float *ln1_g, *ln1_b, *lnc_g, *lnc_b, *ln2_g, *ln2_b;
};
struct ModelW {
    specdec_model_dims dm;
    void* embed;
    float *pos_enc, *pos_dec;
    std::vector<LayerW> enc, dec;
    float *enc_lnf_g, *enc_lnf_b, *dec_lnf_g, *dec_lnf_b;
    // cross-attention K | V of the session for every decoder layer: one buffer [B*S_max, dec_layers * 2d] written by a
    // single projection of the encoder memory (the layers' K/V matrices are stored back to back); ckv[l] = its
    // column block l, ckv_stride = elements per row
    std::vector<void*> ckv;
    int ckv_stride = 0;
};

// Bump allocator over one device allocation.  Every block is followed by a 256-byte red zone (see k_red_check).
struct Arena {
    char* base = nullptr;
    size_t off = 0;
    std::vector<unsigned long long> zones;         // byte offsets of the red zones, in allocation order
    void* take(size_t n) {
        off = (off + 255) & ~size_t(255);
        void* p = base ? base + off : nullptr;
        off = (off + n + 255) & ~size_t(255);
        zones.push_back(off);
        off += 256;
        return p;
    }
};

}  // namespace

struct specdec_handle {
    specdec_config cfg;
    int dtype;
    size_t esz;                    // bytes per operand element
    ModelW ver, dra;
    Arena arena;
    // capacities
    int B_cap, S_cap, T_cap, k_cap, R_cap, R2_cap, M_cap, d_max, f_max, v_max, pages_per_seq, n_tiles_cap;
    // activations
    float *x, *x2;                          // the workspace in use (one of ws[0], ws[1])
    void *y, *qkv, *att, *q, *hbuf, *mem;
    struct WorkSet { float* x; void *y, *qkv, *att, *q, *hbuf, *mem; } ws[2];   // ws[1]: second encoder, own stream
    cudaStream_t enc_stream = nullptr;
    cudaEvent_t enc_fork = nullptr, enc_join = nullptr;
    // verifier KV cache
    std::vector<void*> kc, vc;
    // drafter KV cache of its decoder layers (prefix-causal reading only; same page geometry as the verifier's)
    std::vector<void*> dkc, dvc;
    int drafter_pc = 0;             // option "drafter_prefix_causal", as set
    int drafter_pc_session = 0;     // ... as in force for the running session (latched by specdec_encode)
    bool fuse_commit = false;       // the generation loop: the acceptance scan commits its own decision (no commit kernel)
    bool commit_done = false;       // ... and did so in the verify pass just issued
    int dnew_ub = 1;                // upper bound on the prefix positions the next draft pass has to add to that cache
    int* page_table;
    // rows
    Rows rows, mrows;
    // vocabulary statistics
    RowPart* part;
    float *ld, *row_stats;
    int* ld_id;
    int *accepted, *bif, *v_draft, *g_draft;
    int *stage_src, *stage_len, *stage_mt;   // device staging of specdec_generate_host
    Session ses;
    // session (host side)
    int B = 0, S_max = 0, last_k = 0, len_ub = 0;
    bool encoded = false, verified = false, drafted = false;
    int last_draft_rows_ub = 0;
    // options
    int use_tc = 1, use_graphs = 1, use_tc_attn = 1, want_lse = 0, use_skinny = 1, use_pdl = 1;
    long long* trace_buf = nullptr; // device [256] in-kernel time stamps (option "trace")
    int want_trace = 0;
    size_t skinny_smem_cap = 0;
    int poll_lag = -1;              // -1: chosen by batch size
    int stats_timing = 0;           // 1: specdec_generate records an event after every phase (option "stats_timing")
    int use_gate = 1;               // whole iterations as one graph behind a device-side IF node (option "gate")
    bool gate_ok = true;            // false once building such a graph failed: the plain graphs are used from then on
    // LayerNorm fused into the residual GEMM that feeds it (tensor-core path): what the next residual GEMM should
    // also produce, and what the last one did produce
    struct NextLn { const float* g; const float* b; void* out; };
    NextLn next_ln = {nullptr, nullptr, nullptr};
    const float* fused_x = nullptr; const float* fused_g = nullptr; const void* fused_out = nullptr;
    // integrity checks (option "debug_checks", specdec_debug_integrity)
    unsigned long long* integ_report = nullptr; ScanBuf* integ_bufs = nullptr; unsigned long long* zone_tab = nullptr;
    int zone_cap = 0, n_zones = 0, n_scan = 0;
    std::vector<std::string> scan_names;
    int debug_checks = 0;
    int enc_skinny = 1;             // option "enc_skinny": 1 = the drafter's encoder (the longer of the two side-by-side chains) uses the weight-streaming GEMM for sources of at most 32 positions (default: 360 -> 340 us for a 29-token source), 2 = both encoders (no better: they get in each other's way), 0 = neither
    bool enc_skinny_now = false;
    int use_ln_fuse = 0;            // option "ln_fuse": measured slower than the separate LayerNorm launch, kept for comparison
    int use_sk_cluster = 1;         // option "sk_cluster": 1 = LayerNorm-fused weight-streaming GEMMs share the normalised rows in clusters of 8; 2 = the plain ones too (measured slower)
    bool splitk_ready = false;
    int diag_repeat = 0;            // diagnostics: launch every attention (1) / LayerNorm (2) / non-residual GEMM (4) / vocabulary (8) kernel twice (same result) to
                                    // read its cost inside the pipeline off the step time (option "diag_repeat")
    int use_splitk = 1;             // residual GEMMs with K >= 1024 over few row tiles split K across a cluster of 4 / 6 CTAs (option "splitk")
    bool pair_ready = false;
    int use_pair = 0;               // two-SM tiles (cta_group::2) for wide GEMMs over many rows (option "pair")
    int attn_rs = 1;                // tile attention keeps the scores in registers when the keys allow (option "attn_rs")
    int attn_stream = 1;            // streaming tile attention: 0 never, 1 by rule, 2 always, 3 always with the 2-stage ring (option "attn_stream")
    int attn_stream_keys = 320;     // option "attn_stream_keys"
    int attn_warps = 0;             // 0 = choose per launch, else 4 or 8 warps per tile-attention CTA (option "attn_warps")
    int skinny_groups = 1;          // 8-row weight groups per CTA of the weight-streaming GEMM (1, 2 or 4)
    // CUDA graphs of whole draft / verify(+commit) steps, keyed by everything their launches depend on
    struct GraphEntry { cudaGraphExec_t exec; long long kernels; };
    std::map<std::vector<long long>, GraphEntry> graphs;
    size_t attn_tc_smem_cap = 0;
    long long launches = 0;
    // polling
    int* h_poll = nullptr;          // pinned
    unsigned long long* h_post = nullptr;   // pinned, written by k_commit: (commits of this handle so far) << 32 | unfinished sequences
    unsigned commits_issued = 0;    // commit kernels launched so far: what the posted count reaches once the stream drains
    int poll_flag = 1;              // the generation loop polls h_post instead of copying the counter back (option "poll_flag")
    unsigned long long* h_stats = nullptr;  // pinned [4]
    std::vector<cudaEvent_t> poll_ev;
    // device error word (counters[7], raised by bounded device-side waits) mirrored into pinned memory: h_poll[ERRW_SLOT]
    cudaEvent_t errw_ev = nullptr;
    bool errw_pending = false;      // a copy of the word is in flight
    std::vector<cudaEvent_t> time_ev;
    sd::TmaEncoder tma;
    // work submitted on the legacy default stream (which cannot be captured into a graph) is run on this
    // stream instead, fenced by events at both ends of the call
    cudaStream_t own_stream = nullptr;
    cudaEvent_t fence_in = nullptr, fence_out = nullptr;
    // scripted drafts (benchmark / test hook) and dominant-kernel timing
    int* script = nullptr;          // device [B_cap, T_cap + k_cap] or unset
    bool script_on = false;
    int profile = 0;
    std::vector<cudaEvent_t> prof_ev;
    size_t prof_n = 0;
    double prof_ms = 0.0;
    long long prof_launches = 0;
    std::string err;
};

namespace {

constexpr int ERRW_SLOT = 32;       // index into h_poll of the error word's host mirror

int fail(specdec_handle* h, int code, const std::string& msg) {
    if (h) h->err = msg; else g_create_error = msg;
    return code;
}
#define CUDA_TRY(h, expr)                                                                   \
    do {                                                                                    \
        cudaError_t e__ = (expr);                                                           \
        if (e__ != cudaSuccess)                                                             \
            return fail(h, SPECDEC_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
    } while (0)
#define KCHECK(h)                                                                           \
    do {                                                                                    \
        cudaError_t e__ = cudaGetLastError();                                               \
        if (e__ != cudaSuccess)                                                             \
            return fail(h, SPECDEC_ERR_CUDA, std::string("kernel launch: ") + cudaGetErrorString(e__) + \
                        " at line " + std::to_string(__LINE__));                            \
        ++h->launches;                                                                      \
    } while (0)

#define TRY(expr) do { int rc__ = (expr); if (rc__ != 0) return rc__; } while (0)

inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// Bounded device-side waits raise a code in counters[7].  The step calls (draft / verify / commit / get_output) are
// asynchronous, so they report it one call late: commit and get_output queue a 4-byte copy of the word into pinned
// memory, and every step call first looks at the last copy that has landed.  Reporting clears the word.
int errw_check(specdec_handle* h, cudaStream_t st, const char* who) {
    if (h->errw_pending) {
        if (cudaEventQuery(h->errw_ev) != cudaSuccess) { cudaGetLastError(); return 0; }
        h->errw_pending = false;
    }
    const int code = ((volatile int*)h->h_poll)[ERRW_SLOT];
    if (code == 0) return 0;
    h->h_poll[ERRW_SLOT] = 0;
    cudaMemsetAsync(h->ses.counters + 7, 0, 4, st);
    return fail(h, SPECDEC_ERR_TIMEOUT, std::string(who) + ": a bounded device-side wait gave up (code " + std::to_string(code) + ")");
}
void errw_fetch(specdec_handle* h, cudaStream_t st) {
    if (h->errw_pending) return;
    if (cudaMemcpyAsync(h->h_poll + ERRW_SLOT, h->ses.counters + 7, 4, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
        cudaEventRecord(h->errw_ev, st) == cudaSuccess) h->errw_pending = true;
}

// ---------------------------------------------------------------- layout of the arena
void layout_model(specdec_handle* h, ModelW& m, const specdec_model_dims& dm) {
    Arena& A = h->arena;
    const size_t e = h->esz;
    const size_t d = dm.d_model, f = dm.d_ffn;
    m.dm = dm;
    m.embed = A.take((size_t)dm.vocab * d * e);
    m.pos_enc = (float*)A.take((size_t)dm.max_pos * d * 4);
    m.pos_dec = (float*)A.take((size_t)dm.max_pos * d * 4);
    auto vec = [&](size_t n) { return (float*)A.take(n * 4); };
    auto layer = [&](LayerW& w, bool dec) {
        w.qkv_w = A.take(3 * d * d * e); w.qkv_b = vec(3 * d);
        w.o_w = A.take(d * d * e); w.o_b = vec(d);
        w.w1 = A.take(f * d * e); w.b1 = vec(f);
        w.w2 = A.take(d * f * e); w.b2 = vec(d);
        w.ln1_g = vec(d); w.ln1_b = vec(d); w.ln2_g = vec(d); w.ln2_b = vec(d);
        if (dec) {
            w.cq_w = A.take(d * d * e); w.cq_b = vec(d);
            w.co_w = A.take(d * d * e); w.co_b = vec(d);
            w.lnc_g = vec(d); w.lnc_b = vec(d);
        }
    };
    m.enc.resize(dm.enc_layers);
    m.dec.resize(dm.dec_layers);
    for (auto& w : m.enc) layer(w, false);
    for (auto& w : m.dec) layer(w, true);
    {   // the decoder layers' cross K/V projections, contiguous: [dec_layers * 2d, d] and [dec_layers * 2d]
        char* wall = (char*)A.take((size_t)dm.dec_layers * 2 * d * d * e);
        float* ball = vec((size_t)dm.dec_layers * 2 * d);
        for (int l = 0; l < dm.dec_layers; ++l) {
            m.dec[l].ckv_w = wall ? wall + (size_t)l * 2 * d * d * e : nullptr;
            m.dec[l].ckv_b = ball ? ball + (size_t)l * 2 * d : nullptr;
        }
    }
    m.enc_lnf_g = vec(d); m.enc_lnf_b = vec(d); m.dec_lnf_g = vec(d); m.dec_lnf_b = vec(d);
    m.ckv.resize(dm.dec_layers);
    m.ckv_stride = dm.dec_layers * 2 * (int)d;
    {
        char* all = (char*)A.take((size_t)h->B_cap * h->S_cap * m.ckv_stride * e);
        for (int l = 0; l < dm.dec_layers; ++l) m.ckv[l] = all ? all + (size_t)l * 2 * d * e : nullptr;
    }
}

void layout_rows(Arena& A, Rows& r, int n, int B) {
    auto iv = [&](size_t c) { return (int*)A.take(c * 4); };
    r.tok = iv(n); r.pos = iv(n); r.seq = iv(n); r.nk_self = iv(n); r.nk_cross = iv(n);
    r.src_row = iv(n); r.slot = iv(n);
    r.kv_off = iv(B); r.kv_off_cross = iv(B); r.q_off = iv(B); r.q_cnt = iv(B);
}

void layout_all(specdec_handle* h) {
    Arena& A = h->arena;
    A.off = 0;
    A.zones.clear();
    const size_t e = h->esz;
    layout_model(h, h->ver, h->cfg.verifier);
    layout_model(h, h->dra, h->cfg.drafter);
    const size_t R = h->R_cap, d = h->d_max, f = h->f_max;
    h->x = (float*)A.take(R * d * 4);
    h->x2 = (float*)A.take((size_t)h->R2_cap * d * 4);
    h->y = A.take(R * d * e);
    h->qkv = A.take(R * 3 * d * e);
    h->att = A.take(R * d * e);
    h->q = A.take(R * d * e);
    h->hbuf = A.take(R * f * e);
    h->mem = A.take((size_t)h->B_cap * h->S_cap * d * e);
    h->ws[0] = {h->x, h->y, h->qkv, h->att, h->q, h->hbuf, h->mem};
    {   // a second, encoder-sized workspace so the two encoders can run side by side
        const size_t Re = (size_t)h->B_cap * h->S_cap;
        specdec_handle::WorkSet& w = h->ws[1];
        w.x = (float*)A.take(Re * d * 4); w.y = A.take(Re * d * e); w.qkv = A.take(Re * 3 * d * e); w.att = A.take(Re * d * e);
        w.q = A.take(Re * d * e); w.hbuf = A.take(Re * f * e); w.mem = A.take(Re * d * e);
    }
    const size_t cache_rows = (size_t)h->B_cap * h->pages_per_seq * h->cfg.page_tokens;
    h->kc.resize(h->cfg.verifier.dec_layers);
    h->vc.resize(h->cfg.verifier.dec_layers);
    for (auto& p : h->kc) p = A.take(cache_rows * h->cfg.verifier.d_model * e);
    for (auto& p : h->vc) p = A.take(cache_rows * h->cfg.verifier.d_model * e);
    h->dkc.resize(h->cfg.drafter.dec_layers);
    h->dvc.resize(h->cfg.drafter.dec_layers);
    for (auto& p : h->dkc) p = A.take(cache_rows * h->cfg.drafter.d_model * e);
    for (auto& p : h->dvc) p = A.take(cache_rows * h->cfg.drafter.d_model * e);
    h->page_table = (int*)A.take((size_t)h->B_cap * h->pages_per_seq * 4);
    layout_rows(A, h->rows, h->R_cap, h->B_cap);
    layout_rows(A, h->mrows, h->R2_cap > 0 ? h->R2_cap : 1, h->B_cap);
    const size_t stat_rows = (size_t)(h->M_cap > h->R2_cap ? h->M_cap : h->R2_cap);
    h->part = (RowPart*)A.take(stat_rows * h->n_tiles_cap * sizeof(RowPart));
    h->ld = (float*)A.take((size_t)h->M_cap * 4);
    h->ld_id = (int*)A.take((size_t)h->M_cap * 4);
    h->row_stats = (float*)A.take((size_t)h->M_cap * 6 * 4);
    h->accepted = (int*)A.take((size_t)h->B_cap * 4);
    h->bif = (int*)A.take((size_t)h->B_cap * 4);
    h->v_draft = (int*)A.take((size_t)h->B_cap * h->k_cap * 4);
    h->g_draft = (int*)A.take((size_t)h->B_cap * h->k_cap * 4);
    h->stage_src = (int*)A.take((size_t)h->B_cap * h->S_cap * 4);
    h->stage_len = (int*)A.take((size_t)h->B_cap * 4);
    h->stage_mt = (int*)A.take((size_t)h->B_cap * 4);
    h->script = (int*)A.take((size_t)h->B_cap * (h->T_cap + h->k_cap) * 4);
    h->trace_buf = (long long*)A.take(256 * 8);
    Session& s = h->ses;
    s.len = (int*)A.take((size_t)h->B_cap * 4);
    s.finished = (int*)A.take((size_t)h->B_cap * 4);
    s.max_tgt = (int*)A.take((size_t)h->B_cap * 4);
    s.src_len = (int*)A.take((size_t)h->B_cap * 4);
    s.out_stride = h->T_cap > 0 ? h->T_cap : 1;
    s.out = (int*)A.take((size_t)h->B_cap * s.out_stride * 4);
    s.dlen = (int*)A.take((size_t)h->B_cap * 4);
    s.dticket = (int*)A.take(4);
    s.counters = (int*)A.take(8 * 4);
    s.stats = (unsigned long long*)A.take(4 * 8);
    // integrity checks: report words, the table of scanned buffers, the table of red-zone offsets (sized by the dry run)
    h->integ_report = (unsigned long long*)A.take(4 * 8);
    h->integ_bufs = (ScanBuf*)A.take(128 * sizeof(ScanBuf));
    h->zone_tab = (unsigned long long*)A.take((size_t)h->zone_cap * 8);
}

// ---------------------------------------------------------------- weight loading
struct Manifest {
    std::unordered_map<std::string, const specdec_tensor*> map;
    std::string missing, bad;
    const float* get(const std::string& name, std::initializer_list<long long> shape) {
        auto it = map.find(name);
        if (it == map.end()) { if (missing.empty()) missing = name; return nullptr; }
        const specdec_tensor* t = it->second;
        bool ok = t->dtype == SPECDEC_DTYPE_F32 && t->ndim == (int)shape.size() && t->d_ptr != nullptr;
        int i = 0;
        for (long long s : shape) { if (ok && t->shape[i] != s) ok = false; ++i; }
        if (!ok) { if (bad.empty()) bad = name; return nullptr; }
        return (const float*)t->d_ptr;
    }
};

template <typename T>
void conv(specdec_handle* h, const float* src, void* dst, size_t n, cudaStream_t st) {
    if (!src) return;
    int blocks = (int)std::min<size_t>((n + 255) / 256, 4096);
    k_convert<T><<<blocks, 256, 0, st>>>(src, (T*)dst, n);
    ++h->launches;
}

template <typename T>
void load_model(specdec_handle* h, ModelW& m, const std::string& pre, Manifest& mf, cudaStream_t st) {
    const long long d = m.dm.d_model, f = m.dm.d_ffn, V = m.dm.vocab, P = m.dm.max_pos;
    const size_t e = h->esz;
    auto mat = [&](const std::string& n, long long r, long long c, void* dst) {
        conv<T>(h, mf.get(pre + n, {r, c}), dst, (size_t)r * c, st);
    };
    auto vec = [&](const std::string& n, long long c, float* dst) { conv<float>(h, mf.get(pre + n, {c}), dst, (size_t)c, st); };
    mat("embed", V, d, m.embed);
    conv<float>(h, mf.get(pre + "pos_enc", {P, d}), m.pos_enc, (size_t)P * d, st);
    conv<float>(h, mf.get(pre + "pos_dec", {P, d}), m.pos_dec, (size_t)P * d, st);
    auto attn_qkv = [&](const std::string& p, void* w, float* b) {
        const char* nm[3] = {"q", "k", "v"};
        for (int i = 0; i < 3; ++i) {
            mat(p + "." + nm[i] + ".w", d, d, (char*)w + (size_t)i * d * d * e);
            vec(p + "." + nm[i] + ".b", d, b + (size_t)i * d);
        }
    };
    auto layer = [&](LayerW& w, const std::string& p, bool dec) {
        vec(p + ".ln1.g", d, w.ln1_g); vec(p + ".ln1.b", d, w.ln1_b);
        attn_qkv(p + ".self", w.qkv_w, w.qkv_b);
        mat(p + ".self.o.w", d, d, w.o_w); vec(p + ".self.o.b", d, w.o_b);
        vec(p + ".ln2.g", d, w.ln2_g); vec(p + ".ln2.b", d, w.ln2_b);
        mat(p + ".ffn.w1", f, d, w.w1); vec(p + ".ffn.b1", f, w.b1);
        mat(p + ".ffn.w2", d, f, w.w2); vec(p + ".ffn.b2", d, w.b2);
        if (dec) {
            vec(p + ".ln_cross.g", d, w.lnc_g); vec(p + ".ln_cross.b", d, w.lnc_b);
            mat(p + ".cross.q.w", d, d, w.cq_w); vec(p + ".cross.q.b", d, w.cq_b);
            mat(p + ".cross.k.w", d, d, w.ckv_w); vec(p + ".cross.k.b", d, w.ckv_b);
            mat(p + ".cross.v.w", d, d, (char*)w.ckv_w + (size_t)d * d * e); vec(p + ".cross.v.b", d, w.ckv_b + d);
            mat(p + ".cross.o.w", d, d, w.co_w); vec(p + ".cross.o.b", d, w.co_b);
        }
    };
    for (int l = 0; l < m.dm.enc_layers; ++l) layer(m.enc[l], "enc." + std::to_string(l), false);
    for (int l = 0; l < m.dm.dec_layers; ++l) layer(m.dec[l], "dec." + std::to_string(l), true);
    vec("enc.ln_f.g", d, m.enc_lnf_g); vec("enc.ln_f.b", d, m.enc_lnf_b);
    vec("dec.ln_f.g", d, m.dec_lnf_g); vec("dec.ln_f.b", d, m.dec_lnf_b);
}

// ---------------------------------------------------------------- launch helpers
// Launch that lets the kernel start before its predecessor in the stream has finished (the kernel itself
// calls pdl_wait() before it touches anything the predecessor wrote).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(specdec_handle* h, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = h->use_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename T>
int ln(specdec_handle* h, const float* x, const float* g, const float* b, int cnt, int rows_ub, void* y, int d,
       cudaStream_t st) {
    if (rows_ub <= 0) return 0;
    {
        cudaError_t e = launch_pdl(h, k_layernorm<T>, dim3(cdiv(rows_ub, 8)), dim3(256), 0, st, x, g, b,
                                   (const int*)(h->ses.counters + cnt), (T*)y, d, 1e-5f,
                                   (cnt == CNT_VERIFY || cnt == CNT_ENC) ? rows_ub : -1);
        if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("layer norm launch: ") + cudaGetErrorString(e));
    }
    KCHECK(h);
    return 0;
}

// LayerNorm of rows x into y, unless the residual GEMM that produced x already wrote exactly that.
template <typename T>
int ln_or_fused(specdec_handle* h, const float* x, const float* g, const float* b, int cnt, int rows_ub, void* y, int d,
                cudaStream_t st) {
    if (x == h->fused_x && g == h->fused_g && y == h->fused_out) return 0;
    TRY(ln<T>(h, x, g, b, cnt, rows_ub, y, d, st));
    if (h->diag_repeat & 2) TRY(ln<T>(h, x, g, b, cnt, rows_ub, y, d, st));
    return 0;
}

// Where the K and V columns of a fused QKV projection go (the verifier's paged cache).
struct KvDest { const int* seq; const int* pos; void* kc; void* vc; int d; };

template <typename T> bool tc_usable(const specdec_handle* h, int N, int K) {
    return std::is_same<T, bf16>::value && h->use_tc && sd::tc_supported(N, K);
}

// LayerNorm fused in front of a GEMM: x fp32 rows, gain, bias.
struct LnSpec { const float* x; const float* g; const float* b; };

// The weight-streaming kernel serves bf16 GEMMs over at most 32 rows (see skinny_gemm.cuh; 64-row variants of its
// row-sharing LayerNorm kernels were tried too: 422 vs 356 us per 2-sequence verify step, and 360 vs 315 us after the
// kernel's bank conflicts were gone): measured on a
// verify step, 26 rows take 362 us with it against 391 us with 64-wide tensor-core tiles, but 52 rows take
// 500 us against 391 us, so anything beyond two 16-row tiles goes to the tile GEMM.
constexpr int SK_ROWS_MAX = 32;
template <typename T>
bool skinny_ok(const specdec_handle* h, int epi, int rows_ub, int N, int K, bool with_ln) {
    if (!std::is_same<T, bf16>::value || !h->use_skinny || rows_ub > SK_ROWS_MAX) return false;
    if (epi != EPI_STORE && epi != EPI_RELU && epi != EPI_GELU && epi != EPI_RESID && epi != EPI_QKV) return false;
    if (K % 32 || (with_ln && (K % 128 || K > 512))) return false;
    return skinny_smem(2, K) <= h->skinny_smem_cap;
}

template <int EPI, int MT, int G>
int skinny_launch_g(specdec_handle* h, SkinnyArgs& a, cudaStream_t st) {
    const int grid = cdiv(a.g.N, SK_NB * G);
    const size_t smem = skinny_smem(MT, a.g.K);
    cudaError_t e;
    if (G == 1 && h->use_sk_cluster && grid % 8 == 0 && (a.ln_x ? a.g.K % 128 == 0 : (a.g.K % 8 == 0 && a.g.lda % 8 == 0 && (h->use_sk_cluster >= 3 || (h->use_sk_cluster == 2 && a.g.K <= 512))))) {
        // clusters of 8 CTAs share the (normalised) input rows (see skinny_gemm.cuh)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(SK_WARPS * 32); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 8; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = h->use_pdl ? 2 : 1;
        e = a.ln_x ? cudaLaunchKernelEx(&cfg, k_skinny<EPI, MT, true, 1, true>, a)
                   : cudaLaunchKernelEx(&cfg, k_skinny<EPI, MT, false, 1, true>, a);
    } else {
        e = a.ln_x ? launch_pdl(h, k_skinny<EPI, MT, true, G>, dim3(grid), dim3(SK_WARPS * 32), smem, st, a)
                   : launch_pdl(h, k_skinny<EPI, MT, false, G>, dim3(grid), dim3(SK_WARPS * 32), smem, st, a);
    }
    if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("skinny GEMM launch: ") + cudaGetErrorString(e));
    KCHECK(h);
    return 0;
}
template <int EPI, int MT>
int skinny_launch_ln(specdec_handle* h, SkinnyArgs& a, cudaStream_t st) {
    return skinny_launch_g<EPI, MT, 1>(h, a, st);
}
template <int EPI>
int skinny_launch_mt(specdec_handle* h, SkinnyArgs& a, int rows_ub, cudaStream_t st) {
    (void)rows_ub;
    return skinny_launch_ln<EPI, 2>(h, a, st);
}
int skinny_launch(specdec_handle* h, int epi, SkinnyArgs& a, int rows_ub, cudaStream_t st) {
    switch (epi) {
        case EPI_STORE: return skinny_launch_mt<EPI_STORE>(h, a, rows_ub, st);
        case EPI_RELU: return skinny_launch_mt<EPI_RELU>(h, a, rows_ub, st);
        case EPI_GELU: return skinny_launch_mt<EPI_GELU>(h, a, rows_ub, st);
        case EPI_RESID: return skinny_launch_mt<EPI_RESID>(h, a, rows_ub, st);
        default: return skinny_launch_mt<EPI_QKV>(h, a, rows_ub, st);
    }
}
template <int EPI, int MT>
cudaError_t skinny_attr(int bytes) {
    cudaError_t e = cudaSuccess;
    auto set = [&](auto* f) { if (e == cudaSuccess) e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes); };
    set(k_skinny<EPI, MT, true, 1>); set(k_skinny<EPI, MT, false, 1>); set(k_skinny<EPI, MT, true, 1, true>); set(k_skinny<EPI, MT, false, 1, true>);
    return e;
}
template <int EPI>
cudaError_t skinny_attr_mt(int bytes) { return skinny_attr<EPI, 2>(bytes); }

// out = A W^T (+bias) with one of the epilogues; rows_ub bounds the grid, the live count is on the device.
template <typename T>
int gemm_once(specdec_handle* h, int epi, const void* A, int lda, const void* W, const float* bias, int N, int K, int cnt,
              int rows_ub, void* out, int ldo, float* resid, cudaStream_t st, const float* ldv, const int* ld_id,
              int* n_tiles_out, const KvDest* kv, const LnSpec* lnp);

template <typename T>
int gemm(specdec_handle* h, int epi, const void* A, int lda, const void* W, const float* bias, int N, int K, int cnt,
         int rows_ub, void* out, int ldo, float* resid, cudaStream_t st, const float* ldv = nullptr,
         const int* ld_id = nullptr, int* n_tiles_out = nullptr, const KvDest* kv = nullptr,
         const LnSpec* lnp = nullptr) {
    TRY(gemm_once<T>(h, epi, A, lda, W, bias, N, K, cnt, rows_ub, out, ldo, resid, st, ldv, ld_id, n_tiles_out, kv, lnp));
    // diagnostics: GEMMs that only write outputs (no residual accumulation) can run twice with the same result
    if ((h->diag_repeat & 4) && epi != EPI_RESID && epi != EPI_STATS)
        TRY(gemm_once<T>(h, epi, A, lda, W, bias, N, K, cnt, rows_ub, out, ldo, resid, st, ldv, ld_id, n_tiles_out, kv, lnp));
    if ((h->diag_repeat & 8) && epi == EPI_STATS)
        TRY(gemm_once<T>(h, epi, A, lda, W, bias, N, K, cnt, rows_ub, out, ldo, resid, st, ldv, ld_id, n_tiles_out, kv, lnp));
    return 0;
}

template <typename T>
int gemm_once(specdec_handle* h, int epi, const void* A, int lda, const void* W, const float* bias, int N, int K, int cnt,
              int rows_ub, void* out, int ldo, float* resid, cudaStream_t st, const float* ldv, const int* ld_id,
              int* n_tiles_out, const KvDest* kv, const LnSpec* lnp) {
    if (rows_ub <= 0) return 0;
    // (not in the encoders: the two encoders run side by side on two streams, and the weight-streaming kernels' 64-256
    // CTAs per launch get in each other's way there -- 440 us against 386 us with 8-32-CTA tile GEMMs for a 32-token source)
    const bool skinny = (cnt != CNT_ENC || h->enc_skinny_now) && skinny_ok<T>(h, epi, rows_ub, N, K, lnp != nullptr);
    if (lnp && !skinny) {           // separate normalisation launch, then a plain GEMM on its output
        TRY(ln_or_fused<T>(h, lnp->x, lnp->g, lnp->b, cnt, rows_ub, h->y, K, st));
        A = h->y; lda = K;
    }
    const specdec_handle::NextLn want_ln = h->next_ln;
    if (epi == EPI_RESID) { h->fused_x = nullptr; h->next_ln = {nullptr, nullptr, nullptr}; }   // the residual rows change
    GemmArgs<T> g;
    g.A = (const T*)A; g.lda = lda; g.W = (const T*)W; g.bias = bias; g.N = N; g.K = K;
    g.n_rows = h->ses.counters + cnt; g.rows_static = (cnt == CNT_VERIFY || cnt == CNT_ENC) ? rows_ub : -1; g.out = (T*)out; g.ldo = ldo; g.resid = resid;
    g.one_m_tile = 0; g.act = h->cfg.ffn_activation;
    g.ln_g = nullptr; g.ln_b = nullptr; g.ln_eps = 1e-5f; g.ln_out = nullptr;
    g.part = h->part; g.ld = ldv; g.ld_id = ld_id; g.n_tiles = cdiv(N, 64); g.want_sum = h->want_lse;
    g.seq = nullptr; g.pos = nullptr; g.kc = nullptr; g.vc = nullptr; g.kv_d = 0;
    g.pg.table = h->page_table; g.pg.page_tokens = h->cfg.page_tokens; g.pg.max_pages = h->pages_per_seq;
    g.trace = (h->want_trace && epi == (h->want_trace >= 10 ? h->want_trace - 10 : EPI_STATS)) ? h->trace_buf + 200 : nullptr;
    if (kv) { g.seq = kv->seq; g.pos = kv->pos; g.kc = (T*)kv->kc; g.vc = (T*)kv->vc; g.kv_d = kv->d; }
    if constexpr (std::is_same<T, bf16>::value) {
        if (skinny) {
            SkinnyArgs sa; sa.g = g;
            sa.ln_x = lnp ? lnp->x : nullptr; sa.ln_g = lnp ? lnp->g : nullptr; sa.ln_b = lnp ? lnp->b : nullptr;
            sa.ln_eps = 1e-5f; sa.ln_out = nullptr; sa.err_word = h->ses.counters + 7;
            sa.trace = h->want_trace ? h->trace_buf + 216 + 6 * ((epi == EPI_RELU || epi == EPI_GELU) ? 0 : epi == EPI_RESID ? 1 : epi == EPI_QKV ? 2 : 3) : nullptr;
            TRY(skinny_launch(h, epi, sa, rows_ub, st));
            return 0;
        }
    }
    if constexpr (std::is_same<T, bf16>::value) {
        if (h->use_tc && sd::tc_supported(N, K) && (epi != EPI_STATS || N >= 128)) {
            if (epi == EPI_RESID && h->use_ln_fuse && want_ln.g && want_ln.out && sd::tc_ln_fusable(N, K)) {
                g.ln_g = want_ln.g; g.ln_b = want_ln.b; g.ln_out = (T*)want_ln.out;
                if (sd::gemm_tc_launch_ln(h->tma, g, rows_ub, st) != 0)
                    return fail(h, SPECDEC_ERR_CUDA, "tensor-core GEMM launch failed: " + h->tma.err);
                h->fused_x = resid; h->fused_g = want_ln.g; h->fused_out = want_ln.out;
                ++h->launches;
                return 0;
            }
            if (epi == EPI_RESID && h->use_splitk && h->splitk_ready && sd::spk_supported(N, K, rows_ub, h->tma.n_sm)) {
                if (sd::spk_launch(h->tma, g, rows_ub, st) != 0)
                    return fail(h, SPECDEC_ERR_CUDA, "tensor-core GEMM launch failed: " + h->tma.err);
                ++h->launches;
                return 0;
            }
            int rc = (h->use_pair && sd::tc_pair_wanted(epi, N, K, rows_ub))
                         ? sd::gemm_tc_pair_launch(h->tma, epi, g, rows_ub, st, n_tiles_out)
                         : sd::gemm_tc_launch(h->tma, epi, g, rows_ub, st, n_tiles_out);
            if (rc != 0) return fail(h, SPECDEC_ERR_CUDA, "tensor-core GEMM launch failed: " + h->tma.err);
            if (epi == EPI_STATS && g.n_tiles > h->n_tiles_cap) return fail(h, SPECDEC_ERR_CAPACITY, "row statistics: more vocabulary tiles than the table holds");
            ++h->launches;
            return 0;
        }
    }
    if (n_tiles_out) *n_tiles_out = g.n_tiles;
    dim3 grid(cdiv(N, 64), cdiv(rows_ub, 64));
    switch (epi) {
        case EPI_STORE: k_gemm_simt<T, EPI_STORE><<<grid, 256, 0, st>>>(g); break;
        case EPI_RELU: case EPI_GELU: k_gemm_simt<T, EPI_RELU><<<grid, 256, 0, st>>>(g); break;   // activation chosen by g.act
        case EPI_RESID: k_gemm_simt<T, EPI_RESID><<<grid, 256, 0, st>>>(g); break;
        case EPI_STATS: k_gemm_simt<T, EPI_STATS><<<grid, 256, 0, st>>>(g); break;
        default: k_gemm_simt<T, EPI_F32><<<grid, 256, 0, st>>>(g); break;
    }
    KCHECK(h);
    return 0;
}

// Attention of the pass described by `r`.  bf16 handles with 64-wide heads use the tensor-core tile
// kernel (one CTA per 32-query tile, head, sequence; q_ub bounds the queries of one sequence);
// everything else uses the warp-per-(row, head) kernel.
template <typename T>
int attn_once(specdec_handle* h, bool paged, const void* q, int q_stride, const int* q_index, const void* k, const void* v,
         int kv_stride, const int* kv_off, const Rows& r, const int* nkeys, int cnt, int rows_ub, int q_ub, void* out,
         int out_stride, int n_heads, int d_head, int max_keys, cudaStream_t st, const int* pre_keys = nullptr) {
    if (rows_ub <= 0) return 0;
    if constexpr (std::is_same<T, bf16>::value) {
        const size_t smem = attn_tc_smem(max_keys);
        // the streaming kernel where the one-shot kernel cannot hold the keys, and where the SMs are full of CTAs
        // and the keys are many (its small footprint keeps the occupancy up; with few CTAs its block-by-block walk
        // is slower than one big request)
        const long long attn_ctas = (long long)cdiv(q_ub, ATT_Q) * n_heads * h->B;
        const bool stream = h->use_tc_attn && d_head == 64 &&
                            (h->attn_stream >= 2 ||
                             (h->attn_stream == 1 && (smem > h->attn_tc_smem_cap ||
                                                      (max_keys > h->attn_stream_keys && attn_ctas >= 4LL * h->tma.n_sm))));
        if (stream || (h->use_tc_attn && d_head == 64 && smem <= h->attn_tc_smem_cap)) {
            AttnTcArgs a;
            a.q = (const bf16*)q; a.q_stride = q_stride; a.q_index = q_index;
            a.k = (const bf16*)k; a.v = (const bf16*)v; a.kv_stride = kv_stride; a.kv_off = kv_off;
            a.pg.table = h->page_table; a.pg.page_tokens = h->cfg.page_tokens; a.pg.max_pages = h->pages_per_seq;
            a.q_off = r.q_off; a.q_cnt = r.q_cnt; a.nkeys = nkeys; a.pre_keys = h->use_pdl ? pre_keys : nullptr;
            a.out = (bf16*)out; a.out_stride = out_stride; a.max_keys = max_keys;
            a.scale = 1.0f / sqrtf((float)d_head);
            dim3 grid(cdiv(q_ub, ATT_Q), n_heads, h->B);
            if (stream) {          // key blocks through a ring of stages: shared memory independent of the key count
                const bool deep = h->attn_stream != 3 && (long long)grid.x * grid.y * grid.z < 4LL * h->tma.n_sm;    // few CTAs: more bytes in flight per CTA
                cudaError_t e = deep ? (paged ? launch_pdl(h, k_attn_stream<true, 4>, grid, dim3(128), (size_t)ats_smem(4), st, a)
                                              : launch_pdl(h, k_attn_stream<false, 4>, grid, dim3(128), (size_t)ats_smem(4), st, a))
                                     : (paged ? launch_pdl(h, k_attn_stream<true, 2>, grid, dim3(128), (size_t)ats_smem(2), st, a)
                                              : launch_pdl(h, k_attn_stream<false, 2>, grid, dim3(128), (size_t)ats_smem(2), st, a));
                if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(e));
                KCHECK(h);
                return 0;
            }
            // 4 warps when the SMs are saturated with CTAs anyway, 8 when a CTA's own latency chain is what counts;
            // scores stay in registers (smaller shared memory: more CTAs per SM) when the keys fit 6 tiles per warp
            const long long ctas = (long long)grid.x * grid.y * grid.z;
            const int nkp = (max_keys + 15) & ~15;
            auto per_sm_of = [](size_t sm) { return (long long)(227 * 1024) / (long long)(sm + 1024); };
            // (measured: the register variant is slower per CTA, 357 -> 387 us per batch-1 step, and pays off only where
            // shared memory held the occupancy down: 1018 -> 873 us per step at batch 128 over a 256-token prefix)
            // (choosing it wherever it saves a wave of CTAs was tried too: 479 vs 469 us per 128-sequence draft step)
            bool rs = nkp <= attn_tc_rs_max_keys(8) &&
                      (h->attn_rs == 2 || (h->attn_rs == 1 && per_sm_of(smem) <= 2 && ctas > 2LL * h->tma.n_sm));
            size_t smem_l = rs ? attn_tc_smem_rs(max_keys) : smem;
            bool wide = h->attn_warps ? h->attn_warps == 8 : (per_sm_of(smem_l) <= 2 || ctas < 4LL * h->tma.n_sm);
            if (rs && !wide && nkp > attn_tc_rs_max_keys(4)) {       // too many keys for four warps' registers
                if (h->attn_warps == 4) { rs = false; smem_l = smem; } else wide = true;
            }
            cudaError_t e;
            if (rs) e = wide ? (paged ? launch_pdl(h, k_attn_tc<true, 8, true>, grid, dim3(256), smem_l, st, a)
                                      : launch_pdl(h, k_attn_tc<false, 8, true>, grid, dim3(256), smem_l, st, a))
                             : (paged ? launch_pdl(h, k_attn_tc<true, 4, true>, grid, dim3(128), smem_l, st, a)
                                      : launch_pdl(h, k_attn_tc<false, 4, true>, grid, dim3(128), smem_l, st, a));
            else e = wide ? (paged ? launch_pdl(h, k_attn_tc<true, 8>, grid, dim3(256), smem, st, a)
                                   : launch_pdl(h, k_attn_tc<false, 8>, grid, dim3(256), smem, st, a))
                          : (paged ? launch_pdl(h, k_attn_tc<true, 4>, grid, dim3(128), smem, st, a)
                                   : launch_pdl(h, k_attn_tc<false, 4>, grid, dim3(128), smem, st, a));
            if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(e));
            KCHECK(h);
            return 0;
        }
    }
    AttnArgs<T> a;
    a.q = (const T*)q; a.q_stride = q_stride; a.q_index = q_index;
    a.k = (const T*)k; a.v = (const T*)v; a.kv_stride = kv_stride; a.kv_off = kv_off;
    a.pg.table = h->page_table; a.pg.page_tokens = h->cfg.page_tokens; a.pg.max_pages = h->pages_per_seq;
    a.seq = r.seq; a.nkeys = nkeys; a.n_rows = h->ses.counters + cnt;
    a.out = (T*)out; a.out_stride = out_stride;
    a.n_heads = n_heads; a.d_head = d_head; a.max_keys = max_keys;
    a.scale = 1.0f / sqrtf((float)d_head);
    const int wpb = 4;
    size_t smem = (size_t)wpb * (max_keys + d_head) * sizeof(float);
    long long warps = (long long)rows_ub * n_heads;
    int blocks = (int)((warps + wpb - 1) / wpb);
    if (paged) k_attention<T, true><<<blocks, wpb * 32, smem, st>>>(a);
    else k_attention<T, false><<<blocks, wpb * 32, smem, st>>>(a);
    KCHECK(h);
    return 0;
}


template <typename T>
int attn(specdec_handle* h, bool paged, const void* q, int q_stride, const int* q_index, const void* k, const void* v,
         int kv_stride, const int* kv_off, const Rows& r, const int* nkeys, int cnt, int rows_ub, int q_ub, void* out,
         int out_stride, int n_heads, int d_head, int max_keys, cudaStream_t st, const int* pre_keys = nullptr) {
    TRY(attn_once<T>(h, paged, q, q_stride, q_index, k, v, kv_stride, kv_off, r, nkeys, cnt, rows_ub, q_ub, out, out_stride,
                     n_heads, d_head, max_keys, st, pre_keys));
    if (h->diag_repeat & 1)
        TRY(attn_once<T>(h, paged, q, q_stride, q_index, k, v, kv_stride, kv_off, r, nkeys, cnt, rows_ub, q_ub, out, out_stride,
                         n_heads, d_head, max_keys, st, pre_keys));
    return 0;
}

// With the "profile" option on, the vocabulary-projection launches are bracketed by event pairs.
void prof_mark(specdec_handle* h, cudaStream_t st) {
    if (!h->profile) return;
    if (h->prof_n >= h->prof_ev.size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        h->prof_ev.push_back(e);
    }
    cudaEventRecord(h->prof_ev[h->prof_n++], st);
}
void prof_collect(specdec_handle* h) {
    for (size_t i = 0; i + 1 < h->prof_n; i += 2) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, h->prof_ev[i], h->prof_ev[i + 1]) == cudaSuccess) { h->prof_ms += t; ++h->prof_launches; }
    }
    h->prof_n = 0;
}

// One pre-LN block on `rows_ub` rows of the residual stream x (encoder: no cross-attention).
// Self-attention keys come from the block's own QKV rows (contiguous) or, for the verifier,
// from the paged cache after the block's K/V were scattered into it.
// kc / vc: the paged cache the block's K / V go to and its attention reads (verifier; prefix-causal drafter), or null:
// keys and values are the block's own rows.  pre_keys: per sequence, cache positions that predate the step.
template <typename T>
int block_self(specdec_handle* h, const ModelW& m, const LayerW& w, float* x, const Rows& r, int cnt, int rows_ub,
               int q_ub, void* kc, void* vc, const int* pre_keys, int max_keys, cudaStream_t st, const float* next_g = nullptr,
               const float* next_b = nullptr) {
    const int d = m.dm.d_model, H = m.dm.n_heads, dh = d / H;
    const size_t e = h->esz;
    const bool verify = kc != nullptr;
    const LnSpec l1{x, w.ln1_g, w.ln1_b};
    if (verify && tc_usable<T>(h, 3 * d, d) && d % 32 == 0) {
        // K and V columns leave the GEMM epilogue straight into the paged cache
        KvDest kv{r.seq, r.pos, kc, vc, d};
        TRY(gemm<T>(h, EPI_QKV, h->y, d, w.qkv_w, w.qkv_b, 3 * d, d, cnt, rows_ub, h->qkv, 3 * d, nullptr, st, nullptr,
                    nullptr, nullptr, &kv, &l1));
    } else {
        TRY(gemm<T>(h, EPI_STORE, h->y, d, w.qkv_w, w.qkv_b, 3 * d, d, cnt, rows_ub, h->qkv, 3 * d, nullptr, st, nullptr,
                    nullptr, nullptr, nullptr, &l1));
        if (verify) {
            Paged pg{h->page_table, h->cfg.page_tokens, h->pages_per_seq};
            k_kv_scatter<T><<<rows_ub, 128, 0, st>>>((const T*)h->qkv, r.seq, r.pos, h->ses.counters + cnt, pg,
                                                     (T*)kc, (T*)vc, d);
            KCHECK(h);
        }
    }
    if (verify) {
        TRY(attn<T>(h, true, h->qkv, 3 * d, nullptr, kc, vc, d, nullptr, r, r.nk_self, cnt,
                    rows_ub, q_ub, h->att, d, H, dh, max_keys, st, pre_keys));
    } else {
        TRY(attn<T>(h, false, h->qkv, 3 * d, nullptr, (char*)h->qkv + (size_t)d * e, (char*)h->qkv + (size_t)2 * d * e,
                    3 * d, r.kv_off, r, r.nk_self, cnt, rows_ub, q_ub, h->att, d, H, dh, max_keys, st));
    }
    h->next_ln = {next_g, next_b, h->y};             // the LayerNorm that reads the residual stream next
    TRY(gemm<T>(h, EPI_RESID, h->att, d, w.o_w, w.o_b, d, d, cnt, rows_ub, nullptr, 0, x, st));
    return 0;
}

template <typename T>
int block_cross(specdec_handle* h, const ModelW& m, const LayerW& w, float* x, const Rows& r, int cnt, int rows_ub,
                int q_ub, int layer, cudaStream_t st) {
    const int d = m.dm.d_model, H = m.dm.n_heads, dh = d / H;
    const size_t e = h->esz;
    const LnSpec lc{x, w.lnc_g, w.lnc_b};
    TRY(gemm<T>(h, EPI_STORE, h->y, d, w.cq_w, w.cq_b, d, d, cnt, rows_ub, h->q, d, nullptr, st, nullptr, nullptr, nullptr,
                nullptr, &lc));
    TRY(attn<T>(h, false, h->q, d, nullptr, m.ckv[layer], (char*)m.ckv[layer] + (size_t)d * e, m.ckv_stride, r.kv_off_cross,
                r, r.nk_cross, cnt, rows_ub, q_ub, h->att, d, H, dh, h->S_max, st, h->ses.src_len));   // encoder K/V: all of it
    h->next_ln = {w.ln2_g, w.ln2_b, h->y};           // the feed-forward sublayer's LayerNorm comes next
    TRY(gemm<T>(h, EPI_RESID, h->att, d, w.co_w, w.co_b, d, d, cnt, rows_ub, nullptr, 0, x, st));
    return 0;
}

template <typename T>
int block_ffn(specdec_handle* h, const ModelW& m, const LayerW& w, float* x, int cnt, int rows_ub, cudaStream_t st,
              const float* next_g = nullptr, const float* next_b = nullptr, void* next_out = nullptr) {
    const int d = m.dm.d_model, f = m.dm.d_ffn;
    const LnSpec l2{x, w.ln2_g, w.ln2_b};
    TRY(gemm<T>(h, h->cfg.ffn_activation == SPECDEC_ACT_GELU ? EPI_GELU : EPI_RELU, h->y, d, w.w1, w.b1, f, d, cnt, rows_ub, h->hbuf, f, nullptr, st, nullptr, nullptr, nullptr,
                nullptr, &l2));
    h->next_ln = {next_g, next_b, next_out ? next_out : h->y};
    TRY(gemm<T>(h, EPI_RESID, h->hbuf, f, w.w2, w.b2, d, f, cnt, rows_ub, nullptr, 0, x, st));
    return 0;
}

template <typename T>
int embed(specdec_handle* h, const ModelW& m, const Rows& r, const float* pos_table, int cnt, int rows_ub,
          cudaStream_t st) {
    if (rows_ub <= 0) return 0;
    const int d = m.dm.d_model;
    h->fused_x = nullptr;                            // new residual rows: nothing normalised is pending
    CUDA_TRY(h, launch_pdl(h, k_embed<T>, dim3(rows_ub), dim3(128), 0, st, (const int*)r.tok, (const int*)r.pos, (const int*)(h->ses.counters + cnt), (const T*)m.embed, (const float*)pos_table, h->x, d,
                                        sqrtf((float)d), m.dm.vocab, m.dm.max_pos));
    KCHECK(h);
    return 0;
}

// ---------------------------------------------------------------- encode
void use_workset(specdec_handle* h, int i) {
    const specdec_handle::WorkSet& w = h->ws[i];
    h->x = w.x; h->y = w.y; h->qkv = w.qkv; h->att = w.att; h->q = w.q; h->hbuf = w.hbuf; h->mem = w.mem;
}

template <typename T>
int encode_model(specdec_handle* h, ModelW& m, cudaStream_t st) {
    const int R = h->B * h->S_max, d = m.dm.d_model;
    h->enc_skinny_now = h->enc_skinny == 2 || (h->enc_skinny == 1 && &m == &h->dra);
    struct Off { specdec_handle* h; ~Off() { h->enc_skinny_now = false; } } off{h};
    TRY(embed<T>(h, m, h->rows, m.pos_enc, CNT_ENC, R, st));
    for (int l = 0; l < m.dm.enc_layers; ++l) {
        const bool last = l + 1 == m.dm.enc_layers;
        TRY(block_self<T>(h, m, m.enc[l], h->x, h->rows, CNT_ENC, R, h->S_max, nullptr, nullptr, nullptr, h->S_max, st, m.enc[l].ln2_g, m.enc[l].ln2_b));
        TRY(block_ffn<T>(h, m, m.enc[l], h->x, CNT_ENC, R, st, last ? m.enc_lnf_g : m.enc[l + 1].ln1_g,
                         last ? m.enc_lnf_b : m.enc[l + 1].ln1_b, last ? h->mem : nullptr));
    }
    TRY(ln_or_fused<T>(h, h->x, m.enc_lnf_g, m.enc_lnf_b, CNT_ENC, R, h->mem, d, st));
    // cross-attention K / V of every decoder layer in one projection ("the encoder is forwarded only once", Section 3.1.2)
    TRY(gemm<T>(h, EPI_STORE, h->mem, d, m.dec[0].ckv_w, m.dec[0].ckv_b, m.ckv_stride, d, CNT_ENC, R, m.ckv[0], m.ckv_stride,
                nullptr, st));
    return 0;
}

template <typename T>
int encode_impl(specdec_handle* h, const int* d_src, const int* d_src_len, const int* d_max_tgt, int B, int S_max,
                cudaStream_t st) {
    h->B = B; h->S_max = S_max; h->len_ub = 0;
    h->dnew_ub = 1; h->drafter_pc_session = h->drafter_pc;
    h->encoded = false; h->verified = false; h->drafted = false;
    k_session_init<<<cdiv(B, 128), 128, 0, st>>>(h->ses, d_src_len, d_max_tgt, B, h->T_cap, S_max);
    KCHECK(h);
    k_count_active<<<1, 32, 0, st>>>(h->ses, B);
    KCHECK(h);
    {
        const int R = B * S_max;
        k_enc_prep<<<cdiv(R, 256), 256, 0, st>>>(d_src, h->ses.src_len, B, S_max, h->rows, h->ses.counters);
        KCHECK(h);
    }
    // the two encoders are independent: the drafter's runs on a second stream in its own workspace
    const bool side = h->enc_stream != nullptr;
    cudaStream_t st2 = side ? h->enc_stream : st;
    if (side) {
        CUDA_TRY(h, cudaEventRecord(h->enc_fork, st));
        CUDA_TRY(h, cudaStreamWaitEvent(st2, h->enc_fork, 0));
    }
    int rc = encode_model<T>(h, h->ver, st);
    if (rc == 0) {
        if (side) use_workset(h, 1);
        rc = encode_model<T>(h, h->dra, st2);
        use_workset(h, 0);
    }
    if (side) {
        cudaEventRecord(h->enc_join, st2);
        cudaStreamWaitEvent(st, h->enc_join, 0);
    }
    if (rc != 0) return rc;
    h->encoded = true;
    return 0;
}

// ---------------------------------------------------------------- draft (Section 3.1.3)
template <typename T>
int draft_impl(specdec_handle* h, int k, int* d_draft, cudaStream_t st) {
    ModelW& m = h->dra;
    const int B = h->B, d = m.dm.d_model, H = m.dm.n_heads, dh = d / H, L = m.dm.dec_layers;
    const size_t e = h->esz;
    const int len_ub = std::min(h->len_ub, h->T_cap);
    const bool pc = h->drafter_pc_session != 0;
    // rows of the full pass per sequence: the whole [BOS, committed, MASK x k] input, or (prefix-causal reading) only the
    // prefix positions its K/V cache does not hold yet plus the k [MASK] rows
    const int per_seq = pc ? std::min(h->dnew_ub, len_ub + 1) + k : len_ub + 1 + k;
    const int R1 = B * per_seq, R2 = B * k, max_keys = len_ub + 1 + k;
    // row metadata of the pass and the embedding of its rows in one kernel (one block per sequence)
    h->fused_x = nullptr;
    // blocks per sequence: enough to fill the machine at small batches, never fewer than two rows a block
    const int parts = std::max(1, std::min(cdiv(592, B), cdiv(h->T_cap + k + 1, 2)));
    if (pc) CUDA_TRY(h, launch_pdl(h, k_draft_prep_pc<T>, dim3(B, parts), dim3(128), 0, st, h->ses, B, k, h->S_max, h->cfg.bos_id, h->cfg.mask_id, h->rows, h->mrows,
                                   (const T*)m.embed, (const float*)m.pos_dec, h->x, d, sqrtf((float)d), m.dm.vocab, m.dm.max_pos));
    else CUDA_TRY(h, launch_pdl(h, k_draft_prep<T>, dim3(B, parts), dim3(128), 0, st, h->ses, B, k, h->S_max, h->cfg.bos_id, h->cfg.mask_id, h->rows, h->mrows,
                                (const T*)m.embed, (const float*)m.pos_dec, h->x, d, sqrtf((float)d), m.dm.vocab, m.dm.max_pos));
    KCHECK(h);
    for (int l = 0; l + 1 < L; ++l) {
        TRY(block_self<T>(h, m, m.dec[l], h->x, h->rows, CNT_DRAFT_ALL, R1, per_seq, pc ? h->dkc[l] : nullptr, pc ? h->dvc[l] : nullptr, nullptr,
                          max_keys, st, m.dec[l].lnc_g, m.dec[l].lnc_b));
        TRY(block_cross<T>(h, m, m.dec[l], h->x, h->rows, CNT_DRAFT_ALL, R1, per_seq, l, st));
        TRY(block_ffn<T>(h, m, m.dec[l], h->x, CNT_DRAFT_ALL, R1, st, m.dec[l + 1].ln1_g, m.dec[l + 1].ln1_b));
    }
    // last layer: K/V from every row, queries and everything after them from the k mask rows only
    const LayerW& w = m.dec[L - 1];
    const LnSpec l1{h->x, w.ln1_g, w.ln1_b};
    const bool scatter_in_gemm = pc && tc_usable<T>(h, 3 * d, d) && d % 32 == 0;
    if (scatter_in_gemm) {
        KvDest kv{h->rows.seq, h->rows.pos, h->dkc[L - 1], h->dvc[L - 1], d};
        TRY(gemm<T>(h, EPI_QKV, h->y, d, w.qkv_w, w.qkv_b, 3 * d, d, CNT_DRAFT_ALL, R1, h->qkv, 3 * d, nullptr, st, nullptr,
                    nullptr, nullptr, &kv, &l1));
    } else {
        TRY(gemm<T>(h, EPI_STORE, h->y, d, w.qkv_w, w.qkv_b, 3 * d, d, CNT_DRAFT_ALL, R1, h->qkv, 3 * d, nullptr, st, nullptr,
                    nullptr, nullptr, nullptr, &l1));
        if (pc) {
            Paged pg{h->page_table, h->cfg.page_tokens, h->pages_per_seq};
            k_kv_scatter<T><<<R1, 128, 0, st>>>((const T*)h->qkv, h->rows.seq, h->rows.pos, h->ses.counters + CNT_DRAFT_ALL, pg,
                                                (T*)h->dkc[L - 1], (T*)h->dvc[L - 1], d);
            KCHECK(h);
        }
    }
    CUDA_TRY(h, launch_pdl(h, k_gather_rows, dim3(R2), dim3(128), 0, st, (const float*)h->x, (const int*)h->mrows.src_row, (const int*)(h->ses.counters + CNT_DRAFT_MASK), h->x2, d));
    KCHECK(h);
    if (pc)
        TRY(attn<T>(h, true, h->qkv, 3 * d, h->mrows.src_row, h->dkc[L - 1], h->dvc[L - 1], d, nullptr, h->mrows, h->mrows.nk_self,
                    CNT_DRAFT_MASK, R2, k, h->att, d, H, dh, max_keys, st));
    else
        TRY(attn<T>(h, false, h->qkv, 3 * d, h->mrows.src_row, (char*)h->qkv + (size_t)d * e,
                    (char*)h->qkv + (size_t)2 * d * e, 3 * d, h->mrows.kv_off, h->mrows, h->mrows.nk_self,
                    CNT_DRAFT_MASK, R2, k, h->att, d, H, dh, max_keys, st));
    TRY(gemm<T>(h, EPI_RESID, h->att, d, w.o_w, w.o_b, d, d, CNT_DRAFT_MASK, R2, nullptr, 0, h->x2, st));
    TRY(block_cross<T>(h, m, w, h->x2, h->mrows, CNT_DRAFT_MASK, R2, k, L - 1, st));
    TRY(block_ffn<T>(h, m, w, h->x2, CNT_DRAFT_MASK, R2, st, m.dec_lnf_g, m.dec_lnf_b));
    TRY(ln_or_fused<T>(h, h->x2, m.dec_lnf_g, m.dec_lnf_b, CNT_DRAFT_MASK, R2, h->y, d, st));
    int n_tiles = 0;
    TRY(gemm<T>(h, EPI_STATS, h->y, d, m.embed, nullptr, m.dm.vocab, d, CNT_DRAFT_MASK, R2, nullptr, 0, nullptr, st,
                nullptr, nullptr, &n_tiles));
    CUDA_TRY(h, launch_pdl(h, k_draft_argmax, dim3(cdiv(R2, 4)), dim3(128), 0, st, (const RowPart*)h->part, n_tiles,
                           (const int*)(h->ses.counters + CNT_DRAFT_MASK), (const int*)h->mrows.slot, d_draft,
                           (const int*)(h->script_on ? h->script : nullptr), h->T_cap + h->k_cap, (const int*)h->ses.len, k));
    KCHECK(h);
    h->drafted = true; h->verified = false;
    h->last_draft_rows_ub = R2;
    h->dnew_ub = 0;                                  // the cache now holds every committed position
    return 0;
}

// ---------------------------------------------------------------- verify (Section 2, Section 3.2)
template <typename T>
int verify_impl(specdec_handle* h, const int* d_draft, int k, int beta, float tau, int* d_accepted, int* d_bif,
                cudaStream_t st) {
    ModelW& m = h->ver;
    const int B = h->B, d = m.dm.d_model, L = m.dm.dec_layers, M = B * (k + 1);
    const int max_keys = std::min(h->len_ub, h->T_cap) + k + 1;
    if (d_draft != h->v_draft && k > 0)
        CUDA_TRY(h, cudaMemcpyAsync(h->v_draft, d_draft, (size_t)B * k * 4, cudaMemcpyDeviceToDevice, st));
    // row metadata and embedding of the block in one kernel
    h->fused_x = nullptr;
    CUDA_TRY(h, launch_pdl(h, k_verify_prep_embed<T>, dim3(M), dim3(128), 0, st, h->ses, (const int*)h->v_draft, B, k, h->S_max, h->cfg.bos_id,
                           h->rows, (const T*)m.embed, (const float*)m.pos_dec, h->x, d, sqrtf((float)d), m.dm.vocab, m.dm.max_pos));
    KCHECK(h);
    for (int l = 0; l < L; ++l) {
        const bool last = l + 1 == L;
        TRY(block_self<T>(h, m, m.dec[l], h->x, h->rows, CNT_VERIFY, M, k + 1, h->kc[l], h->vc[l], h->ses.len /* cached prefix: positions < len */,
                          max_keys, st, m.dec[l].lnc_g, m.dec[l].lnc_b));
        TRY(block_cross<T>(h, m, m.dec[l], h->x, h->rows, CNT_VERIFY, M, k + 1, l, st));
        TRY(block_ffn<T>(h, m, m.dec[l], h->x, CNT_VERIFY, M, st, last ? m.dec_lnf_g : m.dec[l + 1].ln1_g,
                         last ? m.dec_lnf_b : m.dec[l + 1].ln1_b));
    }
    const bool ln_pending = !(h->x == h->fused_x && m.dec_lnf_g == h->fused_g && h->y == h->fused_out);
    if (ln_pending && d % 128 == 0 && d <= 1024 && !(h->diag_repeat & 2)) {
        // final LayerNorm and the pre-pass logit of every row's draft in one kernel
        cudaError_t e = cudaSuccess;
        const dim3 grid(cdiv(M, 8)), block(256);
#define LN_LD(NC) e = launch_pdl(h, k_layernorm_ld<T, NC>, grid, block, 0, st, (const float*)h->x, (const float*)m.dec_lnf_g, (const float*)m.dec_lnf_b, (T*)h->y, d, 1e-5f, \
                                 (const T*)m.embed, (const int*)h->v_draft, B, k, m.dm.vocab, h->ld, h->ld_id)
        switch (d / 128) {
            case 1: LN_LD(1); break; case 2: LN_LD(2); break; case 3: LN_LD(3); break; case 4: LN_LD(4); break;
            case 5: LN_LD(5); break; case 6: LN_LD(6); break; case 7: LN_LD(7); break; default: LN_LD(8); break;
        }
#undef LN_LD
        if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("final layer norm launch: ") + cudaGetErrorString(e));
        KCHECK(h);
    } else {
        TRY(ln_or_fused<T>(h, h->x, m.dec_lnf_g, m.dec_lnf_b, CNT_VERIFY, M, h->y, d, st));
        CUDA_TRY(h, launch_pdl(h, k_draft_logit<T>, dim3(cdiv(M, 4)), dim3(128), 0, st, (const T*)h->y, (const T*)m.embed,
                               (const int*)h->v_draft, B, k, d, m.dm.vocab, h->ld, h->ld_id));
        KCHECK(h);
    }
    int n_tiles = 0;
    prof_mark(h, st);
    TRY(gemm<T>(h, EPI_STATS, h->y, d, m.embed, nullptr, m.dm.vocab, d, CNT_VERIFY, M, nullptr, 0, nullptr, st, h->ld,
                h->ld_id, &n_tiles));
    prof_mark(h, st);
    FusedCommit fc{h->ses, h->v_draft, h->cfg.eos_id, h->h_post, h->fuse_commit ? 1 : 0};
    CUDA_TRY(h, launch_pdl(h, k_accept, dim3(B), dim3(1024), (size_t)(k + 1) * sizeof(RowPart), st, (const RowPart*)h->part, n_tiles,
                           (const float*)h->ld, (const int*)h->ld_id, k, beta, tau, h->accepted, h->bif, h->row_stats, h->want_lse, fc));
    KCHECK(h);
    h->commit_done = h->fuse_commit;
    if (d_accepted) CUDA_TRY(h, cudaMemcpyAsync(d_accepted, h->accepted, (size_t)B * 4, cudaMemcpyDeviceToDevice, st));
    if (d_bif) CUDA_TRY(h, cudaMemcpyAsync(d_bif, h->bif, (size_t)B * 4, cudaMemcpyDeviceToDevice, st));
    h->last_k = k; h->verified = true; h->drafted = false;
    return 0;
}

int commit_impl(specdec_handle* h, const int* d_keep, const int* d_next, cudaStream_t st) {
    const int k = h->last_k;
    if (h->commit_done && !d_keep && !d_next) {
        h->commit_done = false;                    // the acceptance scan of this verify pass has committed already
    } else {
        CUDA_TRY(h, launch_pdl(h, k_commit, dim3(cdiv(h->B, 128)), dim3(128), 0, st, h->ses, (const int*)h->v_draft,
                               (const int*)(d_keep ? d_keep : h->accepted), (const int*)(d_next ? d_next : h->bif), h->B, k, h->cfg.eos_id, h->h_post));
        KCHECK(h);
    }
    h->len_ub = std::min(h->len_ub + k + 1, h->T_cap);
    h->dnew_ub = std::min(h->dnew_ub + k + 1, h->T_cap + 1);
    h->verified = false;
    return 0;
}

// Stream a call really runs on: the caller's, or the handle's own when the caller gave a default stream.
struct StreamScope {
    specdec_handle* h; cudaStream_t user, st; bool redirected;
    StreamScope(specdec_handle* h_, void* stream) : h(h_), user((cudaStream_t)stream), st((cudaStream_t)stream), redirected(false) {
        if ((user == nullptr || user == cudaStreamLegacy || user == cudaStreamPerThread) && h->own_stream) {
            cudaEventRecord(h->fence_in, user);
            cudaStreamWaitEvent(h->own_stream, h->fence_in, 0);
            st = h->own_stream;
            redirected = true;
        }
    }
    ~StreamScope() {
        if (redirected) {
            cudaEventRecord(h->fence_out, st);
            cudaStreamWaitEvent(user, h->fence_out, 0);
        }
    }
};

void drop_graphs(specdec_handle* h) {
    for (auto& g : h->graphs) cudaGraphExecDestroy(g.second.exec);
    h->graphs.clear();
}

// Runs `body` (a sequence of launches on `st`) through a cached CUDA graph: captured on first use,
// replayed afterwards.  The key must name everything the launches depend on besides device memory.
inline void graph_key_tail(const specdec_handle* h, std::vector<long long>& key) {
    for (long long v : {(long long)h->use_tc, (long long)h->use_tc_attn, (long long)h->want_lse, (long long)h->use_skinny,
                        (long long)h->use_pdl, (long long)h->use_ln_fuse, (long long)h->use_sk_cluster,
                        (long long)h->use_pair, (long long)h->diag_repeat, (long long)h->use_splitk, (long long)h->attn_stream, (long long)h->attn_stream_keys, (long long)h->attn_warps, (long long)h->attn_rs,
                        (long long)h->skinny_groups, (long long)h->want_trace,
                        (long long)(h->script_on ? 1 : 0), (long long)h->B, (long long)h->S_max, (long long)h->drafter_pc_session, (long long)(h->fuse_commit ? 1 : 0), (long long)h->enc_skinny})
        key.push_back(v);
}

template <typename F>
int graph_call(specdec_handle* h, std::vector<long long> key, cudaStream_t st, F body) {
    graph_key_tail(h, key);
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
        const long long before = h->launches;
        CUDA_TRY(h, cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
        int rc = body();
        cudaGraph_t g = nullptr;
        cudaError_t e = cudaStreamEndCapture(st, &g);
        if (rc != 0) { if (g) cudaGraphDestroy(g); return rc; }
        if (e != cudaSuccess || !g) return fail(h, SPECDEC_ERR_CUDA, std::string("graph capture: ") + cudaGetErrorString(e));
        cudaGraphExec_t ex = nullptr;
        e = cudaGraphInstantiate(&ex, g, 0);
        cudaGraphDestroy(g);
        if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
        if (h->graphs.size() > 256) drop_graphs(h);
        specdec_handle::GraphEntry ge{ex, h->launches - before};
        h->launches = before;
        it = h->graphs.emplace(std::move(key), ge).first;
    }
    CUDA_TRY(h, cudaGraphLaunch(it->second.exec, st));
    h->launches += it->second.kernels;
    return 0;
}

// One kernel in front of an IF node: the body runs only while a sequence is still decoding.
__global__ void k_gate(const int* __restrict__ counters, cudaGraphConditionalHandle cond) {
    if (threadIdx.x == 0) cudaGraphSetConditional(cond, counters[CNT_ACTIVE] > 0 ? 1u : 0u);
}

// A whole draft -> verify -> commit iteration as ONE graph whose launches sit in the body of a conditional node:
// the host can queue iterations ahead of the "unfinished sequences" counter it reads back (no bubble between
// iterations), and an iteration queued after the last sequence finished costs one tiny kernel instead of a full pass.
// Returns 1 (nothing launched) when such a graph cannot be built here; the caller then uses the plain graphs.
template <typename F>
int graph_call_gated(specdec_handle* h, std::vector<long long> key, cudaStream_t st, F body, long long* kernels_out) {
    graph_key_tail(h, key);
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
        const long long before = h->launches;
        cudaGraph_t g = nullptr, bg = nullptr;
        cudaGraphConditionalHandle cond;
        cudaGraphNode_t gate_node, if_node;
        auto give_up = [&](const char*) { if (g) cudaGraphDestroy(g); cudaGetLastError(); h->gate_ok = false; h->launches = before; return 1; };
        if (cudaGraphCreate(&g, 0) != cudaSuccess) return give_up("create");
        if (cudaGraphConditionalHandleCreate(&cond, g, 0, cudaGraphCondAssignDefault) != cudaSuccess) return give_up("handle");
        const int* counters = h->ses.counters;
        void* gate_args[] = {(void*)&counters, (void*)&cond};
        cudaKernelNodeParams kp{};
        kp.func = (void*)k_gate; kp.gridDim = dim3(1); kp.blockDim = dim3(32); kp.sharedMemBytes = 0; kp.kernelParams = gate_args;
        if (cudaGraphAddKernelNode(&gate_node, g, nullptr, 0, &kp) != cudaSuccess) return give_up("gate");
        cudaGraphNodeParams cp{};
        cp.type = cudaGraphNodeTypeConditional;
        cp.conditional.handle = cond; cp.conditional.type = cudaGraphCondTypeIf; cp.conditional.size = 1;
        if (cudaGraphAddNode(&if_node, g, &gate_node, 1, &cp) != cudaSuccess) return give_up("if node");
        bg = cp.conditional.phGraph_out[0];
        if (cudaStreamBeginCaptureToGraph(st, bg, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return give_up("capture");
        int rc = body();
        cudaGraph_t got = nullptr;
        cudaError_t e = cudaStreamEndCapture(st, &got);
        if (rc != 0) { cudaGraphDestroy(g); h->launches = before; return rc; }
        if (e != cudaSuccess) return give_up("end capture");
        cudaGraphExec_t ex = nullptr;
        if (cudaGraphInstantiate(&ex, g, 0) != cudaSuccess) return give_up("instantiate");
        cudaGraphDestroy(g);
        if (h->graphs.size() > 256) drop_graphs(h);
        specdec_handle::GraphEntry ge{ex, h->launches - before + 1};
        h->launches = before;
        it = h->graphs.emplace(std::move(key), ge).first;
    }
    CUDA_TRY(h, cudaGraphLaunch(it->second.exec, st));
    h->launches += it->second.kernels;
    *kernels_out = it->second.kernels;
    return 0;
}

// encode through a CUDA graph: the inputs are first copied into the handle's own staging buffers so that the
// captured launches never depend on the caller's pointers
template <typename T>
int encode_staged(specdec_handle* h, const int* d_src, const int* d_src_len, const int* d_max_tgt, int B, int S_max,
                  cudaStream_t st) {
    if (!h->use_graphs || h->profile) return encode_impl<T>(h, d_src, d_src_len, d_max_tgt, B, S_max, st);
    if (d_src != h->stage_src) CUDA_TRY(h, cudaMemcpyAsync(h->stage_src, d_src, (size_t)B * S_max * 4, cudaMemcpyDeviceToDevice, st));
    if (d_src_len != h->stage_len) CUDA_TRY(h, cudaMemcpyAsync(h->stage_len, d_src_len, (size_t)B * 4, cudaMemcpyDeviceToDevice, st));
    if (d_max_tgt && d_max_tgt != h->stage_mt) CUDA_TRY(h, cudaMemcpyAsync(h->stage_mt, d_max_tgt, (size_t)B * 4, cudaMemcpyDeviceToDevice, st));
    h->B = B; h->S_max = S_max;
    h->drafter_pc_session = h->drafter_pc;
    TRY(graph_call(h, {5, d_max_tgt ? 1 : 0}, st, [&]() {
        return encode_impl<T>(h, h->stage_src, h->stage_len, d_max_tgt ? h->stage_mt : nullptr, B, S_max, st); }));
    h->len_ub = 0; h->encoded = true; h->verified = false; h->drafted = false;
    h->dnew_ub = 1;
    return 0;
}

inline int len_bucket(const specdec_handle* h, int len_ub) { return std::min(h->T_cap, (len_ub + 31) / 32 * 32); }

template <typename T>
int generate_loop(specdec_handle* h, const int* d_src, const int* d_src_len, const int* d_max_tgt, int B, int S_max,
                  int k, int beta, float tau, int* d_out, int out_stride, int* d_out_len, specdec_stats* hs,
                  cudaStream_t st) {
    const bool timed = hs != nullptr, phases = timed && h->stats_timing;
    // the acceptance scan commits its own decision (one kernel less per iteration) unless the phases are timed apart
    struct FuseGuard { specdec_handle* h; ~FuseGuard() { h->fuse_commit = false; h->commit_done = false; } } fuse_guard{h};
    h->fuse_commit = !phases;
    size_t ev = 0;
    auto mark_always = [&]() { if (timed && ev < h->time_ev.size()) cudaEventRecord(h->time_ev[ev++], st); };
    auto mark = [&]() { if (phases) mark_always(); };
    mark_always();
    TRY(encode_staged<T>(h, d_src, d_src_len, d_max_tgt, B, S_max, st));
    mark_always();
    const int max_iters = h->T_cap;            // every iteration commits >= 1 token per unfinished sequence
    const bool graphs = h->use_graphs && !h->profile;
    // the conditional node costs more per iteration than the bubble it removes: worth it only where the host ran
    // ahead anyway (larger batches), to make the iterations queued after the last sequence finished free
    bool gated = graphs && h->gate_ok && !phases && (h->use_gate == 1 ? B > 4 : h->use_gate == 2);
    // how many iterations the host runs ahead of the "unfinished sequences" counter it reads back.  Plain graphs:
    // every iteration launched after the last sequence finished is wasted work, every wait for the counter is a
    // bubble.  Gated graphs: an iteration too many costs one small kernel, so the host always runs ahead.
    const int slots = (int)h->poll_ev.size();
    int lag = h->poll_lag >= 0 ? std::min(h->poll_lag, slots - 1) : (gated ? 2 : (B <= 4 ? 0 : 2));
    int it = 0, skipped = 0;
    long long skipped_kernels = 0;
    const bool flag = h->poll_flag != 0;
    if (flag && cudaStreamQuery(st) == cudaSuccess) h->commits_issued = (unsigned)(*(volatile unsigned long long*)h->h_post >> 32);
    const unsigned commits_base = h->commits_issued;
    std::vector<long long> it_kernels;
    int tau_bits; memcpy(&tau_bits, &tau, 4);
    // the drafter writes its block straight into the verifier's draft buffer: no copy between the two steps
    for (; it < max_iters; ++it) {
        if (graphs) {
            // the launches depend on the host-side length bound only through its 32-token bucket
            const int true_ub = h->len_ub, lb = len_bucket(h, true_ub);
            // (prefix-causal drafter: the pass is also sized by how many prefix positions its cache still lacks)
            const int dn = h->dnew_ub, dkey = (h->drafter_pc_session && k > 0) ? dn : -1;
            bool done = false;
            if (gated) {
                h->len_ub = lb;
                long long nk = 0;
                int rc = graph_call_gated(h, {3, k, lb, beta, tau_bits, dkey}, st, [&]() {
                    int r = k > 0 ? draft_impl<T>(h, k, h->v_draft, st) : 0;
                    h->len_ub = lb;
                    if (!r) r = verify_impl<T>(h, h->v_draft, k, beta, tau, nullptr, nullptr, st);
                    return r ? r : commit_impl(h, nullptr, nullptr, st);
                }, &nk);
                if (rc == 1) { gated = false; if (h->poll_lag < 0) lag = std::min(lag, B <= 4 ? 0 : 2); }
                else if (rc != 0) return rc;
                else { done = true; it_kernels.push_back(nk); }
            }
            if (!done && !phases) {
                // one graph per iteration: no graph-to-graph gap between the drafter and the verifier
                h->len_ub = lb;
                h->dnew_ub = dn;
                TRY(graph_call(h, {4, k, lb, beta, tau_bits, dkey}, st, [&]() {
                    int r = k > 0 ? draft_impl<T>(h, k, h->v_draft, st) : 0;
                    h->len_ub = lb;
                    if (!r) r = verify_impl<T>(h, h->v_draft, k, beta, tau, nullptr, nullptr, st);
                    return r ? r : commit_impl(h, nullptr, nullptr, st);
                }));
                it_kernels.push_back(0);
                done = true;
            }
            if (!done) {
                h->len_ub = lb;
                h->dnew_ub = dn;
                if (k > 0) TRY(graph_call(h, {1, k, lb, dkey}, st, [&]() { return draft_impl<T>(h, k, h->v_draft, st); }));
                mark();
                h->len_ub = lb;
                TRY(graph_call(h, {2, k, lb, beta, tau_bits}, st, [&]() {
                    int rc = verify_impl<T>(h, h->v_draft, k, beta, tau, nullptr, nullptr, st);
                    return rc ? rc : commit_impl(h, nullptr, nullptr, st);
                }));
                mark();
                it_kernels.push_back(0);
            }
            h->len_ub = std::min(true_ub + k + 1, h->T_cap);
            h->dnew_ub = std::min((k > 0 ? 0 : dn) + k + 1, h->T_cap + 1);      // (a replayed graph does not run the host code that counts)
            h->last_k = k; h->verified = false; h->drafted = false;
        } else {
            if (k > 0) TRY(draft_impl<T>(h, k, h->v_draft, st));
            mark();
            TRY(verify_impl<T>(h, h->v_draft, k, beta, tau, nullptr, nullptr, st));
            mark();
            TRY(commit_impl(h, nullptr, nullptr, st));
            it_kernels.push_back(0);
        }
        mark();
        int active_seen = 1;
        if (flag) {
            // spin on the word k_commit posts; a look at the stream now and then surfaces a failed launch
            if (it >= lag) {
                const unsigned want = commits_base + (unsigned)(it - lag + 1);
                const auto t0 = std::chrono::steady_clock::now();
                for (unsigned spins = 1;; ++spins) {
                    const unsigned long long v = *(volatile unsigned long long*)h->h_post;
                    if ((int)((unsigned)(v >> 32) - want) >= 0) { active_seen = (int)(unsigned)v; break; }
                    if ((spins & 0xfffu) == 0) {
                        cudaError_t q = cudaStreamQuery(st);
                        if (q != cudaSuccess && q != cudaErrorNotReady) return fail(h, SPECDEC_ERR_CUDA, std::string("generate: ") + cudaGetErrorString(q));
                        if (q == cudaSuccess) {       // the stream drained: the word must be there now
                            const unsigned long long v2 = *(volatile unsigned long long*)h->h_post;
                            if ((int)((unsigned)(v2 >> 32) - want) >= 0) { active_seen = (int)(unsigned)v2; break; }
                            // behind a gate no commit kernel runs once nothing is left to decode (for instance when
                            // every budget was zero from the start): ask the device
                            int active_now = -1;
                            CUDA_TRY(h, cudaMemcpyAsync(&active_now, h->ses.counters + CNT_ACTIVE, 4, cudaMemcpyDeviceToHost, st));
                            CUDA_TRY(h, cudaStreamSynchronize(st));
                            if (active_now == 0) { active_seen = 0; break; }
                            return fail(h, SPECDEC_ERR_CUDA, "generate: the commit kernel did not post its counter");
                        }
                        if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(60))
                            return fail(h, SPECDEC_ERR_TIMEOUT, "generate: no commit within 60 s");
                    }
                }
            }
        } else {
            CUDA_TRY(h, cudaMemcpyAsync(h->h_poll + (it % slots), h->ses.counters + CNT_ACTIVE, 4, cudaMemcpyDeviceToHost, st));
            CUDA_TRY(h, cudaEventRecord(h->poll_ev[it % slots], st));
            if (it >= lag) {
                CUDA_TRY(h, cudaEventSynchronize(h->poll_ev[(it - lag) % slots]));
                active_seen = h->h_poll[(it - lag) % slots];
            }
        }
        if (it >= lag) {
            if (active_seen == 0) {
                // iterations it - lag + 1 .. it found nothing to do: behind a gate only the gate kernel ran
                for (int j = it - lag + 1; j <= it; ++j)
                    if (it_kernels[j] > 0) { ++skipped; skipped_kernels += it_kernels[j] - 1; }
                ++it;
                break;
            }
        }
    }
    h->launches -= skipped_kernels;
    if (d_out || d_out_len) TRY(specdec_get_output(h, d_out, out_stride, d_out_len, nullptr, st));
    CUDA_TRY(h, cudaMemcpyAsync(h->h_stats, h->ses.stats, 32, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(h, cudaMemcpyAsync(h->h_stats + 4, h->ses.counters + 7, 4, cudaMemcpyDeviceToHost, st));
    mark_always();
    CUDA_TRY(h, cudaStreamSynchronize(st));
    h->commits_issued = (unsigned)(*(volatile unsigned long long*)h->h_post >> 32);    // gated iterations that found nothing to do posted nothing
    if (h->profile) prof_collect(h);
    if (*(int*)(h->h_stats + 4) != 0)
        return fail(h, SPECDEC_ERR_TIMEOUT, "generate: a bounded device-side wait gave up (code " + std::to_string(*(int*)(h->h_stats + 4)) + ")");
    if (hs) {
        memset(hs, 0, sizeof(*hs));
        hs->iterations = it - skipped;
        hs->seq_iterations = (long long)h->h_stats[0];
        hs->drafted = (long long)h->h_stats[1];
        hs->accepted = (long long)h->h_stats[2];
        hs->emitted = (long long)h->h_stats[3];
        auto ms = [&](size_t a, size_t b) { float t = 0.f; if (b < ev) cudaEventElapsedTime(&t, h->time_ev[a], h->time_ev[b]); return (double)t; };
        hs->ms_encode = ms(0, 1);
        for (int i = 0; i < it && phases; ++i) {
            size_t b0 = 1 + (size_t)i * 3;
            hs->ms_draft += ms(b0, b0 + 1);
            hs->ms_verify += ms(b0 + 1, b0 + 2);
            hs->ms_commit += ms(b0 + 2, b0 + 3);
        }
        hs->ms_total = ms(0, ev - 1);
    }
    return 0;
}

template <typename T>
int generate_impl(specdec_handle* h, const int* d_src, const int* d_src_len, const int* d_max_tgt, int B, int S_max,
                  int k, int beta, float tau, int* d_out, int out_stride, int* d_out_len, specdec_stats* hs,
                  cudaStream_t st) {
    TRY(errw_check(h, st, "generate"));
    const int rc = generate_loop<T>(h, d_src, d_src_len, d_max_tgt, B, S_max, k, beta, tau, d_out, out_stride, d_out_len, hs, st);
    if (rc != 0) {
        // leave the handle usable: drain the stream, take the commit count from what was really posted, and clear the
        // error word now that it has been reported
        const std::string msg = h->err;
        cudaStreamSynchronize(st);
        cudaGetLastError();
        h->commits_issued = (unsigned)(*(volatile unsigned long long*)h->h_post >> 32);
        cudaMemsetAsync(h->ses.counters + 7, 0, 4, st);
        h->h_poll[ERRW_SLOT] = 0; h->errw_pending = false;
        h->encoded = false; h->verified = false; h->drafted = false;
        h->err = msg;
    }
    return rc;
}

int check_model(const specdec_model_dims& m, const char* who, std::string& why) {
    if (m.d_model <= 0 || m.n_heads <= 0 || m.d_ffn <= 0 || m.vocab <= 0 || m.enc_layers < 0 || m.dec_layers < 1 ||
        m.max_pos <= 0) { why = std::string(who) + ": non-positive dimension"; return -1; }
    if (m.d_model % m.n_heads) { why = std::string(who) + ": d_model not divisible by n_heads"; return -1; }
    if (m.d_model % 16 || m.d_ffn % 16) { why = std::string(who) + ": d_model and d_ffn must be multiples of 16"; return -1; }
    return 0;
}

}  // namespace

// ================================================================== C ABI
// Red zones and non-finite scan on `st`; synchronises.  Returns SPECDEC_OK with the report filled in.
int integrity_run(specdec_handle* h, cudaStream_t st, specdec_integrity* rep) {
    const unsigned long long init[4] = {0ull, ~0ull, 0ull, ~0ull};
    CUDA_TRY(h, cudaMemcpyAsync(h->integ_report, init, sizeof(init), cudaMemcpyHostToDevice, st));
    k_red_check<<<cdiv(h->n_zones, 8), 256, 0, st>>>((const unsigned char*)h->arena.base, h->zone_tab, h->n_zones, h->integ_report);
    if (h->n_scan > 0) k_nonfinite_scan<<<dim3(2 * h->tma.n_sm, h->n_scan), 256, 0, st>>>(h->integ_bufs, h->integ_report);
    KCHECK(h);
    unsigned long long out[4];
    CUDA_TRY(h, cudaMemcpyAsync(out, h->integ_report, sizeof(out), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(h, cudaStreamSynchronize(st));
    rep->zones = h->n_zones;
    rep->damaged_zones = (int)out[0];
    rep->first_damaged_zone = out[0] ? (int)out[1] : -1;
    rep->nonfinite = (long long)out[2];
    rep->first_nonfinite_buffer = out[2] ? (int)out[3] : -1;
    return SPECDEC_OK;
}

// A named range around every public step call, for timeline tools (header-only NVTX: no cost without a tool attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

// With option "debug_checks" every step call ends with the integrity check and fails when it finds something.
int post_check(specdec_handle* h, int rc, void* stream) {
    if (rc != SPECDEC_OK || !h || !h->debug_checks) return rc;
    specdec_integrity rep;
    TRY(integrity_run(h, (cudaStream_t)stream, &rep));
    if (rep.damaged_zones)
        return fail(h, SPECDEC_ERR_CORRUPT, "integrity: " + std::to_string(rep.damaged_zones) + " damaged red zone(s), first behind arena block " +
                                                std::to_string(rep.first_damaged_zone));
    if (rep.nonfinite)
        return fail(h, SPECDEC_ERR_CORRUPT, "integrity: " + std::to_string(rep.nonfinite) + " non-finite value(s), first in " +
                                                h->scan_names[rep.first_nonfinite_buffer]);
    return SPECDEC_OK;
}

extern "C" {

const char* specdec_last_error(const specdec_handle* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

long long specdec_launch_count(const specdec_handle* h) { return h ? h->launches : 0; }

int specdec_create(const specdec_config* cfg, const specdec_tensor* weights, int n_weights, void* stream,
                   specdec_handle** out) {
    if (out) *out = nullptr;
    if (!cfg || !weights || !out || n_weights <= 0) return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "null argument");
    std::string why;
    if (check_model(cfg->verifier, "verifier", why) || check_model(cfg->drafter, "drafter", why))
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, why);
    if (cfg->k_max < 1 || cfg->max_batch < 1 || cfg->max_src < 1 || cfg->max_tgt < 1)
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "k_max, max_batch, max_src, max_tgt must be >= 1");
    if (cfg->page_tokens < 1 || (cfg->page_tokens & (cfg->page_tokens - 1)))
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "page_tokens must be a power of two");
    if (cfg->compute_dtype != SPECDEC_DTYPE_F32 && cfg->compute_dtype != SPECDEC_DTYPE_BF16)
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "compute_dtype must be 0 (fp32) or 1 (bf16)");
    if (cfg->ffn_activation != SPECDEC_ACT_RELU && cfg->ffn_activation != SPECDEC_ACT_GELU)
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "ffn_activation must be 0 (ReLU) or 1 (GELU)");
    if (cfg->verifier.vocab != cfg->drafter.vocab)
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "verifier and drafter must share the vocabulary");
    const int need_pos = cfg->max_tgt + cfg->k_max + 1;
    if (cfg->verifier.max_pos < need_pos || cfg->drafter.max_pos < need_pos || cfg->verifier.max_pos < cfg->max_src ||
        cfg->drafter.max_pos < cfg->max_src)
        return fail(nullptr, SPECDEC_ERR_CAPACITY, "max_pos must cover max_src and max_tgt + k_max + 1");
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
        return fail(nullptr, SPECDEC_ERR_CUDA, "no CUDA device: this library has no CPU path");
    cudaStream_t st = (cudaStream_t)stream;
    specdec_handle* h = new specdec_handle();
    h->cfg = *cfg;
    h->dtype = cfg->compute_dtype;
    h->esz = h->dtype == SPECDEC_DTYPE_BF16 ? 2 : 4;
    h->B_cap = cfg->max_batch; h->S_cap = cfg->max_src; h->T_cap = cfg->max_tgt; h->k_cap = cfg->k_max;
    h->d_max = std::max(cfg->verifier.d_model, cfg->drafter.d_model);
    h->f_max = std::max(cfg->verifier.d_ffn, cfg->drafter.d_ffn);
    h->v_max = cfg->verifier.vocab;
    h->M_cap = h->B_cap * (h->k_cap + 1);
    h->R2_cap = h->B_cap * h->k_cap;
    h->R_cap = std::max(std::max(h->B_cap * h->S_cap, h->B_cap * (h->T_cap + 1 + h->k_cap)), h->M_cap);
    h->pages_per_seq = cdiv(h->T_cap + h->k_cap + 1, cfg->page_tokens);
    // partial row statistics per vocabulary tile: 64-column tiles on the SIMT path, two column halves per 128- to 256-wide
    // tile on the tensor-core path (2 * ceil(V / 128) exceeds ceil(V / 64) when V mod 128 is in 1..64)
    h->n_tiles_cap = std::max(cdiv(h->v_max, 64), 2 * cdiv(h->v_max, 128));
    layout_all(h);                       // dry runs: the number of red zones, then the sizes
    h->zone_cap = (int)h->arena.zones.size();
    layout_all(h);
    const size_t total = h->arena.off + 256;
    char* base = nullptr;
    cudaError_t ce = cudaMalloc((void**)&base, total);
    if (ce != cudaSuccess) {
        std::string msg = std::string("arena allocation of ") + std::to_string(total) + " bytes: " + cudaGetErrorString(ce);
        delete h;
        return fail(nullptr, SPECDEC_ERR_CUDA, msg);
    }
    h->arena.base = base;
    layout_all(h);
    cudaMemsetAsync(base, 0, total, st);          // dead rows of every buffer read as zeros, never as NaN patterns
    {   // red zones behind every block, and the table of buffers the non-finite scan walks
        h->n_zones = (int)h->arena.zones.size();
        cudaMemcpyAsync(h->zone_tab, h->arena.zones.data(), (size_t)h->n_zones * 8, cudaMemcpyHostToDevice, st);
        k_red_fill<<<cdiv(h->n_zones, 8), 256, 0, st>>>((unsigned char*)base, h->zone_tab, h->n_zones);
        std::vector<ScanBuf> sb;
        auto add = [&](const char* name, const void* p, size_t bytes, bool f32) {
            if (!p || bytes < 16 || sb.size() >= 128) return;
            sb.push_back(ScanBuf{p, (unsigned long long)(bytes / 16), f32 ? 1 : 0, 0});
            h->scan_names.push_back(name);
        };
        const size_t e = h->esz, R = h->R_cap, d = h->d_max, f = h->f_max, Re = (size_t)h->B_cap * h->S_cap;
        const bool f32 = h->dtype != SPECDEC_DTYPE_BF16;
        add("residual rows x", h->ws[0].x, R * d * 4, true); add("mask rows x2", h->x2, (size_t)h->R2_cap * d * 4, true);
        add("normalised rows y", h->ws[0].y, R * d * e, f32); add("qkv rows", h->ws[0].qkv, R * 3 * d * e, f32);
        add("attention output", h->ws[0].att, R * d * e, f32); add("cross query rows", h->ws[0].q, R * d * e, f32);
        add("feed-forward rows", h->ws[0].hbuf, R * f * e, f32); add("encoder memory", h->ws[0].mem, Re * d * e, f32);
        add("second encoder x", h->ws[1].x, Re * d * 4, true); add("second encoder y", h->ws[1].y, Re * d * e, f32);
        add("second encoder qkv", h->ws[1].qkv, Re * 3 * d * e, f32); add("second encoder attention output", h->ws[1].att, Re * d * e, f32);
        add("second encoder feed-forward rows", h->ws[1].hbuf, Re * f * e, f32); add("second encoder memory", h->ws[1].mem, Re * d * e, f32);
        const size_t cache_rows = (size_t)h->B_cap * h->pages_per_seq * h->cfg.page_tokens;
        for (auto p : h->kc) add("verifier K cache", p, cache_rows * h->cfg.verifier.d_model * e, f32);
        for (auto p : h->vc) add("verifier V cache", p, cache_rows * h->cfg.verifier.d_model * e, f32);
        for (auto p : h->dkc) add("drafter K cache", p, cache_rows * h->cfg.drafter.d_model * e, f32);
        for (auto p : h->dvc) add("drafter V cache", p, cache_rows * h->cfg.drafter.d_model * e, f32);
        add("verifier cross K/V", h->ver.ckv.empty() ? nullptr : h->ver.ckv[0], Re * h->ver.ckv_stride * e, f32);
        add("drafter cross K/V", h->dra.ckv.empty() ? nullptr : h->dra.ckv[0], Re * h->dra.ckv_stride * e, f32);
        h->n_scan = (int)sb.size();
        cudaMemcpyAsync(h->integ_bufs, sb.data(), sb.size() * sizeof(ScanBuf), cudaMemcpyHostToDevice, st);
        cudaStreamSynchronize(st);               // the host vectors go out of scope
    }
    auto bail = [&](int code, const std::string& msg) { cudaFree(base); delete h; return fail(nullptr, code, msg); };
    Manifest mf;
    for (int i = 0; i < n_weights; ++i)
        if (weights[i].name) mf.map[weights[i].name] = &weights[i];
    if (h->dtype == SPECDEC_DTYPE_BF16) {
        load_model<bf16>(h, h->ver, "verifier.", mf, st);
        load_model<bf16>(h, h->dra, "drafter.", mf, st);
    } else {
        load_model<float>(h, h->ver, "verifier.", mf, st);
        load_model<float>(h, h->dra, "drafter.", mf, st);
    }
    if (!mf.missing.empty()) { cudaStreamSynchronize(st); return bail(SPECDEC_ERR_SHAPE, "missing weight: " + mf.missing); }
    if (!mf.bad.empty()) { cudaStreamSynchronize(st); return bail(SPECDEC_ERR_SHAPE, "weight with wrong dtype/shape: " + mf.bad); }
    // page table: sequence b owns pages {i * B_cap + b}: interleaved, so the indirection is exercised
    {
        std::vector<int> pt((size_t)h->B_cap * h->pages_per_seq);
        for (int b = 0; b < h->B_cap; ++b)
            for (int i = 0; i < h->pages_per_seq; ++i) pt[(size_t)b * h->pages_per_seq + i] = i * h->B_cap + b;
        ce = cudaMemcpyAsync(h->page_table, pt.data(), pt.size() * 4, cudaMemcpyHostToDevice, st);
        if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
        if (ce != cudaSuccess) return bail(SPECDEC_ERR_CUDA, std::string("page table upload: ") + cudaGetErrorString(ce));
    }
    ce = cudaStreamSynchronize(st);
    if (ce == cudaSuccess) ce = cudaGetLastError();
    if (ce != cudaSuccess) return bail(SPECDEC_ERR_CUDA, std::string("weight repacking: ") + cudaGetErrorString(ce));
    if (cudaMallocHost((void**)&h->h_post, 64) != cudaSuccess) return bail(SPECDEC_ERR_CUDA, "pinned host allocation failed");
    *h->h_post = 0ull;
    if (cudaMallocHost((void**)&h->h_poll, 64 * 4) != cudaSuccess || cudaMallocHost((void**)&h->h_stats, 64) != cudaSuccess)
        return bail(SPECDEC_ERR_CUDA, "pinned host allocation failed");
    cudaStreamCreateWithFlags(&h->own_stream, cudaStreamNonBlocking);
    cudaStreamCreateWithFlags(&h->enc_stream, cudaStreamNonBlocking);
    cudaEventCreateWithFlags(&h->enc_fork, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&h->enc_join, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&h->fence_in, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&h->fence_out, cudaEventDisableTiming);
    cudaEventCreateWithFlags(&h->errw_ev, cudaEventDisableTiming);
    memset(h->h_poll, 0, 64 * 4);
    h->poll_ev.resize(8);
    for (auto& e : h->poll_ev) cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
    h->time_ev.resize((size_t)3 * h->T_cap + 8);
    for (auto& e : h->time_ev) cudaEventCreate(&e);
    // attention keeps one row of scores per warp in shared memory
    {
        const int max_keys = std::max(h->S_cap, h->T_cap + h->k_cap + 1);
        const int dh = std::max(cfg->verifier.d_model / cfg->verifier.n_heads, cfg->drafter.d_model / cfg->drafter.n_heads);
        const int smem = 4 * (max_keys + dh) * 4;
        if (smem > 200 * 1024) return bail(SPECDEC_ERR_CAPACITY, "max_src / max_tgt too large for the attention kernel");
        if (smem > 48 * 1024) {
            if (h->dtype == SPECDEC_DTYPE_BF16) {
                cudaFuncSetAttribute(k_attention<bf16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
                cudaFuncSetAttribute(k_attention<bf16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            } else {
                cudaFuncSetAttribute(k_attention<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
                cudaFuncSetAttribute(k_attention<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            }
        }
    }
    if (h->dtype == SPECDEC_DTYPE_BF16) {
        const int max_keys = std::max(h->S_cap, h->T_cap + h->k_cap + 1);
        h->attn_tc_smem_cap = std::min<size_t>(attn_tc_smem(max_keys), 227 * 1024);
        cudaFuncSetAttribute(k_attn_stream<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, ats_smem(4));
        cudaFuncSetAttribute(k_attn_stream<false, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, ats_smem(4));
        if (cudaFuncSetAttribute(k_attn_tc<true, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<false, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<false, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<true, 8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<false, 8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<true, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess ||
            cudaFuncSetAttribute(k_attn_tc<false, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->attn_tc_smem_cap) != cudaSuccess) {
            cudaGetLastError();
            h->attn_tc_smem_cap = 48 * 1024;
        }
        {
            const int kmax = std::max(h->d_max, h->f_max);
            size_t need = std::min<size_t>(skinny_smem(2, kmax), 227 * 1024);
            cudaError_t e = skinny_attr_mt<EPI_STORE>((int)need);
            if (e == cudaSuccess) e = skinny_attr_mt<EPI_GELU>((int)need);
            if (e == cudaSuccess) e = skinny_attr_mt<EPI_RELU>((int)need);
            if (e == cudaSuccess) e = skinny_attr_mt<EPI_RESID>((int)need);
            if (e == cudaSuccess) e = skinny_attr_mt<EPI_QKV>((int)need);
            if (e != cudaSuccess) { cudaGetLastError(); need = 48 * 1024; }
            h->skinny_smem_cap = need;
        }
        if (sd::tc_init(h->tma, h->ses.counters + 7) != 0) h->use_tc = 0;     // reported through specdec_last_error; SIMT GEMM still runs on the GPU
        h->splitk_ready = h->use_tc && sd::spk_init() == cudaSuccess;
        if (!h->splitk_ready) cudaGetLastError();
        h->pair_ready = h->use_tc && sd::tc_pair_init() == cudaSuccess;
        if (!h->pair_ready) cudaGetLastError();
        if (!h->use_tc) h->err = "tensor-core GEMM unavailable: " + h->tma.err;
    } else {
        h->use_tc = 0;
    }
    *out = h;
    return SPECDEC_OK;
}

int specdec_destroy(specdec_handle* h) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    drop_graphs(h);
    if (h->own_stream) cudaStreamDestroy(h->own_stream);
    if (h->enc_stream) cudaStreamDestroy(h->enc_stream);
    if (h->enc_fork) cudaEventDestroy(h->enc_fork);
    if (h->enc_join) cudaEventDestroy(h->enc_join);
    if (h->fence_in) cudaEventDestroy(h->fence_in);
    if (h->fence_out) cudaEventDestroy(h->fence_out);
    if (h->errw_ev) cudaEventDestroy(h->errw_ev);
    for (auto& e : h->poll_ev) cudaEventDestroy(e);
    for (auto& e : h->time_ev) cudaEventDestroy(e);
    for (auto& e : h->prof_ev) cudaEventDestroy(e);
    if (h->h_poll) cudaFreeHost(h->h_poll);
    if (h->h_post) cudaFreeHost(h->h_post);
    if (h->h_stats) cudaFreeHost(h->h_stats);
    if (h->arena.base) cudaFree(h->arena.base);
    delete h;
    return SPECDEC_OK;
}

int specdec_set_option(specdec_handle* h, const char* name, int value) {
    if (!h || !name) return SPECDEC_ERR_INVALID_ARG;
    drop_graphs(h);
    if (!strcmp(name, "gemm")) {
        if (value && (h->dtype != SPECDEC_DTYPE_BF16 || !h->tma.ready))
            return fail(h, SPECDEC_ERR_UNSUPPORTED, "tensor-core GEMM needs a bf16 handle on an sm_100 device");
        h->use_tc = value ? 1 : 0;
        return SPECDEC_OK;
    }
    if (!strcmp(name, "trace")) { h->want_trace = value; return SPECDEC_OK; }   // 10 + e: stamp the tensor-core GEMM with epilogue e instead of the vocabulary one
    if (!strcmp(name, "inject_error")) {
        // test hook: the error word reads as if a bounded device-side wait had given up; nothing waits, nothing faults
        CUDA_TRY(h, cudaDeviceSynchronize());
        CUDA_TRY(h, cudaMemcpy(h->ses.counters + 7, &value, 4, cudaMemcpyHostToDevice));
        h->h_poll[ERRW_SLOT] = value; h->errw_pending = false;
        return SPECDEC_OK;
    }
    if (!strcmp(name, "drafter_prefix_causal")) { h->drafter_pc = value ? 1 : 0; return SPECDEC_OK; }   // latched by the next specdec_encode
    if (!strcmp(name, "poll_lag")) { h->poll_lag = value; return SPECDEC_OK; }
    if (!strcmp(name, "stats_timing")) { h->stats_timing = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "poll_flag")) { h->poll_flag = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "gate")) { h->use_gate = value; return SPECDEC_OK; }
    if (!strcmp(name, "tc_bn")) { h->tma.force_bn = value; return SPECDEC_OK; }
    if (!strcmp(name, "sk_cluster")) { h->use_sk_cluster = value < 0 ? 0 : value; return SPECDEC_OK; }   // 0 off, 1 LayerNorm-fused kernels, 2 + plain ones with K <= 512, 3 all
    if (!strcmp(name, "ln_fuse")) { h->use_ln_fuse = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "enc_skinny")) { h->enc_skinny = value < 0 ? 0 : (value > 2 ? 2 : value); return SPECDEC_OK; }
    if (!strcmp(name, "debug_checks")) { h->debug_checks = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "poke_zone")) {                 // test hook: damage red zone `value` (an in-arena write from the host)
        if (value < 0 || value >= h->n_zones) return fail(h, SPECDEC_ERR_INVALID_ARG, "poke_zone: no such red zone");
        const unsigned int junk = 0xDEADBEEFu;
        CUDA_TRY(h, cudaMemcpy(h->arena.base + h->arena.zones[value] + 100, &junk, 4, cudaMemcpyHostToDevice));
        return SPECDEC_OK;
    }
    if (!strcmp(name, "heal_zones")) {                // test hook: restore every red zone
        k_red_fill<<<cdiv(h->n_zones, 8), 256>>>((unsigned char*)h->arena.base, h->zone_tab, h->n_zones);
        CUDA_TRY(h, cudaDeviceSynchronize());
        return SPECDEC_OK;
    }
    if (!strcmp(name, "poke_nan")) {                  // test hook: a NaN (1) or a zero (0) in the last element of the attention-output buffer (a row no pass reaches)
        const unsigned int word = value ? 0x7FC00000u : 0u;      // bf16: the upper half is the last element
        char* end = (char*)h->ws[0].att + (size_t)h->R_cap * h->d_max * h->esz;
        CUDA_TRY(h, cudaMemcpy(end - 4, &word, 4, cudaMemcpyHostToDevice));
        return SPECDEC_OK;
    }
    if (!strcmp(name, "pair")) {
        if (value && !h->pair_ready) return fail(h, SPECDEC_ERR_UNSUPPORTED, "two-SM GEMM tiles are not available on this handle");
        h->use_pair = value ? 1 : 0; return SPECDEC_OK;
    }
    if (!strcmp(name, "diag_repeat")) { h->diag_repeat = value; return SPECDEC_OK; }
    if (!strcmp(name, "splitk")) { h->use_splitk = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "attn_stream")) { h->attn_stream = value < 0 ? 0 : (value > 3 ? 3 : value); return SPECDEC_OK; }
    if (!strcmp(name, "attn_stream_keys")) { h->attn_stream_keys = value; return SPECDEC_OK; }
    if (!strcmp(name, "attn_rs")) { h->attn_rs = value < 0 ? 0 : (value > 2 ? 2 : value); return SPECDEC_OK; }   // 0 never, 1 choose, 2 whenever possible
    if (!strcmp(name, "attn_warps")) {
        if (value != 0 && value != 4 && value != 8) return fail(h, SPECDEC_ERR_INVALID_ARG, "attn_warps must be 0, 4 or 8");
        h->attn_warps = value; return SPECDEC_OK;
    }
    if (!strcmp(name, "pdl")) { h->use_pdl = value ? 1 : 0; h->tma.pdl = value != 0; return SPECDEC_OK; }
    if (!strcmp(name, "skinny")) { h->use_skinny = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "row_lse")) { h->want_lse = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "attn")) { h->use_tc_attn = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "graphs")) { h->use_graphs = value ? 1 : 0; return SPECDEC_OK; }
    if (!strcmp(name, "profile")) { h->profile = value ? 1 : 0; h->prof_n = 0; h->prof_ms = 0.0; h->prof_launches = 0; return SPECDEC_OK; }
    return fail(h, SPECDEC_ERR_INVALID_ARG, std::string("unknown option: ") + name);
}

#define DISPATCH(h, call_bf16, call_f32) ((h)->dtype == SPECDEC_DTYPE_BF16 ? (call_bf16) : (call_f32))

static int encode_entry(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len, const int32_t* d_max_tgt, int B,
                        int S_max, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!d_src || !d_src_len || B < 1 || S_max < 1) return fail(h, SPECDEC_ERR_INVALID_ARG, "encode: bad argument");
    if (B > h->B_cap || S_max > h->S_cap) return fail(h, SPECDEC_ERR_CAPACITY, "encode: B or S_max beyond capacity");
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    TRY(errw_check(h, st, "encode"));
    return DISPATCH(h, encode_staged<bf16>(h, d_src, d_src_len, d_max_tgt, B, S_max, st),
                    encode_staged<float>(h, d_src, d_src_len, d_max_tgt, B, S_max, st));
}

static int draft_entry(specdec_handle* h, int k, int32_t* d_draft, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!h->encoded) return fail(h, SPECDEC_ERR_NOT_ENCODED, "draft: no session (call specdec_encode)");
    if (!d_draft) return fail(h, SPECDEC_ERR_INVALID_ARG, "draft: null output");
    if (k < 1 || k > h->k_cap) return fail(h, SPECDEC_ERR_CAPACITY, "draft: k outside [1, k_max]");
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    TRY(errw_check(h, st, "draft"));
    if (h->use_graphs && !h->profile) {
        const int true_ub = h->len_ub, lb = len_bucket(h, true_ub);
        h->len_ub = lb;
        const int dn = h->dnew_ub;
        int rc = graph_call(h, {3, k, lb, (long long)(intptr_t)d_draft, h->drafter_pc_session ? dn : -1}, st, [&]() {
            return DISPATCH(h, draft_impl<bf16>(h, k, d_draft, st), draft_impl<float>(h, k, d_draft, st)); });
        h->len_ub = true_ub;
        h->dnew_ub = 0;
        h->drafted = true; h->verified = false; h->last_draft_rows_ub = h->B * k;
        return rc;
    }
    return DISPATCH(h, draft_impl<bf16>(h, k, d_draft, st), draft_impl<float>(h, k, d_draft, st));
}

static int verify_entry(specdec_handle* h, const int32_t* d_draft, int k, int beta, float tau, int32_t* d_accepted,
                   int32_t* d_bif, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!h->encoded) return fail(h, SPECDEC_ERR_NOT_ENCODED, "verify: no session (call specdec_encode)");
    if (!d_draft && k > 0) return fail(h, SPECDEC_ERR_INVALID_ARG, "verify: null drafts");
    if (k < 0 || k > h->k_cap) return fail(h, SPECDEC_ERR_CAPACITY, "verify: k outside [0, k_max]");
    if (beta < 1 || !(tau >= 0.f)) return fail(h, SPECDEC_ERR_INVALID_ARG, "verify: beta >= 1 and tau >= 0 required");
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    TRY(errw_check(h, st, "verify"));
    if (h->use_graphs && !h->profile) {
        const int true_ub = h->len_ub, lb = len_bucket(h, true_ub);
        int tau_bits; memcpy(&tau_bits, &tau, 4);
        h->len_ub = lb;
        int rc = graph_call(h, {4, k, lb, beta, tau_bits, (long long)(intptr_t)d_draft, (long long)(intptr_t)d_accepted,
                                (long long)(intptr_t)d_bif}, st, [&]() {
            return DISPATCH(h, verify_impl<bf16>(h, d_draft, k, beta, tau, d_accepted, d_bif, st),
                            verify_impl<float>(h, d_draft, k, beta, tau, d_accepted, d_bif, st)); });
        h->len_ub = true_ub;
        h->last_k = k; h->verified = true; h->drafted = false;
        return rc;
    }
    return DISPATCH(h, verify_impl<bf16>(h, d_draft, k, beta, tau, d_accepted, d_bif, st),
                    verify_impl<float>(h, d_draft, k, beta, tau, d_accepted, d_bif, st));
}

static int commit_entry(specdec_handle* h, const int32_t* d_keep, const int32_t* d_next, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!h->encoded) return fail(h, SPECDEC_ERR_NOT_ENCODED, "commit: no session (call specdec_encode)");
    if (!h->verified) return fail(h, SPECDEC_ERR_INVALID_ARG, "commit: must follow specdec_verify");
    StreamScope scope(h, stream);
    TRY(errw_check(h, scope.st, "commit"));
    int rc = commit_impl(h, d_keep, d_next, scope.st);
    if (rc == 0) { ++h->commits_issued; errw_fetch(h, scope.st); }
    return rc;
}

int specdec_get_output(specdec_handle* h, int32_t* d_out, int out_stride, int32_t* d_out_len, int32_t* d_finished,
                       void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!h->B) return fail(h, SPECDEC_ERR_NOT_ENCODED, "get_output: no session");
    if (d_out && out_stride < 1) return fail(h, SPECDEC_ERR_INVALID_ARG, "get_output: out_stride < 1");
    StreamScope scope(h, stream);
    k_copy_out<<<h->B, 128, 0, scope.st>>>(h->ses, h->B, d_out, out_stride, d_out_len, d_finished);
    KCHECK(h);
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(scope.st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusNone) errw_fetch(h, scope.st);
    return SPECDEC_OK;
}

static int generate_entry(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len, const int32_t* d_max_tgt, int B,
                     int S_max, int k, int beta, float tau, int32_t* d_out, int out_stride, int32_t* d_out_len,
                     specdec_stats* h_stats, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!d_src || !d_src_len || !d_out || !d_out_len || B < 1 || S_max < 1 || out_stride < 1)
        return fail(h, SPECDEC_ERR_INVALID_ARG, "generate: bad argument");
    if (B > h->B_cap || S_max > h->S_cap) return fail(h, SPECDEC_ERR_CAPACITY, "generate: B or S_max beyond capacity");
    if (k < 0 || k > h->k_cap) return fail(h, SPECDEC_ERR_CAPACITY, "generate: k outside [0, k_max]");
    if (beta < 1 || !(tau >= 0.f)) return fail(h, SPECDEC_ERR_INVALID_ARG, "generate: beta >= 1 and tau >= 0 required");
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    int rc = DISPATCH(h, generate_impl<bf16>(h, d_src, d_src_len, d_max_tgt, B, S_max, k, beta, tau, d_out, out_stride, d_out_len, h_stats, st),
                      generate_impl<float>(h, d_src, d_src_len, d_max_tgt, B, S_max, k, beta, tau, d_out, out_stride, d_out_len, h_stats, st));
    if (h_stats) h_stats->status = rc;
    return rc;
}

static int generate_host_entry(specdec_handle* h, const int32_t* h_src, const int32_t* h_src_len, const int32_t* h_max_tgt,
                          int B, int S_max, int k, int beta, float tau, int32_t* h_out, int out_stride,
                          int32_t* h_out_len, specdec_stats* h_stats, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!h_src || !h_src_len || !h_out || !h_out_len || B < 1 || S_max < 1 || out_stride < 1)
        return fail(h, SPECDEC_ERR_INVALID_ARG, "generate_host: bad argument");
    if (B > h->B_cap || S_max > h->S_cap) return fail(h, SPECDEC_ERR_CAPACITY, "generate_host: B or S_max beyond capacity");
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    int *s_src = h->stage_src, *s_len = h->stage_len, *s_mt = h->stage_mt;
    CUDA_TRY(h, cudaMemcpyAsync(s_src, h_src, (size_t)B * S_max * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(h, cudaMemcpyAsync(s_len, h_src_len, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    if (h_max_tgt) CUDA_TRY(h, cudaMemcpyAsync(s_mt, h_max_tgt, (size_t)B * 4, cudaMemcpyHostToDevice, st));
    if (k < 0 || k > h->k_cap) return fail(h, SPECDEC_ERR_CAPACITY, "generate_host: k outside [0, k_max]");
    if (beta < 1 || !(tau >= 0.f)) return fail(h, SPECDEC_ERR_INVALID_ARG, "generate_host: beta >= 1 and tau >= 0 required");
    // the ids and lengths are read straight from the session arrays afterwards
    const int* mt = h_max_tgt ? s_mt : nullptr;
    int rc = DISPATCH(h, generate_impl<bf16>(h, s_src, s_len, mt, B, S_max, k, beta, tau, nullptr, 1, nullptr, h_stats, st),
                      generate_impl<float>(h, s_src, s_len, mt, B, S_max, k, beta, tau, nullptr, 1, nullptr, h_stats, st));
    if (h_stats) h_stats->status = rc;
    if (rc != 0) return rc;
    const int w = std::min(out_stride, h->ses.out_stride);
    CUDA_TRY(h, cudaMemcpy2DAsync(h_out, (size_t)out_stride * 4, h->ses.out, (size_t)h->ses.out_stride * 4, (size_t)w * 4,
                                  B, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(h, cudaMemcpyAsync(h_out_len, h->ses.len, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(h, cudaStreamSynchronize(st));
    return SPECDEC_OK;
}

int specdec_set_draft_script(specdec_handle* h, const int32_t* d_script, int B, int stride, void* stream) {
    if (!h) return SPECDEC_ERR_INVALID_ARG;
    if (!d_script) { h->script_on = false; return SPECDEC_OK; }
    if (B < 1 || B > h->B_cap || stride < 1) return fail(h, SPECDEC_ERR_CAPACITY, "set_draft_script: bad B or stride");
    StreamScope scope(h, stream);
    const int w = std::min(stride, h->T_cap + h->k_cap);
    CUDA_TRY(h, cudaMemsetAsync(h->script, 0xff, (size_t)h->B_cap * (h->T_cap + h->k_cap) * 4, scope.st));
    CUDA_TRY(h, cudaMemcpy2DAsync(h->script, (size_t)(h->T_cap + h->k_cap) * 4, d_script, (size_t)stride * 4, (size_t)w * 4, B,
                                  cudaMemcpyDeviceToDevice, scope.st));
    h->script_on = true;
    return SPECDEC_OK;
}

int specdec_profile_read(specdec_handle* h, double* h_ms, long long* h_launches) {
    if (!h || !h_ms || !h_launches) return SPECDEC_ERR_INVALID_ARG;
    *h_ms = h->prof_ms; *h_launches = h->prof_launches;
    return SPECDEC_OK;
}

int specdec_accept_scan(const float* d_logits, const int32_t* d_draft, int B, int k, int V, int beta, float tau,
                        int32_t* d_accepted, int32_t* d_bif, void* stream) {
    if (!d_logits || !d_draft || !d_accepted || !d_bif || B < 1 || k < 1 || V < 1 || beta < 1 || !(tau >= 0.f))
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "accept_scan: bad argument");
    k_accept_logits<<<B, 256, 0, (cudaStream_t)stream>>>(d_logits, d_draft, k, V, beta, tau, d_accepted, d_bif);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(nullptr, SPECDEC_ERR_CUDA, std::string("accept_scan: ") + cudaGetErrorString(e));
    return SPECDEC_OK;
}

// ---- acceptance scan for callers that must not allocate ---------------------------------------------
// The per-(row, tile) partial statistics live in a file-scope device array instead of an arena.  In host
// code `g_static_scratch` is only a stand-in for the symbol: the kernels get the device address that
// cudaGetSymbolAddress returns, looked up once per device with that device current.
namespace {
constexpr int NA_MAX_ROWS = 4096;      // B * (k + 1)
constexpr int NA_TILE = 1024;          // vocabulary columns per partial
constexpr int NA_MAX_TILES = 64;       // => V <= 65536
constexpr int NA_MAX_BLOCK = 2048;     // k + 1: 2048 records of 16 bytes + the kernel's static 256 bytes stay below the 48 KB default
constexpr size_t NA_PART_BYTES = (size_t)NA_MAX_ROWS * NA_MAX_TILES * sizeof(RowPart);
constexpr size_t NA_BYTES = NA_PART_BYTES + (size_t)NA_MAX_ROWS * 8;
static __device__ __align__(256) unsigned char g_static_scratch[NA_BYTES];
constexpr int NA_MAX_DEVICES = 64;
void* g_static_scratch_addr[NA_MAX_DEVICES] = {nullptr};
}  // namespace

int specdec_accept_scan_static(const float* d_logits, const int32_t* d_draft, int B, int k, int V, int beta, float tau,
                               int32_t* d_accepted, int32_t* d_bif, void* stream) {
    if (!d_logits || !d_draft || !d_accepted || !d_bif || B < 1 || k < 1 || V < 1 || beta < 1 || !(tau >= 0.f))
        return fail(nullptr, SPECDEC_ERR_INVALID_ARG, "accept_scan_static: bad argument");
    const long long rows = (long long)B * (k + 1);
    const int n_tiles = (V + NA_TILE - 1) / NA_TILE;
    // the second stage keeps one merged record per row of a sequence in (default-sized) dynamic shared memory
    if (rows > NA_MAX_ROWS || n_tiles > NA_MAX_TILES || k + 1 > NA_MAX_BLOCK)
        return fail(nullptr, SPECDEC_ERR_CAPACITY,
                    "accept_scan_static: B*(k+1) = " + std::to_string(rows) + " (limit " + std::to_string(NA_MAX_ROWS) +
                    "), V = " + std::to_string(V) + " (limit " + std::to_string(NA_MAX_TILES * NA_TILE) +
                    ") or k+1 = " + std::to_string(k + 1) + " (limit " + std::to_string(NA_MAX_BLOCK) +
                    ") exceeds the static scratch; use specdec_accept_scan");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES)
        return fail(nullptr, SPECDEC_ERR_CUDA, std::string("accept_scan_static: cudaGetDevice: ") + cudaGetErrorString(e));
    if (!g_static_scratch_addr[dev]) {          // first call on this device: resolve the symbol's device address
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p)
            return fail(nullptr, SPECDEC_ERR_CUDA, std::string("accept_scan_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_static_scratch_addr[dev] = p;
    }
    unsigned char* base = (unsigned char*)g_static_scratch_addr[dev];
    RowPart* part = (RowPart*)base;
    float* ld = (float*)(base + NA_PART_BYTES);
    int* ld_id = (int*)(base + NA_PART_BYTES + (size_t)NA_MAX_ROWS * 4);
    cudaStream_t st = (cudaStream_t)stream;
    // every slot the second stage reads is rewritten by the first, so nothing has to start at zero
    k_logit_tile_stats<<<dim3(n_tiles, (unsigned)rows), 256, 0, st>>>(d_logits, d_draft, k, V, NA_TILE, n_tiles, part, ld, ld_id);
    FusedCommit no_commit{};
    k_accept<<<B, 256, (size_t)(k + 1) * sizeof(RowPart), st>>>(part, n_tiles, ld, ld_id, k, beta, tau, d_accepted, d_bif,
                                                                nullptr, 0, no_commit);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(nullptr, SPECDEC_ERR_CUDA, std::string("accept_scan_static: ") + cudaGetErrorString(e));
    return SPECDEC_OK;
}

int specdec_debug_logits(specdec_handle* h, int which, float* d_logits, void* stream) {
    if (!h || !d_logits) return SPECDEC_ERR_INVALID_ARG;
    StreamScope scope(h, stream);
    cudaStream_t st = scope.st;
    int cnt, rows; const ModelW* m;
    if (which == 0) { if (!h->verified) return fail(h, SPECDEC_ERR_INVALID_ARG, "debug_logits: no verify pass to replay");
        cnt = CNT_VERIFY; rows = h->B * (h->last_k + 1); m = &h->ver; }
    else { if (!h->drafted) return fail(h, SPECDEC_ERR_INVALID_ARG, "debug_logits: no draft pass to replay");
        cnt = CNT_DRAFT_MASK; rows = h->last_draft_rows_ub; m = &h->dra; }
    const int d = m->dm.d_model, V = m->dm.vocab;
    return DISPATCH(h, gemm<bf16>(h, EPI_F32, h->y, d, m->embed, nullptr, V, d, cnt, rows, nullptr, 0, d_logits, st),
                    gemm<float>(h, EPI_F32, h->y, d, m->embed, nullptr, V, d, cnt, rows, nullptr, 0, d_logits, st));
}

int specdec_debug_trace(specdec_handle* h, long long* h_out, int n) {
    if (!h || !h_out || n < 1 || n > 256) return SPECDEC_ERR_INVALID_ARG;
    CUDA_TRY(h, cudaDeviceSynchronize());
    CUDA_TRY(h, cudaMemcpy(h_out, h->trace_buf, (size_t)n * 8, cudaMemcpyDeviceToHost));
    return SPECDEC_OK;
}

int specdec_debug_link_cost(specdec_handle* h, int n_links, int grid, double* h_us_per_link) {
    if (!h || !h_us_per_link || n_links < 1 || n_links > 4096 || grid < 1 || grid > 65535) return SPECDEC_ERR_INVALID_ARG;
    cudaStream_t st = h->own_stream;
    int* word = reinterpret_cast<int*>(h->trace_buf + 255);     // (the last slot of the time-stamp array: no kernel of the path touches it)
    cudaGraph_t g = nullptr; cudaGraphExec_t ex = nullptr;
    CUDA_TRY(h, cudaStreamSynchronize(st));
    CUDA_TRY(h, cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < n_links && e == cudaSuccess; ++i) e = launch_pdl(h, k_link, dim3(grid), dim3(128), 0, st, word);
    cudaError_t e2 = cudaStreamEndCapture(st, &g);
    if (e != cudaSuccess || e2 != cudaSuccess || !g) { if (g) cudaGraphDestroy(g); return fail(h, SPECDEC_ERR_CUDA, "link cost: capture failed"); }
    e = cudaGraphInstantiate(&ex, g, 0);
    cudaGraphDestroy(g);
    if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("link cost: ") + cudaGetErrorString(e));
    cudaEvent_t a, b;
    cudaEventCreate(&a); cudaEventCreate(&b);
    float best = 1e30f;
    for (int rep = 0; rep < 12; ++rep) {
        cudaEventRecord(a, st);
        cudaGraphLaunch(ex, st);
        cudaEventRecord(b, st);
        cudaStreamSynchronize(st);
        float ms = 0.f;
        if (rep >= 2 && cudaEventElapsedTime(&ms, a, b) == cudaSuccess && ms < best) best = ms;
    }
    cudaEventDestroy(a); cudaEventDestroy(b);
    cudaGraphExecDestroy(ex);
    h->launches += 12LL * n_links;
    *h_us_per_link = (double)best * 1e3 / n_links;
    return SPECDEC_OK;
}

int specdec_debug_cluster_round(specdec_handle* h, int cluster_size, int bytes_per_peer, int rounds, double* h_ns_per_round) {
    if (!h || !h_ns_per_round || rounds < 1 || rounds > 4096 || bytes_per_peer < 0 || bytes_per_peer > 8192 || bytes_per_peer % 16)
        return SPECDEC_ERR_INVALID_ARG;
    cudaStream_t st = h->own_stream;
    long long* scratch = reinterpret_cast<long long*>(h->trace_buf + 128);
    cudaError_t e;
    if (cluster_size == 8) e = sd::cluster_round_run<8>(rounds, bytes_per_peer, scratch, h->ses.counters + 7, st, h_ns_per_round);
    else if (cluster_size == 16) e = sd::cluster_round_run<16>(rounds, bytes_per_peer, scratch, h->ses.counters + 7, st, h_ns_per_round);
    else return fail(h, SPECDEC_ERR_INVALID_ARG, "cluster round: clusters of 8 or 16 CTAs");
    if (e != cudaSuccess) { cudaGetLastError(); return fail(h, SPECDEC_ERR_CUDA, std::string("cluster round: ") + cudaGetErrorString(e)); }
    h->launches += 2;
    return SPECDEC_OK;
}

int specdec_debug_mma_rate_bg(specdec_handle* h, int bn, int two_sm, int n_mma, int bg_stages, int commit_every, double* h_issue_clocks,
                              double* h_done_clocks, double* h_bg_bytes_per_clock) {
    if (!h || !h_issue_clocks || !h_done_clocks || n_mma < 16 || n_mma > (1 << 20) || bg_stages < 0 || bg_stages > 6 || commit_every < 0) return SPECDEC_ERR_INVALID_ARG;
    if (h->dtype != SPECDEC_DTYPE_BF16 || !h->tma.ready) return fail(h, SPECDEC_ERR_UNSUPPORTED, "mma rate: needs a bf16 handle on an sm_100 device");
    cudaStream_t st = h->own_stream;
    long long* scratch = reinterpret_cast<long long*>(h->part);          // (the vocabulary partials: at least 4 x 148 words)
    int* errw = h->ses.counters + 7;
    // the background stream reads the verifier's embedding table (any resident bytes will do)
    const void* src = h->ver.embed;
    const long long window = (long long)h->cfg.verifier.vocab * h->cfg.verifier.d_model * 2 / 16384 * 16384;
    if (bg_stages > 0 && window < (8ll << 20)) return fail(h, SPECDEC_ERR_UNSUPPORTED, "mma rate: the background stream needs an embedding table of at least 8 MB");
    double bg = 0.0;
    cudaError_t e;
#define RATE(BN_, PAIR_) e = sd::mma_rate_run<BN_, PAIR_>(h->tma.n_sm, n_mma, scratch, errw, st, h_issue_clocks, h_done_clocks, src, bg_stages, window, &bg, commit_every > 0 ? 1 : 0, bg_stages > 0 ? 2 : 4)
    if (two_sm) {
        if (bn == 128) RATE(128, true);
        else if (bn == 256) RATE(256, true);
        else return fail(h, SPECDEC_ERR_INVALID_ARG, "mma rate: two-SM tiles are 128 or 256 columns wide");
    } else {
        if (bn == 64) RATE(64, false);
        else if (bn == 128) RATE(128, false);
        else if (bn == 256) RATE(256, false);
        else return fail(h, SPECDEC_ERR_INVALID_ARG, "mma rate: tiles are 64, 128 or 256 columns wide");
    }
#undef RATE
    if (e != cudaSuccess) return fail(h, SPECDEC_ERR_CUDA, std::string("mma rate: ") + cudaGetErrorString(e));
    if (h_bg_bytes_per_clock) *h_bg_bytes_per_clock = bg;
    h->launches += 2;
    return SPECDEC_OK;
}

int specdec_debug_mma_rate(specdec_handle* h, int bn, int two_sm, int n_mma, double* h_issue_clocks, double* h_done_clocks) {
    return specdec_debug_mma_rate_bg(h, bn, two_sm, n_mma, 0, 0, h_issue_clocks, h_done_clocks, nullptr);
}

int specdec_debug_row_stats(specdec_handle* h, float* d_stats, void* stream) {
    if (!h || !d_stats) return SPECDEC_ERR_INVALID_ARG;
    if (!h->verified) return fail(h, SPECDEC_ERR_INVALID_ARG, "debug_row_stats: no verify pass");
    StreamScope scope(h, stream);
    CUDA_TRY(h, cudaMemcpyAsync(d_stats, h->row_stats, (size_t)h->B * (h->last_k + 1) * 6 * 4, cudaMemcpyDeviceToDevice,
                                scope.st));
    return SPECDEC_OK;
}

// Public step calls: the entry proper, then (option "debug_checks") the integrity check.
int specdec_encode(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len, const int32_t* d_max_tgt, int B,
                   int S_max, void* stream) {
    NvtxRange r("specdec_encode");
    return post_check(h, encode_entry(h, d_src, d_src_len, d_max_tgt, B, S_max, stream), stream);
}
int specdec_draft(specdec_handle* h, int k, int32_t* d_draft, void* stream) {
    NvtxRange r("specdec_draft");
    return post_check(h, draft_entry(h, k, d_draft, stream), stream);
}
int specdec_verify(specdec_handle* h, const int32_t* d_draft, int k, int beta, float tau, int32_t* d_accepted,
                   int32_t* d_bif, void* stream) {
    NvtxRange r("specdec_verify");
    return post_check(h, verify_entry(h, d_draft, k, beta, tau, d_accepted, d_bif, stream), stream);
}
int specdec_commit(specdec_handle* h, const int32_t* d_keep, const int32_t* d_next, void* stream) {
    NvtxRange r("specdec_commit");
    return post_check(h, commit_entry(h, d_keep, d_next, stream), stream);
}
int specdec_generate(specdec_handle* h, const int32_t* d_src, const int32_t* d_src_len, const int32_t* d_max_tgt, int B,
                     int S_max, int k, int beta, float tau, int32_t* d_out, int out_stride, int32_t* d_out_len,
                     specdec_stats* h_stats, void* stream) {
    NvtxRange r("specdec_generate");
    return post_check(h, generate_entry(h, d_src, d_src_len, d_max_tgt, B, S_max, k, beta, tau, d_out, out_stride, d_out_len, h_stats, stream), stream);
}
int specdec_generate_host(specdec_handle* h, const int32_t* h_src, const int32_t* h_src_len, const int32_t* h_max_tgt,
                          int B, int S_max, int k, int beta, float tau, int32_t* h_out, int out_stride,
                          int32_t* h_out_len, specdec_stats* h_stats, void* stream) {
    NvtxRange r("specdec_generate_host");
    return post_check(h, generate_host_entry(h, h_src, h_src_len, h_max_tgt, B, S_max, k, beta, tau, h_out, out_stride, h_out_len, h_stats, stream), stream);
}

int specdec_debug_integrity(specdec_handle* h, specdec_integrity* out, void* stream) {
    if (!h || !out) return SPECDEC_ERR_INVALID_ARG;
    return integrity_run(h, (cudaStream_t)stream, out);
}

}  // extern "C"
