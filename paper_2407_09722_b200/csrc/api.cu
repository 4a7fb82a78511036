// Host dispatcher behind the C ABI: argument validation, workspace carving, and the launch sequence of one
// verification step.  No device memory is allocated here; everything lives in the caller's workspace.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <new>

#include "common.cuh"
#include "tc_gemm.cuh"

using namespace mtad;

// K and V are rounded to bf16 for the cache: their projection accumulates at most this many k-blocks (512 elements)
// per tensor-memory accumulator, the pieces being added in fp32 (relative error about 4e-7 instead of 4e-6 at K = 8192)
static const int kQkvSegCap = 8;
static const int kCtas = 148;   // SMs the tensor-core GEMM spreads over

// Host-side tensor maps of one model's weight matrices.
struct WeightMaps {                      // index 0, 1, 2: tiles of 128, 256, 512 rows (1, 2, 4 halves)
    std::vector<CUtensorMap> wq[3], wk[3], wv[3], wo[3], gate[3], up[3], down[3];
    CUtensorMap lm_head[3];
    bool ok = false;
};

constexpr size_t kCanaryBytes = 64;
struct Region {                 // one array of the workspace: where it starts and how many elements it holds
    const char* name;
    size_t off, count, elem;
};

// One GEMM launch of the tensor-core forward, and the plan of a whole forward: everything about the launches that
// depends only on (model, sequences per call, rows per sequence, LM-head mode).  Plans are built once per shape and
// kept in the context; a call patches in what changes from call to call (status words, uniforms, debug fields).
struct GemmDesc { TcMaps mp; TcGemmParams p; double bytes; bool cluster; bool attn_before; };
struct ForwardPlan {
    std::vector<GemmDesc> g;           // per layer: QKV (or Q, then K/V), O (the attention pass runs before it),
                                       // gate/up, down; then the LM head
    int lm_tiles128 = 0;
    bool split_kv = false;             // K and V have a launch of their own, fed by sc.xkv with kv_terms terms
    int kv_terms = 0;
    bool maps = false;                 // tensor maps encoded (false: decomposition only, for the extent audit)
};

struct mtad_ctx {
    std::vector<Region> regions;        // the workspace's arrays, each followed by kCanaryBytes of guard pattern
    char* ws_base = nullptr;
    std::map<uint64_t, ForwardPlan> plans;   // by (model, sequences, rows per sequence, LM-head mode)
    WeightMaps tmaps, amaps;
    bool use_tc = false, use_pdl = false;
    size_t tc_ws_floats = 0, tc_counter_n = 0, xf_elems = 0;
    ModelView target, aux;
    bool has_aux = false;
    int max_batch = 0, max_nodes = 0, T_max = 0;
    SeqState st{};
    RowMeta rm{};
    Scratch sc{};
    std::vector<long long> len_ub;      // host upper bound of each sequence's committed length
    std::vector<int> npend_ub;          // host upper bound of each sequence's auxiliary pending count
    DraftState ds{};
    bool draft_active = false;          // the last mtad_draft's tree has not been committed yet
    int draft_B = 0, draft_gamma = 0;
    int32_t draft_seqs[MTAD_MAX_BATCH];
    bool last_chain = false;            // the last verify call was mtad_verify_chain
    int last_B = 0, last_R = 0, last_D = 0;
    int32_t last_seqs[MTAD_MAX_BATCH];
    int last_cuda = 0;
    unsigned int wait_limit = 0;        // debug: iteration limit of the GEMM kernels' bounded waits (0: default)
    int debug_no_operands = 0;          // debug: the GEMM kernels' operand-row copies are left out (waits run out)
    int warp_k = 0;                     // 0: unwarped target rows
    float warp_p = 1.f;
    int dwarp_k = 0;                    // 0: the draft samples from the unwarped auxiliary rows
    float dwarp_p = 1.f;
    // optional per-kernel-class timing (cudaEvent pairs around each launch)
    bool prof_on = false;
    std::vector<cudaEvent_t> prof_ev;        // pool, used pairwise
    std::vector<int> prof_cls;               // class of each recorded pair
    std::vector<double> prof_bytes;          // algorithmic bytes of each recorded pair
    std::vector<int> prof_n;                 // launches inside each recorded pair
    size_t prof_used = 0;
    bool prof_grouped = false;               // one pair around every run of consecutive launches of a class
    int prof_open = -1;                      // class of the run whose closing event is still to be recorded
    cudaStream_t prof_stream = nullptr;
};

unsigned long long g_kernel_launches = 0;    // kernels of this library enqueued since load

#ifdef MTAD_TRACE
// Trace builds only: global-timer stamps of every CTA of the GEMM launches made while tracing is on
constexpr int kTraceLaunches = 320, kTraceCtas = 320;
static __device__ unsigned long long g_trace[kTraceLaunches][kTraceCtas][8];
static unsigned long long* g_trace_dev = nullptr;
static int g_trace_n = -1;                   // launches recorded so far, -1: off
static int g_trace_meta[kTraceLaunches][4];  // cluster?, mode, grid, csize
static unsigned long long* trace_slot(bool cluster, int mode, int grid, int csize) {
    if (g_trace_n < 0 || g_trace_n >= kTraceLaunches || grid > kTraceCtas) return nullptr;
    g_trace_meta[g_trace_n][0] = cluster; g_trace_meta[g_trace_n][1] = mode;
    g_trace_meta[g_trace_n][2] = grid; g_trace_meta[g_trace_n][3] = csize;
    return g_trace_dev + (size_t)(g_trace_n++) * kTraceCtas * 8;
}
extern "C" int mtad_trace_begin(void) {
    if (!g_trace_dev && cudaGetSymbolAddress((void**)&g_trace_dev, g_trace) != cudaSuccess) return -1;
    cudaMemset(g_trace_dev, 0, sizeof(unsigned long long) * kTraceLaunches * kTraceCtas * 8);
    g_trace_n = 0;
    return 0;
}
extern "C" int mtad_trace_end(unsigned long long* host, int* meta, int max_launches) {
    cudaDeviceSynchronize();
    const int n = g_trace_n < max_launches ? g_trace_n : max_launches;
    g_trace_n = -1;
    if (n > 0) {
        cudaMemcpy(host, g_trace_dev, sizeof(unsigned long long) * (size_t)n * kTraceCtas * 8, cudaMemcpyDeviceToHost);
        memcpy(meta, g_trace_meta, sizeof(int) * 4 * n);
    }
    return n;
}
#endif

namespace {

struct Carver {
    char* base;
    size_t off = 0;
    std::vector<Region>* log = nullptr;
    explicit Carver(void* b) : base(static_cast<char*>(b)) {}
    template <typename T>
    T* take(size_t count, const char* name) {
        off = (off + 255) & ~size_t(255);
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        if (log) log->push_back({name, off, count, sizeof(T)});
        off += count * sizeof(T) + kCanaryBytes;          // guard words behind every array (mtad_debug_check_canaries)
        return p;
    }
};

bool model_ok(const mtad_model_desc* m) {
    if (!m) return false;
    if (m->layers < 1 || m->d_model < 8 || m->n_q_heads < 1 || m->n_kv_heads < 1 || m->d_ffn < 8 || m->vocab < 1)
        return false;
    if (m->head_dim != 32 && m->head_dim != 64 && m->head_dim != 128) return false;
    if (m->n_q_heads % m->n_kv_heads) return false;
    if (m->d_model % 8 || m->d_ffn % 8 || (m->n_q_heads * m->head_dim) % 8) return false;
    if (!(m->rope_base > 1.f) || !(m->rms_eps >= 0.f)) return false;
    return true;
}

bool model_ptrs_ok(const mtad_model_desc* m) {
    if (!m->embed || !m->lm_head || !m->final_norm || !m->layer_weights || !m->kv_cache) return false;
    if (m->kv_capacity < 1) return false;
    for (int i = 0; i < m->layers * MTAD_LAYER_TENSORS; ++i)
        if (!m->layer_weights[i]) return false;
    return true;
}

// Lays out the workspace; with base == nullptr only measures it.
size_t carve(mtad_ctx* c, const mtad_model_desc* t, const mtad_model_desc* a, int max_batch, int max_nodes,
             void* base, std::vector<Region>* log = nullptr) {
    Carver k(base);
    k.log = log;
    const size_t T = (size_t)max_batch * (max_nodes + 1);
    auto mx = [&](auto f) { size_t v = f(t); if (a) v = std::max(v, (size_t)f(a)); return v; };
    const size_t d = mx([](const mtad_model_desc* m) { return (size_t)m->d_model; });
    const size_t qkv = mx([](const mtad_model_desc* m) { return (size_t)(m->n_q_heads + 2 * m->n_kv_heads) * m->head_dim; });
    const size_t qd = mx([](const mtad_model_desc* m) { return (size_t)m->n_q_heads * m->head_dim; });
    const size_t F = mx([](const mtad_model_desc* m) { return (size_t)m->d_ffn; });
    const size_t V = mx([](const mtad_model_desc* m) { return (size_t)m->vocab; });
    const size_t hh = mx([](const mtad_model_desc* m) { return (size_t)m->head_dim / 2; });
    // split-KV partials: one split per 64 keys on the tensor-core attention path
    const size_t part = mx([&](const mtad_model_desc* m) {
        const size_t splits = std::max<size_t>(attn_split_cap(m->n_q_heads),
                                               (size_t)((m->kv_capacity + max_nodes + 1 + 63) / 64));
        return (size_t)m->n_q_heads * splits * (m->head_dim + 2);
    });
    SeqState st;
    st.kv_len = k.take<int32_t>(max_batch, "st_kv_len");
    st.root_tok = k.take<int32_t>(max_batch, "st_root_tok");
    st.aux_len = k.take<int32_t>(max_batch, "st_aux_len");
    st.aux_npend = k.take<int32_t>(max_batch, "st_aux_npend");
    st.aux_pend = k.take<int32_t>((size_t)max_batch * (MTAD_MAX_DEPTH + 1), "st_aux_pend");
    RowMeta rm;
    rm.tok = k.take<int32_t>(T, "rm_tok");
    rm.pos = k.take<int32_t>(T, "rm_pos");
    rm.slot = k.take<int32_t>(T, "rm_slot");
    rm.seq = k.take<int32_t>(T, "rm_seq");
    rm.depth = k.take<int32_t>(T, "rm_depth");
    rm.mask = k.take<uint32_t>(T * MTAD_MASK_WORDS, "rm_mask");
    rm.n_rows = k.take<int32_t>(max_batch, "rm_n_rows");
    rm.n_spec = k.take<int32_t>(max_batch, "rm_n_spec");
    rm.kv_base = k.take<int32_t>(max_batch, "rm_kv_base");
    rm.call_seq = k.take<int32_t>(max_batch, "rm_call_seq");
    Scratch sc;
    sc.hidden = k.take<float>(T * d, "hidden");
    sc.xn = k.take<float>(T * d, "xn");
    sc.qkv = k.take<float>(T * qkv, "qkv");
    sc.attn = k.take<float>(T * qd, "attn");
    sc.act = k.take<float>(T * F, "act");
    sc.rope = k.take<float>(T * hh * 2, "rope");
    sc.attn_part = k.take<float>(T * part, "attn_part");
    sc.q_hi = k.take<__nv_bfloat16>(T * qd, "q_hi");
    sc.q_lo = k.take<__nv_bfloat16>(T * qd, "q_lo");
    sc.logits = k.take<float>(T * V, "logits");
    sc.node_lp = k.take<float>(T, "node_lp");
    sc.row_lse = k.take<float>(T, "row_lse");
    sc.row_cand = k.take<int32_t>(T, "row_cand");
    sc.row_cand_lp = k.take<float>(T, "row_cand_lp");
    rm.prow = k.take<int32_t>(T, "rm_prow");
    // tensor-core path buffers (operand rows are always TC_X_ROWS high so that the TMA box never leaves them)
    const size_t Tc = std::min<size_t>(T, TC_MAX_ROWS);
    const size_t rpad = (Tc + 15) / 16 * 16;
    // operand rows, hi and lo interleaved: row 2t = hi(t), row 2t + 1 = lo(t)
    sc.xd = k.take<__nv_bfloat16>((size_t)2 * TC_X_ROWS * d, "xd");
    sc.xa = k.take<__nv_bfloat16>((size_t)2 * TC_X_ROWS * qd, "xa");
    sc.xf = k.take<__nv_bfloat16>((size_t)2 * TC_X_ROWS * F, "xf");
    sc.xkv = k.take<__nv_bfloat16>((size_t)2 * TC_X_ROWS * d, "xkv");
    const size_t dt = (d + TC_TILE_N - 1) / TC_TILE_N;
    sc.sumsq_a = k.take<float>(dt * TC_X_ROWS, "sumsq_a");
    sc.sumsq_b = k.take<float>(dt * TC_X_ROWS, "sumsq_b");
    size_t ws_tiles = 0, max_tiles = 0, lm_tiles = 0;
    auto shape_ws = [&](const mtad_model_desc* m) {
        const int qdm = m->n_q_heads * m->head_dim, kvm = m->n_kv_heads * m->head_dim;
        const int shapes[5][2] = {{(qdm + 127) / 128 + 2 * ((kvm + 127) / 128), m->d_model},
                                  {(m->d_model + 127) / 128, qdm},
                                  {(m->d_ffn + 63) / 64, m->d_model},
                                  {(m->d_model + 127) / 128, m->d_ffn},
                                  {(m->vocab + 127) / 128, m->d_model}};
        for (auto& sh : shapes) {
            for (int mh = 1; mh <= 4; mh *= 2)
                for (int per_sm = 1; per_sm <= 2; ++per_sm) {
                    TcGemmParams tp{};
                    const int tiles = (sh[0] + mh - 1) / mh;
                    tc_decompose(tp, tiles, sh[1], 1, kCtas, per_sm);
                    ws_tiles = std::max(ws_tiles, (size_t)tiles * tp.max_contrib * mh);
                    max_tiles = std::max(max_tiles, (size_t)tiles);
                }
        }
        lm_tiles = std::max(lm_tiles, (size_t)(m->vocab + 127) / 128);
    };
    shape_ws(t);
    if (a) shape_ws(a);
    sc.tc_ws = k.take<float>(ws_tiles * rpad * TC_TILE_N, "tc_ws");
    sc.tc_counters = k.take<int32_t>(max_tiles, "tc_counters");
    sc.lm_part = k.take<float4>(Tc * lm_tiles, "lm_part");
    sc.node_z = k.take<float>(T, "node_z");
    sc.draft_part = a ? k.take<DraftPart>((size_t)max_batch * MTAD_MAX_BEAM * MTAD_DRAFT_CHUNKS, "draft_part") : nullptr;
    sc.warp_part = k.take<WarpPart>(T * MTAD_DRAFT_CHUNKS, "warp_part");
    sc.warp_row = k.take<WarpRow>(T, "warp_row");
    DraftState ds;
    ds.base_len = k.take<int32_t>(max_batch, "ds_base_len");
    ds.npend = k.take<int32_t>(max_batch, "ds_npend");
    ds.gamma = k.take<int32_t>(max_batch, "ds_gamma");
    ds.beam = k.take<int32_t>(max_batch, "ds_beam");
    ds.node_tok = k.take<int32_t>((size_t)max_batch * MTAD_DRAFT_NODES, "ds_node_tok");
    ds.node_parent = k.take<int32_t>((size_t)max_batch * MTAD_DRAFT_NODES, "ds_node_parent");
    ds.node_logq = k.take<float>((size_t)max_batch * MTAD_DRAFT_NODES, "ds_node_logq");
    ds.node_mask = k.take<uint32_t>((size_t)max_batch * MTAD_DRAFT_NODES * MTAD_MASK_WORDS, "ds_node_mask");
    ds.best_path = k.take<int32_t>((size_t)max_batch * MTAD_MAX_DEPTH, "ds_best_path");
    ds.tree_id = k.take<int32_t>((size_t)max_batch * MTAD_DRAFT_NODES, "ds_tree_id");
    ds.tree2slot = k.take<int32_t>((size_t)max_batch * MTAD_DRAFT_NODES, "ds_tree2slot");
    ds.nb = k.take<int32_t>((size_t)max_batch * MTAD_MAX_DEPTH, "ds_nb");
    ds.n_tree = k.take<int32_t>((size_t)max_batch, "ds_n_tree");
    if (c) {
        c->ds = ds;
        c->st = st; c->rm = rm; c->sc = sc;
        c->tc_ws_floats = ws_tiles * rpad * TC_TILE_N;
        c->tc_counter_n = max_tiles;
        c->xf_elems = (size_t)2 * TC_X_ROWS * F;
    }
    return (k.off + 255) & ~size_t(255);
}

#define CU(call)                                                  \
    do {                                                          \
        cudaError_t e__ = (call);                                 \
        if (e__ != cudaSuccess) { ctx->last_cuda = (int)e__; return MTAD_E_CUDA; } \
    } while (0)

// Enqueue one launcher; when profiling is on, bracket it with an event pair on the same stream - or, in grouped mode,
// bracket every run of consecutive launches of one class with a single pair, so that the launches inside a run keep
// their programmatic overlap (an event between two launches serialises them).
template <class F>
int timed(mtad_ctx* ctx, int cls, double bytes, int kernels, cudaStream_t s, F&& f) {
    if (ctx->prof_on) {
        if (ctx->prof_open >= 0 && !(ctx->prof_grouped && ctx->prof_open == cls)) {
            CU(cudaEventRecord(ctx->prof_ev[2 * (ctx->prof_cls.size() - 1) + 1], ctx->prof_stream));
            ctx->prof_open = -1;
        }
        if (ctx->prof_open < 0 && ctx->prof_used + 2 <= ctx->prof_ev.size()) {
            CU(cudaEventRecord(ctx->prof_ev[ctx->prof_used], s));
            ctx->prof_cls.push_back(cls);
            ctx->prof_bytes.push_back(0.0);
            ctx->prof_n.push_back(0);
            ctx->prof_used += 2;
            ctx->prof_open = cls;
            ctx->prof_stream = s;
        }
    }
    CU(f());
    g_kernel_launches += kernels;
    if (ctx->prof_on && ctx->prof_open >= 0) {
        ctx->prof_bytes.back() += bytes;
        ctx->prof_n.back() += 1;
        if (!ctx->prof_grouped) {
            CU(cudaEventRecord(ctx->prof_ev[2 * (ctx->prof_cls.size() - 1) + 1], s));
            ctx->prof_open = -1;
        }
    }
    return MTAD_OK;
}
#define RUN(cls, bytes, kernels, call)                                                    \
    do {                                                                                  \
        int rc__ = timed(ctx, cls, bytes, kernels, s, [&]() -> cudaError_t { return (call); }); \
        if (rc__ != MTAD_OK) return rc__;                                                 \
    } while (0)

// One decoder forward over T = B * R prepared rows, leaving fp32 logits in the workspace.
int forward_rows(mtad_ctx* ctx, const ModelView& m, int B, int R, long long len_ub, cudaStream_t s) {
    const int T = B * R;
    const mtad_model_desc& d = m.d;
    const int qd = d.n_q_heads * d.head_dim, kvd = d.n_kv_heads * d.head_dim, ldq = qd + 2 * kvd;
    const Scratch& sc = ctx->sc;
    // split the keys [0, L + R) over CTAs: about four waves of (head, split, sequence) blocks
    const long long total = std::min<long long>(len_ub, d.kv_capacity) + R;
    int nsplit = (int)std::min<long long>(attn_split_cap(d.n_q_heads), (total + MTAD_ATTN_TILE - 1) / MTAD_ATTN_TILE);
    nsplit = std::max(1, std::min(nsplit, (4 * 148 + d.n_q_heads * B - 1) / (d.n_q_heads * B)));
    long long chunk = (total + nsplit - 1) / nsplit;
    chunk = (chunk + MTAD_ATTN_TILE - 1) / MTAD_ATTN_TILE * MTAD_ATTN_TILE;
    const double wb = 2.0;   // bytes per bf16 weight
    for (int l = 0; l < d.layers; ++l) {
        RUN(MTAD_K_NORM, 0, 1, launch_rmsnorm(sc.hidden, m.w(l, 0), sc.xn, T, d.d_model, d.rms_eps, s));
        RUN(MTAD_K_GEMM, wb * qd * d.d_model, 1,
            launch_gemm_rows(sc.xn, d.d_model, m.w(l, 1), nullptr, sc.qkv, ldq, 0, T, qd, d.d_model, 0, s));
        RUN(MTAD_K_GEMM, wb * kvd * d.d_model, 1,
            launch_gemm_rows(sc.xn, d.d_model, m.w(l, 2), nullptr, sc.qkv, ldq, qd, T, kvd, d.d_model, 0, s));
        RUN(MTAD_K_GEMM, wb * kvd * d.d_model, 1,
            launch_gemm_rows(sc.xn, d.d_model, m.w(l, 3), nullptr, sc.qkv, ldq, qd + kvd, T, kvd, d.d_model, 0, s));
        RUN(MTAD_K_ROPE, 0, 1, launch_rope_append(m, l, ctx->rm, sc, T, s));
        RUN(MTAD_K_ATTN, 0, 2, launch_attention(m, l, ctx->rm, sc, B, R, nsplit, (int)chunk, false, false, s));
        RUN(MTAD_K_GEMM, wb * d.d_model * qd, 1,
            launch_gemm_rows(sc.attn, qd, m.w(l, 4), nullptr, sc.hidden, d.d_model, 0, T, d.d_model, qd, 1, s));
        RUN(MTAD_K_NORM, 0, 1, launch_rmsnorm(sc.hidden, m.w(l, 5), sc.xn, T, d.d_model, d.rms_eps, s));
        RUN(MTAD_K_GEMM, wb * 2.0 * d.d_ffn * d.d_model, 1,
            launch_gemm_rows(sc.xn, d.d_model, m.w(l, 6), m.w(l, 7), sc.act, d.d_ffn, 0, T, d.d_ffn, d.d_model, 2, s));
        RUN(MTAD_K_GEMM, wb * d.d_model * d.d_ffn, 1,
            launch_gemm_rows(sc.act, d.d_ffn, m.w(l, 8), nullptr, sc.hidden, d.d_model, 0, T, d.d_model, d.d_ffn, 1, s));
    }
    RUN(MTAD_K_NORM, 0, 1,
        launch_rmsnorm(sc.hidden, static_cast<const __nv_bfloat16*>(d.final_norm), sc.xn, T, d.d_model, d.rms_eps, s));
    RUN(MTAD_K_GEMM, wb * d.vocab * d.d_model, 1,
        launch_gemm_rows(sc.xn, d.d_model, static_cast<const __nv_bfloat16*>(d.lm_head), nullptr, sc.logits, d.vocab, 0,
                         T, d.vocab, d.d_model, 0, s));
    return MTAD_OK;
}

bool build_weight_maps(const ModelView& m, WeightMaps& w) {
    const mtad_model_desc& d = m.d;
    const int qd = d.n_q_heads * d.head_dim, kvd = d.n_kv_heads * d.head_dim;
    auto aligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
    auto mk = [&](CUtensorMap* o, const void* base, long long rows, long long cols, int box) {
        return aligned(base) && tc_make_map(o, base, rows, cols, box) == 0;
    };
    bool ok = true;
    for (int i = 0; i < 3 && ok; ++i) {
        const int halves = 1 << i;
        const int box = halves == 1 ? 128 : 256;          // a 512-row tile is fetched as two 256-row boxes
        w.wq[i].resize(d.layers); w.wk[i].resize(d.layers); w.wv[i].resize(d.layers); w.wo[i].resize(d.layers);
        w.gate[i].resize(d.layers); w.up[i].resize(d.layers); w.down[i].resize(d.layers);
        for (int l = 0; l < d.layers && ok; ++l) {
            ok = ok && mk(&w.wq[i][l], m.w(l, 1), qd, d.d_model, box);
            ok = ok && mk(&w.wk[i][l], m.w(l, 2), kvd, d.d_model, box);
            ok = ok && mk(&w.wv[i][l], m.w(l, 3), kvd, d.d_model, box);
            ok = ok && mk(&w.wo[i][l], m.w(l, 4), d.d_model, qd, box);
            // gate and up share a tile: its first half are gate rows, its second half the matching up rows
            ok = ok && mk(&w.gate[i][l], m.w(l, 6), d.d_ffn, d.d_model, 64 * halves);
            ok = ok && mk(&w.up[i][l], m.w(l, 7), d.d_ffn, d.d_model, 64 * halves);
            ok = ok && mk(&w.down[i][l], m.w(l, 8), d.d_model, d.d_ffn, box);
        }
        ok = ok && mk(&w.lm_head[i], d.lm_head, d.vocab, d.d_model, box);
    }
    w.ok = ok;
    return ok;
}

bool mma_attention(const ModelView& m) {
    return m.kv_map_ok && (m.d.head_dim == 64 || m.d.head_dim == 128);
}

// K/V tiles of the tensor-core attention arrive by TMA: one map over the whole cache of a model
void build_kv_map(ModelView& m) {
    const mtad_model_desc& d = m.d;
    m.kv_map_ok = (d.head_dim == 64 || d.head_dim == 128) && (reinterpret_cast<uintptr_t>(d.kv_cache) & 15) == 0 &&
                  tc_make_kv_map(&m.kv_map, d.kv_cache, d.head_dim, d.kv_capacity,
                                 (long long)d.layers * m.max_batch * 2 * d.n_kv_heads) == 0;
}

// Builds the plan.  with_maps = false leaves out everything that needs the driver (the operand-row tensor maps) and
// the weight maps: what is left is the index arithmetic of the launches.
int build_plan(ForwardPlan& fp, const Scratch& sc, const RowMeta& rm, const ModelView& m, const WeightMaps* wm, int B,
               int R, bool lm_plain, bool with_maps, bool split_kv_ok) {
    const int T = B * R;
    const mtad_model_desc& d = m.d;
    const int qd = d.n_q_heads * d.head_dim, kvd = d.n_kv_heads * d.head_dim;
    const int rpad = (T + 15) / 16 * 16;
    const int dt = (d.d_model + TC_TILE_N - 1) / TC_TILE_N;
    const int mh = tc_halves(T);                          // weight halves per tile, as many as tensor memory allows
    auto ix = [](int halves) { return halves == 1 ? 0 : (halves == 2 ? 1 : 2); };
    auto up = [](int a, int b) { return (a + b - 1) / b; };
    // Operand rows: `terms` bf16 terms per activation row.  One TMA box covers all terms * rpad interleaved rows, or
    // they are cut into two or three boxes of at most 256 rows.
    // From width 8192 on the K/V rounding decides the accuracy of the whole step (a bf16 element that rounds the
    // other way shifts attention scores that are sharply peaked at that width).  There, with more than 32 rows (up to
    // 32 every row has three terms anyway), the K and V rows get a launch of their own: its input rows carry three
    // terms (a second copy written by the row preparation and the down projection) and its tensor-memory accumulation
    // runs in short chains (tc_gemm.cu), which holds the relative error near 5e-7; Q, which is never rounded to
    // bf16, keeps two terms and whole runs (about 2.5e-6) like every other projection.
    const int terms = tc_terms(T), tkv = tc_qkv_terms(T);
    const bool split_kv = split_kv_ok && d.d_model >= 8192 && T > 32 && tkv > terms;
    int mq = mh;                                          // QKV tiles must not straddle q | k | v
    while (mq > 1 && (qd % (128 * mq) || (!split_kv && kvd % (128 * mq)))) mq /= 2;
    const int xbox = terms * rpad / tc_boxes(terms * rpad), kvbox = tkv * rpad / tc_boxes(tkv * rpad);
    CUtensorMap xd{}, xkv{}, xa{}, xf{};
    if (with_maps &&
        (tc_make_map(&xd, sc.xd, 2 * TC_X_ROWS, d.d_model, xbox) || tc_make_map(&xkv, sc.xkv, 2 * TC_X_ROWS, d.d_model, kvbox) ||
         tc_make_map(&xa, sc.xa, 2 * TC_X_ROWS, qd, xbox) || tc_make_map(&xf, sc.xf, 2 * TC_X_ROWS, d.d_ffn, xbox)))
        return MTAD_E_CUDA;
    TcGemmParams base{};
    base.ws = sc.tc_ws; base.counters = sc.tc_counters;
    base.inv_dim = 1.f / (float)d.d_model; base.eps = d.rms_eps;
    base.Hq = d.n_q_heads; base.Hkv = d.n_kv_heads; base.hd = d.head_dim;
    base.q_out = sc.qkv; base.q_hi = sc.q_hi; base.q_lo = sc.q_lo; base.rope = sc.rope;
    base.cache = static_cast<__nv_bfloat16*>(d.kv_cache);
    base.slot = rm.slot; base.seq = rm.seq; base.max_batch = m.max_batch; base.cap = d.kv_capacity;
    base.hidden = sc.hidden; base.R = R; base.prow = rm.prow; base.tok = rm.tok; base.node_z = sc.node_z;
    base.lm_part = sc.lm_part;
    const double wb = 2.0;
    // The projections whose tiles fit the co-resident CTAs run as clusters that reduce over distributed shared memory
    // (tc_gemm_cluster.cu): QKV, O, down and, with few rows, the LM head; gate / up, with more tiles than half the CTA
    // slots, keeps the stream-K decomposition, which balances it better.  The plan picks the halves per tile itself.
    auto clusterize = [&](TcGemmParams& p, int n_tiles128, int K, bool want) -> bool {
        if (!want) return false;
        TcGemmParams q = p;
        if (!tc_cluster_plan(q, n_tiles128, K, T, kCtas)) return false;

        p = q;
        return true;
    };
    std::vector<GemmDesc>& g = fp.g;
    g.clear();
    g.reserve((size_t)d.layers * 4 + 1);
    const CUtensorMap none{};
    auto wmap = [&](const std::vector<CUtensorMap> (&v)[3], int halves, int l) -> const CUtensorMap& {
        return with_maps ? v[ix(halves)][l] : none;
    };
    for (int l = 0; l < d.layers; ++l) {
        {   // QKV + rotary + append (Q alone when K and V have their own launch)
            TcGemmParams p = base; TcMaps mp{};
            const int qt = up(qd, 128), kt = up(kvd, 128);
            const int n128 = split_kv ? qt : qt + 2 * kt;
            tc_decompose(p, n128 / mq, d.d_model, T, kCtas);
            p.mh = mq; p.n_rows_total = n128 * 128;
            p.mode = TC_QKV; p.N = qd; p.seg_k_tile = qt; p.seg_v_tile = qt + kt; p.layer = l;
            p.sumsq_in = sc.sumsq_a; p.sumsq_in_parts = (l == 0) ? 1 : dt;
            const bool cl = clusterize(p, n128, d.d_model, true);
            if (with_maps) { mp.a0 = wmap(wm->wq, p.mh, l); mp.a1 = wmap(wm->wk, p.mh, l); mp.a2 = wmap(wm->wv, p.mh, l); }
            mp.x = xd;
            g.push_back({mp, p, wb * (qd + (split_kv ? 0.0 : 2.0 * kvd)) * d.d_model, cl, false});
        }
        if (split_kv) {   // K and V rows: three-term input, short accumulation chains
            TcGemmParams p = base; TcMaps mp{};
            const int kt = up(kvd, 128);
            tc_decompose(p, 2 * kt, d.d_model, T, kCtas, 0, tkv);
            p.mh = 1; p.n_rows_total = 2 * kt * 128; p.seg_cap = kQkvSegCap;
            p.mode = TC_QKV; p.N = qd; p.seg_k_tile = 0; p.seg_v_tile = kt; p.layer = l;
            p.sumsq_in = sc.sumsq_a; p.sumsq_in_parts = (l == 0) ? 1 : dt;
            if (with_maps) { mp.a0 = wmap(wm->wk, 1, l); mp.a1 = wmap(wm->wk, 1, l); mp.a2 = wmap(wm->wv, 1, l); }
            mp.x = xkv;
            g.push_back({mp, p, wb * 2.0 * kvd * d.d_model, false, false});
        }
        {   // O projection + residual, emits the FFN norm's operand rows
            TcGemmParams p = base; TcMaps mp{};
            tc_decompose(p, up(d.d_model, 128 * mh), qd, T, kCtas);
            p.mh = mh; p.n_rows_total = d.d_model;
            p.mode = TC_RESID; p.N = d.d_model; p.sumsq_in_parts = 0;
            p.gain = m.w(l, 5); p.x_out = sc.xd; p.xk = d.d_model;
            p.sumsq_out = sc.sumsq_b;
            const bool cl = clusterize(p, up(d.d_model, 128), qd, true);
            if (with_maps) mp.a0 = wmap(wm->wo, p.mh, l);
            mp.x = xa;
            g.push_back({mp, p, wb * d.d_model * qd, cl, true});
        }
        {   // gate / up + SwiGLU
            TcGemmParams p = base; TcMaps mp{};
            tc_decompose(p, up(d.d_ffn, 64 * mh), d.d_model, T, kCtas);
            p.mh = mh; p.n_rows_total = d.d_ffn;
            p.mode = TC_SWIGLU; p.N = d.d_ffn; p.sumsq_in = sc.sumsq_b; p.sumsq_in_parts = dt;
            p.x_out = sc.xf; p.xk = d.d_ffn;
            mp.x = xd;
            TcGemmParams pa = p, pb = p;
            if (tc_ctas_per_sm(T) == 1 && tc_cluster_plan_big_split(pa, pb, up(d.d_ffn, 64), d.d_model, T, kCtas)) {
                // more tiles than SMs: two cluster launches over two ranges of the tiles
                if (with_maps) { mp.a0 = wmap(wm->gate, pa.mh, l); mp.a1 = wmap(wm->up, pa.mh, l); }
                const double all = wb * 2.0 * d.d_ffn * d.d_model, fa = (double)pa.n_tiles / (pa.n_tiles + pb.n_tiles);
                g.push_back({mp, pa, all * fa, true, false});
                g.push_back({mp, pb, all * (1.0 - fa), true, false});
            } else {
                if (with_maps) { mp.a0 = wmap(wm->gate, mh, l); mp.a1 = wmap(wm->up, mh, l); }
                g.push_back({mp, p, wb * 2.0 * d.d_ffn * d.d_model, false, false});
            }
        }
        {   // down projection + residual, emits the next norm's operand rows
            TcGemmParams p = base; TcMaps mp{};
            tc_decompose(p, up(d.d_model, 128 * mh), d.d_ffn, T, kCtas);
            p.mh = mh; p.n_rows_total = d.d_model;
            p.mode = TC_RESID; p.N = d.d_model; p.sumsq_in_parts = 0;
            p.gain = (l + 1 < d.layers) ? m.w(l + 1, 0) : static_cast<const __nv_bfloat16*>(d.final_norm);
            p.x_out = sc.xd; p.xk = d.d_model; p.sumsq_out = sc.sumsq_a;
            if (split_kv && l + 1 < d.layers) { p.x_out2 = sc.xkv; p.out_terms2 = tkv; }
            const bool cl = clusterize(p, up(d.d_model, 128), d.d_ffn, true);
            if (with_maps) mp.a0 = wmap(wm->down, p.mh, l);
            mp.x = xf;
            g.push_back({mp, p, wb * d.d_model * d.d_ffn, cl, false});
        }
    }
    {   // LM head: per-tile log-softmax / Gumbel-argmax partials + gather of the drafted tokens' logits, or plain
        // logits for the draft's beam selection and the warped rows
        TcGemmParams p = base; TcMaps mp{};
        tc_decompose(p, up(d.vocab, 128 * mh), d.d_model, T, kCtas);
        p.mh = mh; p.n_rows_total = d.vocab; p.n_tiles128 = up(d.vocab, 128);
        p.mode = lm_plain ? TC_PLAIN : TC_LMHEAD; p.N = d.vocab; p.sumsq_in = sc.sumsq_a; p.sumsq_in_parts = dt;
        p.out = sc.logits; p.ldo = d.vocab;
        fp.lm_tiles128 = p.n_tiles128;
        const bool cl = clusterize(p, up(d.vocab, 128), d.d_model, true);
        if (with_maps) mp.a0 = wm->lm_head[ix(p.mh)];
        mp.x = xd;
        g.push_back({mp, p, wb * d.vocab * d.d_model, cl, false});
    }
    fp.maps = with_maps;
    fp.split_kv = split_kv;
    fp.kv_terms = tkv;
    return MTAD_OK;
}

// Split of the keys [0, total) of the attention pass on the tensor-core path: tiles per block and blocks per head
struct AttnSplit { int nsp, ns; };
AttnSplit attn_split(const ModelView& m, int B, int R, long long total) {
    const int nsp = attention_mma_tiles_per_block(m, B, R, total);
    return {nsp, (int)(((total + 63) / 64 + nsp - 1) / nsp)};
}

// The forward on the tensor-core path: every projection is one launch of the TMA + tcgen05 GEMM with a fused
// epilogue; activations travel between launches as bf16 operand rows plus per-row sums of squares, so the RMSNorm is
// applied as a per-row scale in the consumer's epilogue.  Leaves lm_part / node_z for launch_lm_merge.
int forward_rows_tc(mtad_ctx* ctx, const ModelView& m, const WeightMaps& wm, int B, int R, long long len_ub,
                    const float* uniforms, uint32_t* status, bool lm_plain, cudaStream_t s) {
    const mtad_model_desc& d = m.d;
    const Scratch& sc = ctx->sc;
    const long long total = std::min<long long>(len_ub, d.kv_capacity) + R;
    const bool pdl = ctx->use_pdl;
    const uint64_t key = ((uint64_t)(&m == &ctx->aux ? 1 : 0) << 40) | ((uint64_t)B << 24) | ((uint64_t)R << 8) |
                         (lm_plain ? 1u : 0u);
    auto it = ctx->plans.find(key);
    if (it == ctx->plans.end()) {
        ForwardPlan fp;
        if (int rc = build_plan(fp, sc, ctx->rm, m, &wm, B, R, lm_plain, true, &m == &ctx->target)) return rc;
        it = ctx->plans.emplace(key, std::move(fp)).first;
    }
    ForwardPlan& fp = it->second;
    auto launch = [&](size_t i) -> int {
        GemmDesc& gd = fp.g[i];
        TcGemmParams& p = gd.p;
        p.status = status; p.uniforms = uniforms;
        p.wait_limit = ctx->wait_limit; p.debug_no_operands = ctx->debug_no_operands;
#ifdef MTAD_TRACE
        p.trace = trace_slot(gd.cluster, p.mode,
                             gd.cluster ? p.n_tiles * p.csize : (p.total_units + p.units_per_cta - 1) / p.units_per_cta,
                             gd.cluster ? p.csize : 0);
#endif
        if (gd.cluster) RUN(MTAD_K_GEMM, gd.bytes, 1, launch_tc_cluster(gd.mp, p, pdl, s));
        else RUN(MTAD_K_GEMM, gd.bytes, 1, launch_tc_gemm(gd.mp, p, kCtas, pdl, s));
        return MTAD_OK;
    };
    int layer = 0;
    for (size_t i = 0; i < fp.g.size(); ++i) {
        if (fp.g[i].attn_before) {                               // the O projection: the attention pass feeds it
            const int l = layer++;
            if (mma_attention(m)) {
                const AttnSplit as = attn_split(m, B, R, total);
                RUN(MTAD_K_ATTN, 0, 2, launch_attention_mma(m, l, ctx->rm, sc, B, R, as.ns, as.nsp, status, pdl, s));
                RUN(MTAD_K_ATTN, 0, 0, launch_attention_combine(m, ctx->rm, sc, B, R, as.ns, true, pdl, s));
            } else {
                int nsplit = (int)std::min<long long>(attn_split_cap(d.n_q_heads), (total + MTAD_ATTN_TILE - 1) / MTAD_ATTN_TILE);
                nsplit = std::max(1, std::min(nsplit, (4 * 148 + d.n_q_heads * B - 1) / (d.n_q_heads * B)));
                long long chunk = (total + nsplit - 1) / nsplit;
                chunk = (chunk + MTAD_ATTN_TILE - 1) / MTAD_ATTN_TILE * MTAD_ATTN_TILE;
                RUN(MTAD_K_ATTN, 0, 2, launch_attention(m, l, ctx->rm, sc, B, R, nsplit, (int)chunk, true, pdl, s));
            }
        }
        if (int rc = launch(i)) return rc;
    }
    if (!lm_plain) RUN(MTAD_K_LMRED, 0, 2, launch_lm_merge(m, ctx->rm, sc, B, R, fp.lm_tiles128, uniforms, status, s));
    return MTAD_OK;
}

bool seqs_ok(const mtad_ctx* ctx, int B, const int32_t* seqs) {
    if (!seqs || B < 1 || B > ctx->max_batch || B > MTAD_MAX_BATCH) return false;
    for (int i = 0; i < B; ++i) {
        if (seqs[i] < 0 || seqs[i] >= ctx->max_batch) return false;
        for (int j = 0; j < i; ++j)
            if (seqs[j] == seqs[i]) return false;
    }
    return true;
}

bool result_ok(const mtad_result* r) {
    return r && r->eta && r->winner && r->path && r->n_out && r->out_tok && r->out_lp && r->status;
}

int verify_common(mtad_ctx* ctx, int B, const int32_t* seqs, const int32_t* n_nodes, int N, int D,
                  const int32_t* tok, const int32_t* parent, const float* logq_ref, float log_tau,
                  const float* bonus_uniform, const mtad_result* out, void* stream,
                  const float* spd_accept_uniform = nullptr) {
    // spd_accept_uniform set: the rule of vanilla speculative decoding on a chain; logq_ref then holds the auxiliary
    // model's log-distributions [B, gamma, V] and bonus_uniform the uniforms of the final draw
    if (!ctx) return MTAD_E_INVALID;
    if (!seqs_ok(ctx, B, seqs)) return B > (ctx ? ctx->max_batch : 0) ? MTAD_E_CAPACITY : MTAD_E_INVALID;
    if (N < 0 || D < 0) return MTAD_E_INVALID;
    if (N > ctx->max_nodes || N > MTAD_MAX_NODES || D > MTAD_MAX_DEPTH) return MTAD_E_CAPACITY;
    if (N > 0 && (!tok || !logq_ref || D < 1)) return MTAD_E_INVALID;
    if (!bonus_uniform || !result_ok(out)) return MTAD_E_INVALID;
    if (isnan(log_tau) || !(log_tau < 0.f)) return MTAD_E_INVALID;       // tau in [0, 1)
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int R = N + 1;
    long long ub = 0;
    for (int i = 0; i < B; ++i) ub = std::max(ub, ctx->len_ub[seqs[i]]);

    CU(cudaMemsetAsync(out->status, 0, sizeof(uint32_t) * B, s));
    // a launch that gave up on a wait leaves split-K arrival counters behind: every call starts from zero
    CU(cudaMemsetAsync(ctx->sc.tc_counters, 0, sizeof(int32_t) * ctx->tc_counter_n, s));
    PrepareArgs pa{};
    for (int i = 0; i < B; ++i) pa.seqs.v[i] = seqs[i];
    pa.B = B; pa.R = R; pa.max_depth = D; pa.n_nodes = n_nodes; pa.tok = tok; pa.parent = parent;
    const bool tc = ctx->use_tc && ctx->tmaps.ok && B * R <= TC_MAX_ROWS;
    if (tc) {
        pa.gain0 = ctx->target.w(0, 0); pa.x = ctx->sc.xd; pa.terms = tc_terms(B * R);
        if (ctx->target.d.d_model >= 8192 && B * R > 32 && tc_qkv_terms(B * R) > pa.terms) {
            pa.x2 = ctx->sc.xkv; pa.terms2 = tc_qkv_terms(B * R);     // rows of the separate K/V launch (build_plan)
        }
        pa.sumsq_out = ctx->sc.sumsq_a;
    }
    RUN(MTAD_K_PREPARE, 0, 1, launch_prepare(ctx->target, ctx->st, ctx->rm, ctx->sc, pa, out->status, s));
    const bool spd = spd_accept_uniform != nullptr;
    const bool warped = ctx->warp_k > 0 && !spd;   // warped rows are made from plain logits, after the forward
    if (tc) {
        int rc = forward_rows_tc(ctx, ctx->target, ctx->tmaps, B, R, ub, bonus_uniform, out->status, warped || spd, s);
        if (rc != MTAD_OK) return rc;
    } else {
        int rc = forward_rows(ctx, ctx->target, B, R, ub, s);
        if (rc != MTAD_OK) return rc;
        if (!warped && !spd)
            RUN(MTAD_K_LMRED, 0, R > 1 ? 2 : 1,
                launch_lm_reduce(ctx->target, ctx->rm, ctx->sc, B, R, bonus_uniform, tok, parent, out->status, s));
    }
    if (warped)
        RUN(MTAD_K_LMRED, 0, 3,
            launch_warp_rows(ctx->target, ctx->rm, ctx->sc, B, R, ctx->warp_k, ctx->warp_p, bonus_uniform,
                             out->status, s));
    if (spd) {
        SpdArgs sa{B, R, D, tok, logq_ref, spd_accept_uniform, bonus_uniform};
        RUN(MTAD_K_ACCEPT, 0, 1, launch_spd_accept(ctx->target, ctx->rm, ctx->sc, sa, *out, s));
    } else {
        AcceptArgs aa{B, R, D, tok, parent, logq_ref, log_tau};
        RUN(MTAD_K_ACCEPT, 0, 1, launch_accept(ctx->rm, ctx->sc, aa, *out, s));
    }
    ctx->last_B = B; ctx->last_R = R; ctx->last_D = D;
    ctx->last_chain = (parent == nullptr);
    memcpy(ctx->last_seqs, seqs, sizeof(int32_t) * B);
    return MTAD_OK;
}

}  // namespace

extern "C" {

int mtad_workspace_bytes(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                         size_t* out_bytes) {
    if (!out_bytes || !model_ok(target) || (aux && !model_ok(aux))) return MTAD_E_INVALID;
    if (max_batch < 1 || max_nodes < 0) return MTAD_E_INVALID;
    if (max_batch > MTAD_MAX_BATCH || max_nodes > MTAD_MAX_NODES) return MTAD_E_CAPACITY;
    *out_bytes = carve(nullptr, target, aux, max_batch, max_nodes, nullptr);
    return MTAD_OK;
}

int mtad_create(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                void* workspace, size_t workspace_bytes, mtad_ctx** out) {
    if (!out) return MTAD_E_INVALID;
    *out = nullptr;
    size_t need = 0;
    int rc = mtad_workspace_bytes(target, aux, max_batch, max_nodes, &need);
    if (rc != MTAD_OK) return rc;
    if (!model_ptrs_ok(target) || (aux && !model_ptrs_ok(aux))) return MTAD_E_INVALID;
    if (aux && aux->vocab != target->vocab) return MTAD_E_INVALID;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return MTAD_E_WORKSPACE;
    mtad_ctx* ctx = new (std::nothrow) mtad_ctx();
    if (!ctx) return MTAD_E_INVALID;
    auto fill = [&](ModelView& v, const mtad_model_desc* m) {
        v.d = *m;
        v.lw.assign(m->layer_weights, m->layer_weights + (size_t)m->layers * MTAD_LAYER_TENSORS);
        v.d.layer_weights = v.lw.data();
        v.max_batch = max_batch;
    };
    fill(ctx->target, target);
    if (aux) { fill(ctx->aux, aux); ctx->has_aux = true; }
    ctx->max_batch = max_batch;
    ctx->max_nodes = max_nodes;
    ctx->T_max = max_batch * (max_nodes + 1);
    ctx->len_ub.assign(max_batch, 0);
    ctx->npend_ub.assign(max_batch, 1);
    carve(ctx, target, aux, max_batch, max_nodes, workspace, &ctx->regions);
    ctx->ws_base = static_cast<char*>(workspace);
    // tensor-core path unless MTAD_PATH=simt asks for the CUDA-core kernels (or a weight pointer is not 16-byte aligned)
    const char* path = getenv("MTAD_PATH");
    ctx->use_tc = !(path && strcmp(path, "simt") == 0) && build_weight_maps(ctx->target, ctx->tmaps);
    if (ctx->use_tc && aux) build_weight_maps(ctx->aux, ctx->amaps);
    if (ctx->use_tc) {
        build_kv_map(ctx->target);
        if (aux) build_kv_map(ctx->aux);
    }
    const char* pdl = getenv("MTAD_PDL");
    ctx->use_pdl = !(pdl && strcmp(pdl, "0") == 0);        // programmatic dependent launch unless MTAD_PDL=0
    cudaError_t e = cudaMemset(workspace, 0, need);
    for (const Region& r : ctx->regions)
        if (e == cudaSuccess) e = cudaMemset(ctx->ws_base + r.off + r.count * r.elem, 0xC5, kCanaryBytes);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete ctx; return MTAD_E_CUDA; }
    *out = ctx;
    return MTAD_OK;
}

int mtad_destroy(mtad_ctx* ctx) {
    if (ctx)
        for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
    delete ctx;
    return MTAD_OK;
}

int mtad_profile_begin(mtad_ctx* ctx, int max_launches) {
    if (!ctx || max_launches < 1 || max_launches > (1 << 20)) return MTAD_E_INVALID;
    while (ctx->prof_ev.size() < (size_t)max_launches * 2) {
        cudaEvent_t e;
        CU(cudaEventCreate(&e));
        ctx->prof_ev.push_back(e);
    }
    ctx->prof_cls.clear();
    ctx->prof_bytes.clear();
    ctx->prof_n.clear();
    ctx->prof_used = 0;
    ctx->prof_open = -1;
    ctx->prof_on = true;
    return MTAD_OK;
}

int mtad_profile_grouped(mtad_ctx* ctx, int on) {
    if (!ctx || ctx->prof_on) return MTAD_E_INVALID;
    ctx->prof_grouped = on != 0;
    return MTAD_OK;
}

int mtad_profile_end(mtad_ctx* ctx, double* ms, double* bytes, int64_t* launches) {
    if (!ctx || !ms || !bytes || !launches) return MTAD_E_INVALID;
    ctx->prof_on = false;
    if (ctx->prof_open >= 0) {
        CU(cudaEventRecord(ctx->prof_ev[2 * (ctx->prof_cls.size() - 1) + 1], ctx->prof_stream));
        ctx->prof_open = -1;
    }
    for (int c = 0; c < MTAD_K_CLASSES; ++c) { ms[c] = 0; bytes[c] = 0; launches[c] = 0; }
    CU(cudaDeviceSynchronize());
    for (size_t i = 0; i < ctx->prof_cls.size(); ++i) {
        float t = 0.f;
        CU(cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
        const int c = ctx->prof_cls[i];
        ms[c] += t;
        bytes[c] += ctx->prof_bytes[i];
        launches[c] += ctx->prof_n[i];
    }
    ctx->prof_used = 0;
    return MTAD_OK;
}

uint64_t mtad_kernel_launches(void) { return g_kernel_launches; }

int mtad_debug_gemm(mtad_ctx* ctx, const void* W, int N, int K, const float* x, int T, float* y, int variant,
                    void* stream) {
    if (!ctx || !W || !x || !y || N < 1 || K < 8 || (K % 8) || T < 1) return MTAD_E_INVALID;
    if (T > TC_MAX_ROWS || (size_t)2 * TC_X_ROWS * K > ctx->xf_elems) return MTAD_E_CAPACITY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TcGemmParams p{};
    const int mh = tc_halves(T);
    tc_decompose(p, (N + TC_TILE_N * mh - 1) / (TC_TILE_N * mh), K, T, kCtas);
    p.mh = mh; p.n_rows_total = N;
    if ((size_t)p.n_tiles * p.max_contrib * mh * p.rpad * TC_TILE_N > ctx->tc_ws_floats ||
        (size_t)p.n_tiles > ctx->tc_counter_n)
        return MTAD_E_WORKSPACE;
    TcMaps mp{};
    const int xbox = p.terms * p.rpad / tc_boxes(p.terms * p.rpad);
    if (tc_make_map(&mp.a0, W, N, K, mh == 1 ? 128 : 256) || tc_make_map(&mp.x, ctx->sc.xf, 2 * TC_X_ROWS, K, xbox))
        return MTAD_E_CUDA;
    p.mode = TC_PLAIN; p.N = N; p.out = y; p.ldo = N;
    p.ws = ctx->sc.tc_ws; p.counters = ctx->sc.tc_counters; p.status = nullptr;
    RUN(MTAD_K_PREPARE, 0, 1, launch_split_rows(x, K, ctx->sc.xf, p.terms, T, K, s));
    TcGemmParams q = p;
    if (variant == 1) {
        if (!tc_cluster_plan(q, (N + TC_TILE_N - 1) / TC_TILE_N, K, T, kCtas)) return MTAD_E_UNIMPLEMENTED;
        if (q.mh != mh && tc_make_map(&mp.a0, W, N, K, q.mh == 1 ? 128 : 256)) return MTAD_E_CUDA;
        RUN(MTAD_K_GEMM, 2.0 * N * K, 1, launch_tc_cluster(mp, q, false, s));
        return MTAD_OK;
    }
    if (variant != 0) return MTAD_E_INVALID;
    RUN(MTAD_K_GEMM, 2.0 * N * K, 1, launch_tc_gemm(mp, p, kCtas, false, s));
    return MTAD_OK;
}

int mtad_seq_set(mtad_ctx* ctx, int seq, int32_t kv_len, int32_t root_token, int32_t aux_len,
                 const int32_t* pending_tok, void* stream) {
    if (!ctx || seq < 0 || seq >= ctx->max_batch) return MTAD_E_INVALID;
    if (kv_len < 0 || root_token < 0 || root_token >= ctx->target.d.vocab) return MTAD_E_INVALID;
    if (kv_len > ctx->target.d.kv_capacity) return MTAD_E_CAPACITY;
    if (aux_len < 0 || aux_len > kv_len) return MTAD_E_INVALID;
    const int npend = kv_len - aux_len;
    if (npend > MTAD_MAX_DEPTH) return MTAD_E_CAPACITY;
    if (npend > 0 && !pending_tok) return MTAD_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RUN(MTAD_K_PREPARE, 0, 1, launch_seq_set(ctx->st, seq, kv_len, root_token, aux_len, npend, pending_tok, s));
    ctx->len_ub[seq] = kv_len;
    ctx->npend_ub[seq] = npend + 1;
    return MTAD_OK;
}

int mtad_set_warp(mtad_ctx* ctx, int top_k, float top_p) {
    if (!ctx || top_k < 0 || isnan(top_p) || !(top_p > 0.f) || top_p > 1.f) return MTAD_E_INVALID;
    if (top_k > MTAD_MAX_TOPK) return MTAD_E_CAPACITY;
    ctx->warp_k = top_k;
    ctx->warp_p = top_p;
    return MTAD_OK;
}

int mtad_set_draft_warp(mtad_ctx* ctx, int top_k, float top_p) {
    if (!ctx || !ctx->has_aux || top_k < 0 || isnan(top_p) || !(top_p > 0.f) || top_p > 1.f) return MTAD_E_INVALID;
    if (top_k > MTAD_MAX_TOPK) return MTAD_E_CAPACITY;
    ctx->dwarp_k = top_k;
    ctx->dwarp_p = top_p;
    return MTAD_OK;
}

int mtad_seq_hint(mtad_ctx* ctx, int seq, int32_t kv_len) {
    if (!ctx || seq < 0 || seq >= ctx->max_batch || kv_len < 0) return MTAD_E_INVALID;
    if (kv_len > ctx->target.d.kv_capacity) return MTAD_E_CAPACITY;
    ctx->len_ub[seq] = kv_len;
    return MTAD_OK;
}

int mtad_debug_check_canaries(mtad_ctx* ctx, void* stream, const char** damaged) {
    if (!ctx) return MTAD_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(cudaStreamSynchronize(s));
    unsigned char buf[kCanaryBytes];
    int bad = 0;
    for (size_t i = 0; i < ctx->regions.size(); ++i) {
        const Region& r = ctx->regions[i];
        CU(cudaMemcpy(buf, ctx->ws_base + r.off + r.count * r.elem, kCanaryBytes, cudaMemcpyDeviceToHost));
        for (size_t k = 0; k < kCanaryBytes; ++k)
            if (buf[k] != 0xC5) {
                if (!bad && damaged) *damaged = r.name;
                ++bad;
                break;
            }
    }
    return bad;
}

int mtad_debug_region(const mtad_ctx* ctx, const char* name, size_t* offset, size_t* count, size_t* elem_bytes) {
    if (!ctx || !name || !offset || !count || !elem_bytes) return MTAD_E_INVALID;
    for (const Region& r : ctx->regions)
        if (strcmp(r.name, name) == 0) {
            *offset = r.off; *count = r.count; *elem_bytes = r.elem;
            return MTAD_OK;
        }
    return MTAD_E_INVALID;
}

int mtad_debug_set_wait(mtad_ctx* ctx, unsigned int wait_limit, int no_operands) {
    if (!ctx) return MTAD_E_INVALID;
    ctx->wait_limit = wait_limit;
    ctx->debug_no_operands = no_operands ? 1 : 0;
    return MTAD_OK;
}

int mtad_seq_get(mtad_ctx* ctx, int seq, int32_t* kv_len, int32_t* root_token, void* stream) {
    if (!ctx || seq < 0 || seq >= ctx->max_batch) return MTAD_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t v[2];
    CU(cudaMemcpyAsync(&v[0], ctx->st.kv_len + seq, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(&v[1], ctx->st.root_tok + seq, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    ctx->len_ub[seq] = v[0];
    if (kv_len) *kv_len = v[0];
    if (root_token) *root_token = v[1];
    return MTAD_OK;
}

int mtad_draft(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, int beam_width, int keep_all_candidates,
               const float* uniforms, int32_t* n_nodes, int32_t* tok, int32_t* parent, int32_t* depth, float* node_logq,
               float* logq_ref, int32_t* best_path, void* stream) {
    if (!ctx) return MTAD_E_INVALID;
    if (!ctx->has_aux) return MTAD_E_INVALID;
    if (!seqs_ok(ctx, B, seqs)) return MTAD_E_INVALID;
    if (!uniforms || !tok || !parent || !depth || !node_logq || !logq_ref || !best_path) return MTAD_E_INVALID;
    if (gamma < 1 || beam_width < 1) return MTAD_E_INVALID;
    if (gamma > MTAD_MAX_DEPTH || beam_width > MTAD_MAX_BEAM || gamma * beam_width > MTAD_DRAFT_NODES - MTAD_MAX_DEPTH - 1 ||
        gamma * beam_width > MTAD_MAX_NODES)
        return MTAD_E_CAPACITY;
    const int keep_all = keep_all_candidates ? 1 : 0;
    // on warped rows a layer may hold fewer nodes than the beam width: the caller needs the count
    const bool dwarp = ctx->dwarp_k > 0;
    if (dwarp && !n_nodes) return MTAD_E_INVALID;
    // the caller's tree: beam_width * beam_width nodes a layer with every candidate kept (a verify call takes
    // MTAD_MAX_NODES at most), and a layer can only be filled from a vocabulary that large
    if (keep_all && (gamma * beam_width * beam_width > MTAD_MAX_NODES || ctx->aux.d.vocab < beam_width * beam_width))
        return MTAD_E_CAPACITY;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const ModelView& m = ctx->aux;
    int R0 = 1;
    long long ub = 0;
    for (int i = 0; i < B; ++i) {
        R0 = std::max(R0, ctx->npend_ub[seqs[i]]);
        ub = std::max(ub, ctx->len_ub[seqs[i]]);
    }
    if (std::max(R0, beam_width) > ctx->max_nodes + 1) return MTAD_E_CAPACITY;    // rows of one step exceed the workspace
    if (ub + 1 + (long long)gamma * beam_width > m.d.kv_capacity) return MTAD_E_CAPACITY;
    SeqList sl{};
    for (int i = 0; i < B; ++i) sl.v[i] = seqs[i];
    DraftOut out{n_nodes, tok, parent, depth, node_logq, logq_ref, best_path};
    const bool tc = ctx->use_tc && ctx->amaps.ok;
    CU(cudaMemsetAsync(ctx->sc.tc_counters, 0, sizeof(int32_t) * ctx->tc_counter_n, s));
    for (int step = 0; step < gamma; ++step) {
        const int R = step == 0 ? R0 : beam_width;
        RUN(MTAD_K_PREPARE, 0, 1, launch_draft_prepare(m, ctx->st, ctx->ds, ctx->rm, ctx->sc, sl, B, R, step, beam_width,
                                                       tc && B * R <= TC_MAX_ROWS, dwarp, ctx->use_pdl, s));
        // keys of the auxiliary cache: committed ones, the pending rows and every node drafted so far
        const long long keys_ub = ub + 1 + (long long)step * beam_width;
        int rc;
        if (tc && B * R <= TC_MAX_ROWS) rc = forward_rows_tc(ctx, m, ctx->amaps, B, R, keys_ub, nullptr, nullptr, true, s);
        else rc = forward_rows(ctx, m, B, R, keys_ub, s);
        if (rc != MTAD_OK) return rc;
        if (dwarp) {
            // warped rows (kept tokens and their renormalised log-probabilities), then the selection over those
            RUN(MTAD_K_LMRED, 0, 2, launch_warp_rows_only(m, ctx->rm, ctx->sc, B, R, ctx->dwarp_k, ctx->dwarp_p, uniforms, s));
            RUN(MTAD_K_LMRED, 0, 1, launch_draft_select_warped(m, ctx->ds, ctx->sc, sl, B, R, step, gamma, beam_width,
                                                               keep_all, uniforms, out, s));
            continue;
        }
        RUN(MTAD_K_LMRED, 0, 2, launch_draft_select(m, ctx->ds, ctx->sc, sl, B, R, step, gamma, beam_width, keep_all, uniforms, out,
                                                     ctx->use_pdl, s));
    }
    ctx->draft_active = true;
    ctx->draft_B = B;
    ctx->draft_gamma = gamma;
    memcpy(ctx->draft_seqs, seqs, sizeof(int32_t) * B);
    return MTAD_OK;
}

int mtad_verify_chain(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, const int32_t* draft_tok,
                      const float* draft_logq, float log_tau, const float* bonus_uniform,
                      const mtad_result* out, void* stream) {
    // a chain is the tree parent[n] = n - 1; node j has depth j + 1, so log q(x**_{1:j+1}) = draft_logq[j]
    return verify_common(ctx, B, seqs, nullptr, gamma, gamma, draft_tok, nullptr, draft_logq, log_tau,
                         bonus_uniform, out, stream);
}

int mtad_verify_chain_spd(mtad_ctx* ctx, int B, const int32_t* seqs, int gamma, const int32_t* draft_tok,
                          const float* draft_logq_rows, const float* accept_uniform, const float* resample_uniform,
                          const mtad_result* out, void* stream) {
    if (gamma < 1 || !accept_uniform || !draft_logq_rows) return MTAD_E_INVALID;
    return verify_common(ctx, B, seqs, nullptr, gamma, gamma, draft_tok, nullptr, draft_logq_rows, -1.f,
                         resample_uniform, out, stream, accept_uniform);
}

int mtad_verify_tree(mtad_ctx* ctx, int B, const int32_t* seqs, const int32_t* n_nodes, int max_nodes,
                     int max_depth, const int32_t* tok, const int32_t* parent, const float* logq_ref,
                     float log_tau, const float* bonus_uniform, const mtad_result* out, void* stream) {
    if (max_nodes > 0 && !parent) return MTAD_E_INVALID;
    return verify_common(ctx, B, seqs, n_nodes, max_nodes, max_depth, tok, parent, logq_ref, log_tau,
                         bonus_uniform, out, stream);
}

int kv_commit(mtad_ctx* ctx, int B, const int32_t* seqs, const mtad_result* res, void* stream) {
    if (!ctx || !result_ok(res)) return MTAD_E_INVALID;
    if (!seqs_ok(ctx, B, seqs)) return MTAD_E_INVALID;
    if (B != ctx->last_B || memcmp(seqs, ctx->last_seqs, sizeof(int32_t) * B) != 0) return MTAD_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (ctx->has_aux) {
        // auxiliary cache: after a draft its accepted rows are kept; otherwise the accepted tokens wait for replay
        const bool after_draft = ctx->draft_active && ctx->draft_B == B &&
                                 memcmp(seqs, ctx->draft_seqs, sizeof(int32_t) * B) == 0;
        const int mode = after_draft ? (ctx->last_chain ? 0 : 1) : 2;
        RUN(MTAD_K_COMMIT, 0, 2,
            launch_aux_commit(ctx->aux, ctx->st, ctx->ds, B, ctx->rm.call_seq, *res, ctx->last_D, mode, s));
        for (int i = 0; i < B; ++i)
            ctx->npend_ub[seqs[i]] = after_draft ? 2 : std::min(ctx->npend_ub[seqs[i]] + ctx->last_D + 1, MTAD_MAX_DEPTH + 1);
        ctx->draft_active = false;
    }
    RUN(MTAD_K_COMMIT, 0, 1, launch_kv_commit(ctx->target, ctx->st, B, ctx->rm.call_seq, *res, ctx->last_D, s));
    RUN(MTAD_K_COMMIT, 0, 1, launch_seq_advance(ctx->st, B, ctx->rm.call_seq, *res, ctx->last_D, ctx->max_batch,
                                              (long long)ctx->target.d.kv_capacity, s));
    for (int i = 0; i < B; ++i)
        ctx->len_ub[seqs[i]] = std::min<long long>(ctx->len_ub[seqs[i]] + ctx->last_D + 1, ctx->target.d.kv_capacity);
    ctx->last_B = 0;
    return MTAD_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Extent audit: for one call shape, the largest element index that the call's kernels form into every array of the
// workspace, into the KV caches and into the caller's arrays, next to how many elements the array holds.  Host
// arithmetic only (no device, no driver): the launch plans are the ones the calls use, the index expressions are the
// kernels' own helpers (idx_*), evaluated at the largest row, head, tile and split of the launch.
// ---------------------------------------------------------------------------------------------------------------
namespace {

struct Audit {
    std::vector<Region> regions;
    std::vector<mtad_extent> out;
    size_t region_count(const char* name) const {
        for (const Region& r : regions)
            if (strcmp(r.name, name) == 0) return r.count;
        return 0;
    }
    void ws(const char* name, size_t reach) { out.push_back({name, (int64_t)reach, (int64_t)region_count(name)}); }
    void ext(const char* name, size_t reach, size_t extent) { out.push_back({name, (int64_t)reach, (int64_t)extent}); }
};

// one decoder forward of B * R rows of model m on the tensor-core path: the prepared rows, every GEMM launch of the
// plan, the attention passes and the LM-head reductions
void audit_forward(Audit& au, const mtad_ctx& c, const ModelView& m, int B, int R, long long len_ub, bool lm_plain,
                   const char* cache_name) {
    const mtad_model_desc& d = m.d;
    const int T = B * R, hd = d.head_dim, Hq = d.n_q_heads, Hkv = d.n_kv_heads;
    const size_t qd = (size_t)Hq * hd;
    const int terms = tc_terms(T);
    // row preparation: row metadata, residual stream, rotary table, first operand rows and their statistics
    for (const char* n : {"rm_tok", "rm_pos", "rm_slot", "rm_seq", "rm_depth", "rm_prow", "node_lp", "row_lse", "row_cand",
                          "row_cand_lp", "node_z"})
        au.ws(n, T);
    au.ws("rm_mask", (size_t)T * MTAD_MASK_WORDS);
    for (const char* n : {"rm_n_rows", "rm_n_spec", "rm_kv_base", "rm_call_seq"}) au.ws(n, B);
    au.ws("hidden", (size_t)T * d.d_model);
    au.ws("rope", ((size_t)(T - 1) * (hd / 2) + (hd / 2 - 1)) * 2 + 2);
    au.ws("xd", idx_xrow(T - 1, terms, terms - 1, d.d_model, d.d_model - 1) + 1);
    au.ws("sumsq_a", T);
    ForwardPlan fp;
    build_plan(fp, c.sc, c.rm, m, nullptr, B, R, lm_plain, false, &m == &c.target);
    if (fp.split_kv) au.ws("xkv", idx_xrow(T - 1, fp.kv_terms, fp.kv_terms - 1, d.d_model, d.d_model - 1) + 1);
    const long long cap = d.kv_capacity;
    const long long slot_max = std::min<long long>(len_ub + R - 1, cap - 1);     // prepare refuses rows past the capacity
    const size_t cache_elems = (size_t)d.layers * m.max_batch * 2 * Hkv * cap * hd;
    for (const GemmDesc& gd : fp.g) {
        const TcGemmParams& p = gd.p;
        if (!gd.cluster) {
            // split-K partial tiles: the last tile's last contributor, last half, last row, last feature
            const size_t part_floats = (size_t)p.mh * p.rpad * TC_TILE_N;
            au.ws("tc_ws", idx_tc_ws(p.n_tiles - 1, p.max_contrib, p.max_contrib - 1, part_floats) + part_floats);
            au.ws("tc_counters", p.n_tiles);
        }
        const int t128_last = p.mode == TC_SWIGLU ? 0 : (p.n_rows_total + TC_TILE_N - 1) / TC_TILE_N - 1;
        switch (p.mode) {
            case TC_QKV:
                au.ws("qkv", (size_t)(T - 1) * (Hq + 2 * Hkv) * hd + qd);
                au.ws("q_hi", (size_t)T * qd);
                au.ws("q_lo", (size_t)T * qd);
                au.ext(cache_name, idx_cache(p.layer, m.max_batch, m.max_batch - 1, 1, Hkv, Hkv - 1, cap, slot_max, hd) + hd,
                       cache_elems);
                break;
            case TC_RESID:
                au.ws("hidden", (size_t)(T - 1) * p.N + p.N);
                au.ws(p.x_out == c.sc.xd ? "xd" : "xf", idx_xrow(T - 1, p.out_terms, p.out_terms - 1, p.xk, p.N - 1) + 1);
                au.ws(p.sumsq_out == c.sc.sumsq_a ? "sumsq_a" : "sumsq_b", (size_t)t128_last * TC_X_ROWS + T);
                break;
            case TC_SWIGLU:
                au.ws("xf", idx_xrow(T - 1, terms, terms - 1, p.xk, p.N - 1) + 1);
                break;
            case TC_PLAIN:
                au.ws("logits", (size_t)(T - 1) * p.ldo + p.N);
                break;
            default:
                au.ws("lm_part", idx_lm_part(T - 1, p.n_tiles128, p.n_tiles128 - 1) + 1);
                break;
        }
        if (p.sumsq_in_parts > 0)
            au.ws(p.sumsq_in == c.sc.sumsq_a ? "sumsq_a" : "sumsq_b", (size_t)(p.sumsq_in_parts - 1) * TC_X_ROWS + T);
    }
    // attention: split-KV partials of the last row, head and split; combined rows and the O projection's operand rows
    const long long total = std::min<long long>(len_ub, cap) + R;
    const AttnSplit as = attn_split(m, B, R, total);
    au.ws("attn_part", idx_attn_part(T - 1, Hq, Hq - 1, as.ns, as.ns - 1, hd) + hd + 2);
    au.ws("attn", (size_t)T * qd);
    au.ws("xa", idx_xrow(T - 1, terms, terms - 1, qd, qd - 1) + 1);
    // the K/V tiles come by TMA from a map over [layers * max_batch * 2 * Hkv planes][cap][hd]: the last plane asked for
    au.ext("kv_map_planes", (size_t)((d.layers - 1) * m.max_batch + (m.max_batch - 1)) * 2 * Hkv + 2 * Hkv,
           (size_t)d.layers * m.max_batch * 2 * Hkv);
}

}  // namespace

int mtad_audit_extents(const mtad_model_desc* target, const mtad_model_desc* aux, int max_batch, int max_nodes,
                       int call, int B, int nodes, int gamma, int beam, int64_t len_ub, mtad_extent* out,
                       int max_out, int* n_out) {
    if (!out || !n_out || max_out < 0 || !model_ok(target) || (aux && !model_ok(aux))) return MTAD_E_INVALID;
    if (max_batch < 1 || max_batch > MTAD_MAX_BATCH || max_nodes < 0 || max_nodes > MTAD_MAX_NODES) return MTAD_E_INVALID;
    if (B < 1 || B > max_batch || nodes < 0 || nodes > max_nodes || len_ub < 0) return MTAD_E_INVALID;
    if ((call == MTAD_AUDIT_DRAFT || (call == MTAD_AUDIT_COMMIT && aux)) && (gamma < 1 || beam < 1)) return MTAD_E_INVALID;
    if (call == MTAD_AUDIT_DRAFT && !aux) return MTAD_E_INVALID;
    mtad_ctx c;
    Audit au;
    auto fill = [&](ModelView& v, const mtad_model_desc* m) {
        v.d = *m;
        v.lw.assign((size_t)m->layers * MTAD_LAYER_TENSORS, nullptr);
        v.d.layer_weights = v.lw.data();
        v.max_batch = max_batch;
    };
    fill(c.target, target);
    if (aux) { fill(c.aux, aux); c.has_aux = true; }
    c.max_batch = max_batch; c.max_nodes = max_nodes;
    carve(&c, target, aux, max_batch, max_nodes, nullptr, &au.regions);
    const int D = gamma > 0 ? gamma : 1;
    if (call == MTAD_AUDIT_VERIFY) {
        const int R = nodes + 1;
        if (B * R > TC_MAX_ROWS) return MTAD_E_CAPACITY;
        audit_forward(au, c, c.target, B, R, len_ub, false, "target_cache");
        // caller's arrays: inputs [B, nodes], logq_ref [B, D], uniforms [B, V], results as documented in mtad_result
        au.ext("tok/parent (caller)", (size_t)(B - 1) * nodes + nodes, (size_t)B * nodes);
        au.ext("logq_ref (caller)", (size_t)(B - 1) * D + D, (size_t)B * D);
        au.ext("bonus_uniform (caller)", (size_t)(B - 1) * target->vocab + target->vocab, (size_t)B * target->vocab);
        au.ext("result.path", (size_t)(B - 1) * D + D, (size_t)B * D);
        au.ext("result.out_tok/out_lp", (size_t)(B - 1) * (D + 1) + D + 1, (size_t)B * (D + 1));
        au.ext("result.node_lp/node_LP", (size_t)(B - 1) * nodes + nodes, (size_t)B * nodes);
        au.ext("result.row_*", (size_t)(B - 1) * R + R, (size_t)B * R);
        au.ext("embed rows (target)", (size_t)(target->vocab - 1) * target->d_model + target->d_model,
               (size_t)target->vocab * target->d_model);
    } else if (call == MTAD_AUDIT_DRAFT) {
        if (gamma > MTAD_MAX_DEPTH || beam > MTAD_MAX_BEAM || gamma * beam > MTAD_DRAFT_NODES - MTAD_MAX_DEPTH - 1)
            return MTAD_E_CAPACITY;
        const int V = aux->vocab;
        int nch = (V + 1023) / 1024;
        nch = nch < 1 ? 1 : (nch > MTAD_DRAFT_CHUNKS ? MTAD_DRAFT_CHUNKS : nch);
        const int P_max = MTAD_MAX_DEPTH + 1;
        for (int step = 0; step < gamma; ++step) {
            // step 0 replays up to `nodes + 1` pending rows (the caller's bound of the pending list), later steps run
            // the beam nodes of a layer
            const int R = step == 0 ? std::min(nodes + 1, P_max) : beam;
            if (B * R > TC_MAX_ROWS) return MTAD_E_CAPACITY;
            audit_forward(au, c, c.aux, B, R, len_ub + 1 + (long long)step * beam, true, "aux_cache");
            // selection: per-chunk parts of every beam row, the draft state of the sequence with the largest id
            au.ws("draft_part", ((size_t)((B - 1) * MTAD_MAX_BEAM + (step == 0 ? 0 : beam - 1))) * nch + nch);
            const size_t n_last = (size_t)step * beam + beam - 1;
            au.ws("ds_node_tok", (size_t)(max_batch - 1) * MTAD_DRAFT_NODES + n_last + 1);
            au.ws("ds_node_parent", (size_t)(max_batch - 1) * MTAD_DRAFT_NODES + n_last + 1);
            au.ws("ds_node_logq", (size_t)(max_batch - 1) * MTAD_DRAFT_NODES + n_last + 1);
            au.ws("ds_node_mask", ((size_t)(max_batch - 1) * MTAD_DRAFT_NODES + n_last) * MTAD_MASK_WORDS + MTAD_MASK_WORDS);
            au.ws("ds_tree_id", (size_t)(max_batch - 1) * MTAD_DRAFT_NODES + n_last + 1);
            au.ws("ds_nb", (size_t)(max_batch - 1) * MTAD_MAX_DEPTH + step + 1);
            au.ws("ds_n_tree", (size_t)max_batch);
            // on warped rows the selection ranks beam x MTAD_MAX_TOPK pairs held in shared memory
            au.ext("warped selection candidates (shared memory)", (size_t)beam * MTAD_MAX_TOPK,
                   (size_t)MTAD_MAX_BEAM * MTAD_MAX_TOPK);
            au.ws("warp_row", (size_t)B * R);
            // node ids of the caller's tree: beam per layer, or beam * beam with every candidate kept (when that fits a
            // verify call); the selection holds the chunks' candidates of all beam rows in shared memory
            const size_t per_layer = gamma * beam * beam <= MTAD_MAX_NODES ? (size_t)beam * beam : (size_t)beam;
            au.ws("ds_tree2slot", (size_t)(max_batch - 1) * MTAD_DRAFT_NODES + step * per_layer + per_layer);
            au.ext("selection candidates (shared memory)",
                   (size_t)(step == 0 ? 1 : beam) * nch * (step == 0 ? per_layer : (size_t)beam),
                   (size_t)MTAD_MAX_BEAM * MTAD_DRAFT_CHUNKS * MTAD_MAX_BEAM);
            // a node's mask bit: virtual row P + n, below MTAD_MASK_WORDS * 32
            au.ext("mask bits (virtual rows)", (size_t)R + n_last + 1 + (step == 0 ? 0 : P_max), (size_t)MTAD_MASK_WORDS * 32);
            au.ext("uniforms (caller)", (((size_t)(B - 1) * gamma + step) * beam + (step == 0 ? 0 : beam - 1)) * V + V,
                   (size_t)B * gamma * beam * V);
        }
        au.ws("ds_best_path", (size_t)(max_batch - 1) * MTAD_MAX_DEPTH + gamma);
        au.ws("st_aux_pend", (size_t)(max_batch - 1) * (MTAD_MAX_DEPTH + 1) + P_max);
        au.ext("tok/parent/depth/node_logq (caller)", (size_t)(B - 1) * gamma * beam + gamma * beam, (size_t)B * gamma * beam);
        au.ext("logq_ref/best_path (caller)", (size_t)(B - 1) * gamma + gamma, (size_t)B * gamma);
        // auxiliary cache slots: committed length + pending rows + every node
        au.ext("aux cache slots", (size_t)len_ub + 1 + (size_t)gamma * beam, (size_t)aux->kv_capacity);
    } else if (call == MTAD_AUDIT_COMMIT) {
        const mtad_model_desc& t = *target;
        const long long L1 = std::min<long long>(len_ub + 1 + nodes, t.kv_capacity);     // one past the last row moved
        au.ext("target_cache", idx_cache(t.layers - 1, max_batch, max_batch - 1, 1, t.n_kv_heads, t.n_kv_heads - 1,
                                         t.kv_capacity, L1 - 1, t.head_dim) + t.head_dim,
               (size_t)t.layers * max_batch * 2 * t.n_kv_heads * t.kv_capacity * t.head_dim);
        au.ext("commit staging (shared memory, bf16)", (size_t)D * t.head_dim, (size_t)D * t.head_dim);
        au.ext("result.path", (size_t)(B - 1) * D + D, (size_t)B * D);
        if (aux) {
            const mtad_model_desc& a = *aux;
            const long long last = len_ub + 1 + (long long)gamma * beam - 1;               // slot of the last draft node
            au.ext("aux_cache", idx_cache(a.layers - 1, max_batch, max_batch - 1, 1, a.n_kv_heads, a.n_kv_heads - 1,
                                          a.kv_capacity, last, a.head_dim) + a.head_dim,
                   (size_t)a.layers * max_batch * 2 * a.n_kv_heads * a.kv_capacity * a.head_dim);
            au.ws("ds_best_path", (size_t)(max_batch - 1) * MTAD_MAX_DEPTH + gamma);
            au.ws("st_aux_pend", (size_t)(max_batch - 1) * (MTAD_MAX_DEPTH + 1) + 2);
        }
    } else {
        return MTAD_E_INVALID;
    }
    *n_out = (int)au.out.size();
    for (int i = 0; i < *n_out && i < max_out; ++i) out[i] = au.out[i];
    return MTAD_OK;
}

const char* mtad_status_str(int status) {
    switch (status) {
        case MTAD_OK: return "ok";
        case MTAD_E_INVALID: return "invalid argument";
        case MTAD_E_CAPACITY: return "capacity exceeded";
        case MTAD_E_CUDA: return "CUDA error";
        case MTAD_E_TIMEOUT: return "device wait timed out";
        case MTAD_E_UNIMPLEMENTED: return "not implemented";
        case MTAD_E_WORKSPACE: return "workspace missing, misaligned or too small";
        default: return "unknown status";
    }
}

int mtad_last_cuda_error(const mtad_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

}  // extern "C"
