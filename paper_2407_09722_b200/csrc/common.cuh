// Internal declarations shared by the host dispatcher and the kernel translation units.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "mtad.h"

#define MTAD_MASK_WORDS 8          // ancestor bitmask words per row (rows per sequence <= 256)
#define MTAD_ATTN_TILE 64          // keys staged per attention tile
#define MTAD_ROW_CHUNK 8           // rows per GEMM / attention pass in the CUDA-core kernels

namespace mtad {

// Per-call view of the rows (device arrays inside the workspace). Global row t = bi * R + r.
struct RowMeta {
    int32_t* tok;        // [T]
    int32_t* pos;        // [T] rotary position
    int32_t* slot;       // [T] cache slot, -1 = row inactive (padding, rejected sequence)
    int32_t* seq;        // [T] sequence id
    int32_t* depth;      // [T]
    uint32_t* mask;      // [T][MTAD_MASK_WORDS] visible rows of the same sequence (ancestors and self)
    int32_t* n_rows;     // [B] active rows of sequence bi (n_nodes + 1, 0 if the sequence is rejected)
    int32_t* n_spec;     // [B] cache slots past L that hold draft rows (this call's and, in the draft, earlier steps')
    int32_t* kv_base;    // [B] committed length L seen by this call
    int32_t* call_seq;   // [B] sequence ids of the call
    int32_t* prow;       // [T] global row of a node row's parent, -1 for roots and inactive rows
};

struct ModelView {
    mtad_model_desc d;
    std::vector<const void*> lw;   // layers * 9 device pointers
    int max_batch;
    CUtensorMap kv_map;            // KV cache as (head_dim, position, plane = ((layer, sequence), K|V, KV head)), boxes of 64 x 64
    bool kv_map_ok = false;
    const __nv_bfloat16* w(int layer, int which) const {
        return static_cast<const __nv_bfloat16*>(lw[(size_t)layer * MTAD_LAYER_TENSORS + which]);
    }
};

struct SeqState {        // device arrays, [max_batch]
    int32_t* kv_len;
    int32_t* root_tok;
    int32_t* aux_len;
    int32_t* aux_npend;
    int32_t* aux_pend;   // [max_batch][MTAD_MAX_DEPTH + 1]
};

#define MTAD_DRAFT_NODES 256       // nodes of one draft tree kept per sequence

// State of the last draft of every sequence (device arrays indexed by sequence id), kept for the cache roll-forward.
struct DraftState {
    int32_t* base_len;     // [max_batch] auxiliary committed length when the draft started
    int32_t* npend;        // [max_batch] pending tokens replayed by that draft
    int32_t* gamma;        // [max_batch]
    int32_t* beam;         // [max_batch]
    int32_t* node_tok;     // [max_batch][MTAD_DRAFT_NODES]
    int32_t* node_parent;  // [max_batch][MTAD_DRAFT_NODES]
    float* node_logq;      // [max_batch][MTAD_DRAFT_NODES]
    uint32_t* node_mask;   // [max_batch][MTAD_DRAFT_NODES][MTAD_MASK_WORDS] visible virtual rows of each node
    int32_t* best_path;    // [max_batch][MTAD_MAX_DEPTH] beam slots of x** (slot = layer * beam + rank)
    // The nodes above are the beams (the rows the auxiliary model runs), indexed by beam slot.  The tree handed to the
    // caller may hold more (mtad_draft with keep_all_candidates): these map between the two numberings.
    int32_t* tree_id;      // [max_batch][MTAD_DRAFT_NODES] beam slot -> node id in the caller's tree
    int32_t* tree2slot;    // [max_batch][MTAD_DRAFT_NODES] node id in the caller's tree -> beam slot, -1: not a beam
    // Beams kept per step (the beam width, or fewer when the warped rows of a step keep fewer (beam, token) pairs)
    // and the nodes written to the caller's tree so far.
    int32_t* nb;           // [max_batch][MTAD_MAX_DEPTH]
    int32_t* n_tree;       // [max_batch]
};

struct DraftOut {          // caller's device arrays of mtad_draft
    int32_t* n_nodes;      // [B] or null
    int32_t *tok, *parent, *depth;
    float* node_logq;
    float* logq_ref;
    int32_t* best_path;
};

#define MTAD_DRAFT_CHUNKS 32       // vocabulary chunks of one beam row in the draft's selection (at most)

// What one chunk of a beam row hands to the draft's selection: its share of the row's log-sum-exp and its largest
// perturbed logits (token -1: none).
#define MTAD_MAX_CAND (MTAD_MAX_BEAM * MTAD_MAX_BEAM)   // candidates of one beam row kept per chunk (at most)
struct DraftPart {
    float m, s;
    float t[MTAD_MAX_CAND];
    int32_t v[MTAD_MAX_CAND];
};

#define MTAD_MAX_TOPK 16           // largest top-k of the warped rows

// Warped rows: a chunk's largest logits (token -1: none), and a row's kept tokens with their log-probabilities
struct WarpPart {
    float z[MTAD_MAX_TOPK];
    int32_t v[MTAD_MAX_TOPK];
};
struct WarpRow {
    int32_t n;
    int32_t idx[MTAD_MAX_TOPK];
    float lp[MTAD_MAX_TOPK];
};

struct Scratch {
    float* hidden;       // [T, d]
    float* xn;           // [T, d]
    float* qkv;          // [T, (Hq + 2 Hkv) hd]
    float* attn;         // [T, Hq hd]
    float* act;          // [T, F]
    float* rope;         // [T, hd/2, 2]
    float* attn_part;    // [T, Hq, nsplit, hd + 2]
    __nv_bfloat16 *q_hi, *q_lo;   // [T, Hq hd] query rows as bf16 hi / lo (tensor-core attention operands)
    float* logits;       // [T, V]
    float* node_lp;      // [T]
    float* row_lse;      // [T]
    int32_t* row_cand;   // [T]
    float* row_cand_lp;  // [T]
    // tensor-core path: bf16 operand rows (see store_terms), deferred-norm statistics, split-K workspace, LM-head
    // partials
    __nv_bfloat16* xd;   // [512, d]     input of QKV / gate-up / LM head (un-normalised hidden * gain)
    __nv_bfloat16* xa;   // [512, Hq hd] attention output
    __nv_bfloat16* xf;   // [512, F]     SwiGLU output
    __nv_bfloat16* xkv;  // [512, d]     input of a separate K/V projection (three terms), see build_plan
    float* sumsq_a;      // [tiles(d)][256] sums of squares of the hidden rows (after down proj / embedding)
    float* sumsq_b;      // [tiles(d)][256] the same after the O projection
    float* tc_ws;        // split-K partial tiles
    int32_t* tc_counters;
    float4* lm_part;     // [T][tiles(V)]
    float* node_z;       // [T]
    DraftPart* draft_part;   // [max_batch][MTAD_MAX_BEAM][MTAD_DRAFT_CHUNKS], only with an auxiliary model
    WarpPart* warp_part;     // [T][MTAD_DRAFT_CHUNKS]
    WarpRow* warp_row;       // [T]
};

// ---- index arithmetic used by the kernels and, on the host, by the extent audit (mtad_audit_extents) -----------
// first element of position `pos` of (layer, sequence, K|V, KV head) in a cache [layer][max_batch][2][Hkv][cap][hd]
__host__ __device__ inline size_t idx_cache(long long layer, long long max_batch, long long seq, int kv, long long Hkv,
                                            long long head, long long cap, long long pos, long long hd) {
    return (size_t)((((((layer * max_batch + seq) * 2 + kv) * Hkv + head) * cap) + pos) * hd);
}
// split-KV partial (m, l, o[hd]) of row t, head h, split sp
__host__ __device__ inline size_t idx_attn_part(long long t, long long Hq, long long h, long long nsplit, long long sp,
                                                long long hd) {
    return (size_t)((((t * Hq + h) * nsplit) + sp) * (hd + 2));
}
// term j of element k of activation row t in an operand-row buffer of row length K
__host__ __device__ inline size_t idx_xrow(long long t, long long terms, long long j, long long K, long long k) {
    return (size_t)((t * terms + j) * K + k);
}
// LM-head partial of (row t, 128-token tile)
__host__ __device__ inline size_t idx_lm_part(long long t, long long n_tiles, long long tile) {
    return (size_t)(t * n_tiles + tile);
}
// split-K partial tile of (tile, contributor): part_floats floats each
__host__ __device__ inline size_t idx_tc_ws(long long tile, long long max_contrib, long long contrib, long long part_floats) {
    return (size_t)((tile * max_contrib + contrib) * part_floats);
}

inline int attn_split_cap(int n_q_heads) {
    int s = (4 * 148 + n_q_heads - 1) / n_q_heads;
    return s < 1 ? 1 : (s > 32 ? 32 : s);
}

// Launch with the programmatic-dependent-launch attribute: the kernel may start while its predecessor in the stream
// is still draining; it must execute griddepcontrol.wait before it touches anything the predecessor writes.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                              Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// An fp32 activation enters the tensor-core GEMM as `terms` bf16 values whose sum is the activation to ~2^-17
// relative (two terms) or to fp32 rounding (three).  The terms of row t are neighbouring rows of the operand
// buffer: term j of element k lives at x[(t * terms + j) * K + k].
int tc_terms(int T);       // terms used for a call of T rows: 3 up to 32 rows, else 2
// Terms of the rows that feed the Q/K/V projection (and the LM head): three whenever their accumulator columns fit
// tensor memory (up to 160 rows).  K and V are rounded to bf16 for the cache, and every element that rounds the other
// way than the exact value would shifts attention scores of later rows; with two terms (2.5e-6 relative error) a few
// tenths of a percent of the elements do, with three (2.5e-7) ten times fewer.
int tc_qkv_terms(int T);
__device__ __forceinline__ void store_terms(float y, __nv_bfloat16* x, size_t K, int terms) {
    const __nv_bfloat16 h = __float2bfloat16_rn(y);
    x[0] = h;
    const float r = y - __bfloat162float(h);
    const __nv_bfloat16 l = __float2bfloat16_rn(r);
    x[K] = l;
    if (terms == 3) x[2 * K] = __float2bfloat16_rn(r - __bfloat162float(l));
}

// One embedding row -> the fp32 hidden row and (tensor-core path) its bf16 operand terms times the first norm's gain;
// returns this thread's share of the row's sum of squares.  16-byte loads, four in flight per thread: a scalar loop
// whose loads wait behind the previous iteration's stores pays one DRAM latency per element (32 us for a 4096-wide
// row).  d is a multiple of 8; rows that are not 16-byte aligned take the scalar loop.
__device__ __forceinline__ float embed_row(const __nv_bfloat16* __restrict__ src_row, bool ok, int d,
                                           float* __restrict__ hidden_row, const __nv_bfloat16* __restrict__ gain,
                                           __nv_bfloat16* x_row, int terms) {
    float ss = 0.f;
    const bool vec = ((reinterpret_cast<uintptr_t>(src_row) | reinterpret_cast<uintptr_t>(hidden_row) |
                       reinterpret_cast<uintptr_t>(gain) | reinterpret_cast<uintptr_t>(x_row)) & 15) == 0;
    if (!vec) {
        for (int i = threadIdx.x; i < d; i += blockDim.x) {
            const float v = ok ? __bfloat162float(src_row[i]) : 0.f;
            hidden_row[i] = v;
            if (x_row) {
                store_terms(v * __bfloat162float(gain[i]), x_row + i, d, terms);
                ss += v * v;
            }
        }
        return ss;
    }
    const int nv = d >> 3;
    const uint4* src = reinterpret_cast<const uint4*>(src_row);
    const uint4* gsrc = reinterpret_cast<const uint4*>(gain);
    for (int c0 = threadIdx.x; c0 < nv; c0 += 4 * blockDim.x) {
        uint4 q[4], gq[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c = c0 + k * blockDim.x;
            q[k] = (ok && c < nv) ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
            gq[k] = (x_row && c < nv) ? __ldg(gsrc + c) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c = c0 + k * blockDim.x;
            if (c >= nv) continue;
            const uint32_t w[4] = {q[k].x, q[k].y, q[k].z, q[k].w}, gw[4] = {gq[k].x, gq[k].y, gq[k].z, gq[k].w};
            float v[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                v[2 * e] = __uint_as_float(w[e] << 16);
                v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
            float4* h4 = reinterpret_cast<float4*>(hidden_row + (size_t)c * 8);
            h4[0] = make_float4(v[0], v[1], v[2], v[3]);
            h4[1] = make_float4(v[4], v[5], v[6], v[7]);
            if (x_row) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    store_terms(v[2 * e] * __uint_as_float(gw[e] << 16), x_row + (size_t)c * 8 + 2 * e, d, terms);
                    store_terms(v[2 * e + 1] * __uint_as_float(gw[e] & 0xffff0000u), x_row + (size_t)c * 8 + 2 * e + 1, d,
                                terms);
                    ss += v[2 * e] * v[2 * e] + v[2 * e + 1] * v[2 * e + 1];
                }
            }
        }
    }
    return ss;
}

// Rotary frequencies base^(-2i/hd), i < hd/2, computed once on the host in double and passed to the kernels that
// build a call's rotary table; the angle pos * frequency is reduced to [-pi, pi] in double (a few fused
// multiply-adds) and its sine and cosine taken in fp32: double-precision sincos of an unreduced angle was most of
// the row-preparation kernels' time.
struct RopeInv {
    double v[64];
};
inline RopeInv rope_inv(double base, int hd) {
    RopeInv r{};
    for (int i = 0; i < hd / 2 && i < 64; ++i) r.v[i] = exp2(-(2.0 * i / hd) * log2(base));
    return r;
}
__device__ __forceinline__ void rope_cs(double pos, double inv, float& cs, float& sn) {
    const double x = pos * inv;
    const double k = rint(x * 0.15915494309189535);
    double r = fma(-k, 6.283185307179586, x);
    r = fma(-k, 2.4492935982947064e-16, r);
    sincosf((float)r, &sn, &cs);
}

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- launchers (each enqueues on `st`, returns the launch error) -------------------------------------------------

struct SeqList {
    int32_t v[MTAD_MAX_BATCH];
};

struct PrepareArgs {
    SeqList seqs;              // sequence ids of the call, by value
    int B, R, max_depth;
    const int32_t* n_nodes;    // device [B] or nullptr (all sequences have R-1 nodes)
    const int32_t* tok;        // device [B, R-1]
    const int32_t* parent;     // device [B, R-1] or nullptr (chain)
    // tensor-core path (null otherwise): first layer's norm gains, operand rows and row statistics to emit
    const __nv_bfloat16* gain0;
    __nv_bfloat16* x;
    int terms;
    __nv_bfloat16* x2;         // second copy of the operand rows with terms2 terms, or null
    int terms2;
    float* sumsq_out;
};

cudaError_t launch_prepare(const ModelView& m, const SeqState& s, const RowMeta& rm, const Scratch& sc,
                           const PrepareArgs& a, uint32_t* status, cudaStream_t st);
cudaError_t launch_rmsnorm(const float* x, const __nv_bfloat16* gain, float* y, int T, int d, float eps,
                           cudaStream_t st);
// y[t, col0 + n] (=|+=) sum_k x[t,k] W[n,k];  mode 0 store, 1 add into y, 2 SwiGLU with W2 (y = silu(xW^T) * (xW2^T))
cudaError_t launch_gemm_rows(const float* x, int ldx, const __nv_bfloat16* W, const __nv_bfloat16* W2, float* y,
                             int ldy, int col0, int T, int N, int K, int mode, cudaStream_t st);
cudaError_t launch_rope_append(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int T,
                               cudaStream_t st);
cudaError_t launch_attention(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int B, int R,
                             int nsplit, int chunk, bool emit_split, bool pdl, cudaStream_t st);
// tensor-core partial pass (one split per 64 keys) and the combine pass on its own
int attention_mma_tiles_per_block(const ModelView& m, int B, int R, long long keys);
cudaError_t launch_attention_mma(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int B, int R,
                                 int nsplit, int nsp, uint32_t* status, bool pdl, cudaStream_t st);
cudaError_t launch_attention_combine(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int nsplit,
                                     bool emit_split, bool pdl, cudaStream_t st);
cudaError_t launch_lm_merge(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int n_tiles,
                            const float* bonus_uniform, uint32_t* status, cudaStream_t st);
cudaError_t launch_lm_reduce(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R,
                             const float* bonus_uniform, const int32_t* tok, const int32_t* parent,
                             uint32_t* status, cudaStream_t st);
// Warped target rows from sc.logits: fills row_lse (over the kept tokens), row_cand, row_cand_lp and node_lp.
cudaError_t launch_warp_rows(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int top_k,
                             float top_p, const float* bonus_uniform, uint32_t* status, cudaStream_t st);
struct AcceptArgs {
    int B, R, max_depth;
    const int32_t* tok;        // [B, R-1]
    const int32_t* parent;     // [B, R-1] or nullptr (chain)
    const float* logq_ref;     // [B, max_depth]
    float log_tau;
};
struct SpdArgs {
    int B, R, max_depth;
    const int32_t* tok;             // [B, R-1]
    const float* logq_rows;         // [B, R-1, V] the auxiliary model's log-distributions at the draft positions
    const float* accept_uniform;    // [B, R-1]
    const float* resample_uniform;  // [B, V]
};
cudaError_t launch_spd_accept(const ModelView& m, const RowMeta& rm, const Scratch& sc, const SpdArgs& a,
                              const mtad_result& out, cudaStream_t st);
cudaError_t launch_accept(const RowMeta& rm, const Scratch& sc, const AcceptArgs& a, const mtad_result& out,
                          cudaStream_t st);
cudaError_t launch_kv_commit(const ModelView& m, const SeqState& s, int B, const int32_t* call_seq_dev,
                             const mtad_result& res, int max_depth, cudaStream_t st);
cudaError_t launch_seq_advance(const SeqState& s, int B, const int32_t* call_seq_dev, const mtad_result& res,
                               int max_depth, int max_batch, long long cap, cudaStream_t st);
cudaError_t launch_draft_prepare(const ModelView& m, const SeqState& s, const DraftState& ds, const RowMeta& rm,
                                 const Scratch& sc, const SeqList& seqs, int B, int R, int step, int beam, bool tc,
                                 bool warped, bool pdl, cudaStream_t st);
cudaError_t launch_draft_select(const ModelView& m, const DraftState& ds, const Scratch& sc, const SeqList& seqs, int B,
                                int R, int step, int gamma, int beam, int keep_all, const float* uniforms,
                                const DraftOut& out, bool pdl, cudaStream_t st);
cudaError_t launch_draft_select_warped(const ModelView& m, const DraftState& ds, const Scratch& sc, const SeqList& seqs,
                                       int B, int R, int step, int gamma, int beam, int keep_all, const float* uniforms,
                                       const DraftOut& out, cudaStream_t st);
cudaError_t launch_warp_rows_only(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int top_k,
                                  float top_p, const float* uni, cudaStream_t st);
cudaError_t launch_aux_commit(const ModelView& aux, const SeqState& s, const DraftState& ds, int B,
                              const int32_t* call_seq_dev, const mtad_result& res, int max_depth, int mode,
                              cudaStream_t st);
cudaError_t launch_seq_set(const SeqState& s, int seq, int kv_len, int root, int aux_len, int npend,
                           const int32_t* pend_host, cudaStream_t st);

}  // namespace mtad
