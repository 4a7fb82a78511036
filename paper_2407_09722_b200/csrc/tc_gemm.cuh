// Interface of the tensor-core weight-streaming GEMM (tcgen05 + TMEM + TMA) and its fused epilogues.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace mtad {

constexpr int TC_TILE_N = 128;      // output features per tile (the MMA M dimension: weights are operand A)
constexpr int TC_TILE_K = 64;       // bf16 elements per k-block: one 128-byte swizzle row
constexpr int TC_MAX_ROWS = 256;    // activation rows per launch (the MMA N dimension)
constexpr int TC_X_ROWS = 256;      // rows allocated in every activation operand buffer

enum TcMode {
    TC_PLAIN = 0,     // out[r, n] = acc
    TC_QKV = 1,       // rotary embedding; q -> fp32 (scaled), k, v -> bf16 KV cache
    TC_RESID = 2,     // hidden[r, n] += acc; emits hidden * gain as bf16 hi/lo and per-tile sums of squares
    TC_SWIGLU = 3,    // rows 0..63 of a tile are gate, 64..127 up: silu(gate) * up as bf16 hi/lo
    TC_LMHEAD = 4     // per (row, tile): max, sum-exp, best perturbed logit; gathers the drafted tokens' logits
};

struct TcGemmParams {
    // decomposition
    int n_tiles, k_blocks, total_units, units_per_cta, max_contrib;
    int T;                 // valid activation rows
    int rpad;              // T rounded up to 16; the operand tile has terms * rpad rows (the terms of a row are neighbours)
    int terms;             // bf16 terms per activation row read (2 or 3)
    int out_terms;         // bf16 terms per activation row emitted (what the GEMM that reads x_out expects)
    int seg_cap;           // stream-K kernel: k-blocks accumulated in tensor memory before the accumulator is drained
    int n_bbox;            // TMA boxes (and MMAs per k step and half) that cover the operand rows: 1, 2 or 3
    int mh;                // 128-row weight halves per tile and stage (1 or 2); a tile is mh * 128 output features
    int nbuf;              // TMEM accumulator buffers (set by the launcher)
    int per_sm;            // CTAs of this launch that share an SM (1 or 2): sets the shared- and tensor-memory budget
    int sliced;            // 1: the passes of a finished tile are shared out among its contributors (more than 8 rows)
    int n_rows_total;      // weight rows, for skipping a half that lies beyond them
    int n_tiles128;        // ceil(N / 128): row stride of lm_part
    int stages;            // smem ring depth
    unsigned int wait_limit;     // iterations a bounded wait may poll (0: the default, 2^22)
    int debug_no_operands;       // test hook: the operand-row producer issues no copies, so the waits on them run out
    unsigned long long* trace;   // MTAD_TRACE builds: [CTA][8] global-timer stamps of this launch, else null
    int csize;             // cluster kernel: CTAs that share a tile's k-range (1..8)
    int rpr;               // cluster kernel: rows per epilogue pass (1..8); pass q is finished by rank q % csize
    int recv_alias;        // cluster kernel: the receive slots of the exchange lie over the copy ring
    int ring_bytes;        // cluster kernel: shared memory below the fixed tail (set by the launch)
    int tile_base;         // cluster kernel (many rows): first tile of this launch, when a matrix takes two launches
    int mode;
    int N;                 // output features (bound for stores)
    // split-K fix-up
    float* ws;             // [n_tiles][max_contrib][mh][rpad][128] partial tiles (terms already summed)
    int* counters;         // [n_tiles], zero between launches
    uint32_t* status;      // device status word for time-outs (may be null)
    // deferred RMSNorm of the input: rstd[r] = rsqrt(sum_parts / dim + eps); parts == 0 -> 1
    const float* sumsq_in;
    int sumsq_in_parts;
    float inv_dim, eps;
    // TC_PLAIN
    float* out;
    int ldo;
    // TC_QKV
    int seg_k_tile, seg_v_tile;     // first tile of the K rows and of the V rows
    int Hq, Hkv, hd;
    float* q_out;                   // [T, (Hq + 2 Hkv) hd], q part written
    __nv_bfloat16 *q_hi, *q_lo;     // [T, Hq hd] each, or null: q * log2(e) / sqrt(hd) split for the MMA attention
    const float* rope;              // [T, hd/2, 2]
    __nv_bfloat16* cache;
    const int32_t* slot;
    const int32_t* seq;
    int layer, max_batch;
    long long cap;
    // TC_RESID / TC_SWIGLU outputs
    float* hidden;                  // [T, N]
    const __nv_bfloat16* gain;      // [N] gains of the norm that follows (TC_RESID)
    __nv_bfloat16* x_out;           // operand rows for the next GEMM (layout of store_terms)
    __nv_bfloat16* x_out2;          // TC_RESID: a second copy with out_terms2 terms (rows of the K/V projection), or null
    int out_terms2;
    int xk;                         // their row length: the next GEMM's K
    float* sumsq_out;               // [n_tiles][TC_X_ROWS]
    // TC_LMHEAD
    float4* lm_part;                // [T][n_tiles] (max, sumexp, best value, best index bits)
    const float* uniforms;          // [B, V]
    int R;                          // rows per sequence
    const int32_t* prow;            // [T] parent row of a node row, -1 otherwise
    const int32_t* tok;             // [T]
    float* node_z;                  // [T] logit of the row's token under its parent row
};

struct TcMaps {
    CUtensorMap a0, a1, a2;         // weight maps (QKV: wq, wk, wv; SwiGLU: gate, up; else a0)
    CUtensorMap x;                  // operand rows [2 * TC_X_ROWS, K]: row terms * t + j = term j of activation row t
};

// What one launch of the stream-K kernel takes: the tensor maps and the parameters, as one kernel argument.
struct TcChain {
    TcMaps maps[1];
    TcGemmParams p[1];
};
cudaError_t launch_tc_chain(const TcChain& chain, bool pdl, cudaStream_t st);

// Encodes a 2-D bf16 tensor map (row-major [rows, cols], 128-byte swizzle, box [box_rows, 64]).
int tc_make_map(CUtensorMap* out, const void* base, long long rows, long long cols, int box_rows);
// KV cache [planes][cap][hd] bf16 as a 3-D map (hd, cap, planes) with boxes of 64 elements x 64 positions, 128-byte
// swizzle (hd = 64 or 128).
int tc_make_kv_map(CUtensorMap* out, const void* cache, int hd, long long cap, long long planes);

// Fills the decomposition fields of p (and p.terms, p.per_sm for T rows) for a problem of n_tiles x k_blocks on
// `sms` SMs with per_sm CTAs each (0: tc_ctas_per_sm(T)).
void tc_decompose(TcGemmParams& p, int n_tiles, int K, int T, int sms, int per_sm = 0, int terms = 0);
// Operand-row boxes for acc_cols accumulator columns: each at most 256 rows and a multiple of 16
int tc_boxes(int acc_cols);
// CTAs per SM for a call of T rows: 2 for few rows (each with half the shared memory and at most 256 columns of
// tensor memory: one CTA's drain, fix-up and epilogue overlap the other's streaming), else 1.
int tc_ctas_per_sm(int T);
// Weight halves per tile that fit tensor memory for T rows, given tc_terms(T) accumulator columns per row.
int tc_halves(int T);
size_t tc_workspace_floats(int n_tiles_max, int max_contrib_max, int rpad_max);

// Cluster variants: a cluster of p.csize CTAs per tile of p.mh 128-feature halves, partial rows exchanged through
// distributed shared memory - tc_gemm_cluster.cu for calls of up to 32 rows (two CTAs on an SM, one half), and
// tc_gemm_cluster_big.cu beyond (one CTA on an SM, two halves).  tc_cluster_plan fills the decomposition (halves per
// tile, CTAs per SM, cluster size, rows per pass) for a matrix of n_tiles128 128-feature tiles on `sms` SMs and
// returns false when the shape does not suit it (more than 256 accumulator columns, more tiles than co-resident
// CTAs).  p.mode and, for QKV, the segment tiles must be set before the call: a tile never straddles q | k | v.  The
// weight maps of the launch must have boxes of p.mh halves.
bool tc_cluster_plan(TcGemmParams& p, int n_tiles128, int K, int T, int sms);
// More tiles than SMs and more than 32 rows: the matrix as two cluster launches over two ranges of its tiles (a and b
// come in as copies of the launch's parameters with p.mode set).  False when that does not apply.
bool tc_cluster_plan_big_split(TcGemmParams& a, TcGemmParams& b, int n_tiles128, int K, int T, int sms);
bool tc_cluster_plan_small(TcGemmParams& p, int n_tiles, int K, int T, int slots);
cudaError_t launch_tc_cluster_small(const TcMaps& maps, const TcGemmParams& p, bool pdl, cudaStream_t st);
cudaError_t launch_tc_cluster(const TcMaps& maps, const TcGemmParams& p, bool pdl, cudaStream_t st);

cudaError_t launch_tc_gemm(const TcMaps& maps, const TcGemmParams& p, int ctas, bool pdl, cudaStream_t st);

// Splits fp32 rows [T, K] into operand rows of `terms` bf16 terms (layout of store_terms).
cudaError_t launch_split_rows(const float* x, int ldx_in, __nv_bfloat16* out, int terms, int T, int K, cudaStream_t st);

}  // namespace mtad
