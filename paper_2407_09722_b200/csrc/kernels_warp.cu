// Warped target rows (the paper's App. F: keep the top-k tokens and renormalise, then keep the first tokens, in
// descending order of probability, whose cumulative probability exceeds top-p; the kept tokens are renormalised)
// for the verification rule and the extra token, from the plain logits of a verify forward.
//
// Three small passes over [T, V] logits that never leave L2: per-chunk top-k lists (one block per chunk and row), a
// merge per row (one warp: overall top-k in descending order, the top-p cut, log-probabilities of the kept tokens,
// Gumbel-argmax of the extra token over the kept tokens), and a lookup of every node's token in its parent row's
// kept list (-inf if it was dropped: such a draft can never be accepted).
#include <math_constants.h>

#include "common.cuh"

namespace mtad {

namespace {

struct Top {
    float z;
    int v;
};
// a ranks ahead of b: larger logit, lower token id among equals
__device__ __forceinline__ bool ahead(const Top& a, const Top& b) { return a.z > b.z || (a.z == b.z && a.v < b.v); }

constexpr int NONE = 0x7fffffff;

}  // namespace

__global__ void __launch_bounds__(256) warp_scan_kernel(const float* __restrict__ logits, int V,
                                                        const int32_t* __restrict__ slot,
                                                        WarpPart* __restrict__ part, int nch, int K) {
    const int c = blockIdx.x, t = blockIdx.y, tid = threadIdx.x;
    if (slot[t] < 0) return;
    const float* z = logits + (size_t)t * V;
    const int len = (V + nch - 1) / nch, v0 = c * len, v1 = min(V, v0 + len);
    Top loc[MTAD_MAX_TOPK];
#pragma unroll
    for (int k = 0; k < MTAD_MAX_TOPK; ++k) loc[k] = Top{-CUDART_INF_F, NONE};
    for (int v = v0 + tid; v < v1; v += 256) {
        const Top cd{z[v], v};
        if (ahead(cd, loc[MTAD_MAX_TOPK - 1])) {
            loc[MTAD_MAX_TOPK - 1] = cd;
#pragma unroll
            for (int k = MTAD_MAX_TOPK - 1; k > 0; --k)
                if (ahead(loc[k], loc[k - 1])) { const Top tmp = loc[k]; loc[k] = loc[k - 1]; loc[k - 1] = tmp; }
        }
    }
    __shared__ Top s_c[256];
    WarpPart* dst = part + (size_t)t * nch + c;
    int head = 0;
    for (int k = 0; k < K; ++k) {
        Top cd{-CUDART_INF_F, NONE};
#pragma unroll
        for (int q = 0; q < MTAD_MAX_TOPK; ++q)
            if (q == head) cd = loc[q];                  // (no dynamic register indexing)
        s_c[tid] = cd;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (tid < o && ahead(s_c[tid + o], s_c[tid])) s_c[tid] = s_c[tid + o];
            __syncthreads();
        }
        const Top win = s_c[0];
        __syncthreads();
        if (cd.v == win.v && win.v != NONE) ++head;      // the owner of the winner moves on (token ids are unique)
        if (tid == 0) { dst->z[k] = win.z; dst->v[k] = win.v == NONE ? -1 : win.v; }
    }
}

__global__ void __launch_bounds__(32) warp_merge_kernel(const WarpPart* __restrict__ part, int nch, int K, float top_p,
                                                        int V, int R, const float* __restrict__ uni,
                                                        const int32_t* __restrict__ slot, WarpRow* __restrict__ rows,
                                                        float* __restrict__ row_lse, int32_t* __restrict__ row_cand,
                                                        float* __restrict__ row_cand_lp, uint32_t* status) {
    const int t = blockIdx.x, bi = t / R, lane = threadIdx.x;
    WarpRow* row = rows + t;
    if (slot[t] < 0) {
        if (lane == 0) { row->n = 0; row_lse[t] = 0.f; row_cand[t] = 0; row_cand_lp[t] = 0.f; }
        return;
    }
    __shared__ float s_z[MTAD_DRAFT_CHUNKS * MTAD_MAX_TOPK];
    __shared__ int s_v[MTAD_DRAFT_CHUNKS * MTAD_MAX_TOPK];
    __shared__ float s_tz[MTAD_MAX_TOPK];
    __shared__ int s_tv[MTAD_MAX_TOPK];
    const int n_cand = nch * K;
    for (int i = lane; i < n_cand; i += 32) {
        const WarpPart& p = part[(size_t)t * nch + i / K];
        const int v = p.v[i % K];
        s_z[i] = v >= 0 ? p.z[i % K] : -CUDART_INF_F;
        s_v[i] = v >= 0 ? v : NONE;
    }
    __syncwarp();
    // the K largest in descending order: K rounds of a warp-wide arg-max
    int found = 0;
    for (int k = 0; k < K; ++k) {
        Top best{-CUDART_INF_F, NONE};
        int bidx = -1;
        for (int i = lane; i < n_cand; i += 32) {
            const Top cd{s_z[i], s_v[i]};
            if (cd.v != NONE && ahead(cd, best)) { best = cd; bidx = i; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const Top ot{__shfl_xor_sync(0xffffffffu, best.z, o), __shfl_xor_sync(0xffffffffu, best.v, o)};
            const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
            if (ot.v != NONE && (best.v == NONE || ahead(ot, best))) { best = ot; bidx = oi; }
        }
        if (best.v == NONE) break;                       // fewer than K tokens in the vocabulary
        if (lane == 0) { s_tz[k] = best.z; s_tv[k] = best.v; s_v[bidx] = NONE; }
        ++found;
        __syncwarp();
    }
    if (lane == 0) {
        // renormalised top-k probabilities, descending; keep the first tokens whose cumulative probability exceeds top_p
        float sum = 0.f;
        for (int i = 0; i < found; ++i) sum += expf(s_tz[i] - s_tz[0]);
        int keep = found;
        float c = 0.f;
        for (int i = 0; i < found; ++i) {
            c += expf(s_tz[i] - s_tz[0]) / sum;
            if (c > top_p) { keep = i + 1; break; }
        }
        float ks = 0.f;
        for (int i = 0; i < keep; ++i) ks += expf(s_tz[i] - s_tz[0]);
        const float lse = s_tz[0] + logf(ks);
        row->n = keep;
        // the extra token: Gumbel-argmax over the kept tokens (lower token id on ties), noise from uniform[token]
        float by = -CUDART_INF_F;
        int bv = NONE;
        float blp = 0.f;
        for (int i = 0; i < keep; ++i) {
            const float lp = s_tz[i] - lse;
            row->idx[i] = s_tv[i];
            row->lp[i] = lp;
            const float y = s_tz[i] - logf(-logf(uni[(size_t)bi * V + s_tv[i]]));
            if (y > by || (y == by && s_tv[i] < bv)) { by = y; bv = s_tv[i]; blp = lp; }
        }
        // a row of NaN logits ranks no token: flag the sequence, as the unwarped path does
        if (status && (found == 0 || bv == NONE || !isfinite(lse))) atomicOr(&status[bi], MTAD_ST_NONFINITE);
        row_lse[t] = lse;
        row_cand[t] = bv == NONE ? 0 : bv;
        row_cand_lp[t] = blp;
    }
}

__global__ void warp_node_lp_kernel(const WarpRow* __restrict__ rows, const int32_t* __restrict__ prow,
                                    const int32_t* __restrict__ tok, float* __restrict__ node_lp, int T) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int pr = prow[t];
    float lp = 0.f;
    if (pr >= 0) {
        lp = -CUDART_INF_F;                              // dropped by the warping: probability 0
        const WarpRow& r = rows[pr];
        const int x = tok[t];
        for (int i = 0; i < r.n; ++i)
            if (r.idx[i] == x) lp = r.lp[i];
    }
    node_lp[t] = lp;
}

// The warped rows alone (kept tokens and their log-probabilities, sc.warp_row), for the draft's selection: `uni` only
// feeds the row's extra-token draw, which the draft does not use, and may be any [B, V] array of uniforms.
cudaError_t launch_warp_rows_only(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int top_k,
                                  float top_p, const float* uni, cudaStream_t st) {
    const int V = m.d.vocab, T = B * R;
    int nch = (V + 1023) / 1024;
    nch = nch < 1 ? 1 : (nch > MTAD_DRAFT_CHUNKS ? MTAD_DRAFT_CHUNKS : nch);
    warp_scan_kernel<<<dim3(nch, T), 256, 0, st>>>(sc.logits, V, rm.slot, sc.warp_part, nch, top_k);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    warp_merge_kernel<<<T, 32, 0, st>>>(sc.warp_part, nch, top_k, top_p, V, R, uni, rm.slot, sc.warp_row, sc.row_lse,
                                        sc.row_cand, sc.row_cand_lp, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_warp_rows(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int top_k,
                             float top_p, const float* bonus_uniform, uint32_t* status, cudaStream_t st) {
    const int V = m.d.vocab, T = B * R;
    int nch = (V + 1023) / 1024;
    nch = nch < 1 ? 1 : (nch > MTAD_DRAFT_CHUNKS ? MTAD_DRAFT_CHUNKS : nch);
    warp_scan_kernel<<<dim3(nch, T), 256, 0, st>>>(sc.logits, V, rm.slot, sc.warp_part, nch, top_k);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    warp_merge_kernel<<<T, 32, 0, st>>>(sc.warp_part, nch, top_k, top_p, V, R, bonus_uniform, rm.slot, sc.warp_row,
                                        sc.row_lse, sc.row_cand, sc.row_cand_lp, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    warp_node_lp_kernel<<<(T + 127) / 128, 128, 0, st>>>(sc.warp_row, rm.prow, rm.tok, sc.node_lp, T);
    return cudaGetLastError();
}

}  // namespace mtad
