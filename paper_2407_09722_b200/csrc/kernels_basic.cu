// Row bookkeeping, RMSNorm, rotary embedding + KV append, CUDA-core skinny GEMM, LM-head reductions,
// accept/select and KV commit kernels.
#include <math_constants.h>

#include "common.cuh"

namespace mtad {

// ---------------------------------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------------------------------

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Deterministic block-wide sum (fixed tree, independent of scheduling). blockDim.x multiple of 32, <= 1024.
__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
    if (w == 0) {
        t = warp_sum(t);
        if (l == 0) red[0] = t;
    }
    __syncthreads();
    t = red[0];
    __syncthreads();
    return t;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---------------------------------------------------------------------------------------------------------------
// sequence state
// ---------------------------------------------------------------------------------------------------------------

struct PendTok {
    int32_t v[MTAD_MAX_DEPTH + 1];
};

__global__ void seq_set_kernel(SeqState s, int seq, int kv_len, int root, int aux_len, int npend, PendTok p) {
    if (threadIdx.x == 0) {
        s.kv_len[seq] = kv_len;
        s.root_tok[seq] = root;
        s.aux_len[seq] = aux_len;
        s.aux_npend[seq] = npend;
    }
    if (threadIdx.x < npend) s.aux_pend[seq * (MTAD_MAX_DEPTH + 1) + threadIdx.x] = p.v[threadIdx.x];
}

cudaError_t launch_seq_set(const SeqState& s, int seq, int kv_len, int root, int aux_len, int npend,
                           const int32_t* pend_host, cudaStream_t st) {
    // pending list of the auxiliary model: the committed tokens it has not seen yet, then the root
    PendTok p;
    for (int i = 0; i <= MTAD_MAX_DEPTH; ++i) p.v[i] = (i < npend && pend_host) ? pend_host[i] : 0;
    p.v[npend] = root;
    seq_set_kernel<<<1, 64, 0, st>>>(s, seq, kv_len, root, aux_len, npend + 1, p);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// prepare: rows of the verify forward (root + draft nodes), validation, embedding gather, rotary table
// ---------------------------------------------------------------------------------------------------------------

__global__ void prepare_kernel(const __nv_bfloat16* __restrict__ embed, int d, int vocab, int hd, RopeInv rinv,
                               long long kv_capacity, SeqState s, RowMeta rm, float* __restrict__ hidden,
                               float* __restrict__ rope, PrepareArgs a, uint32_t* status) {
    const int t = blockIdx.x, bi = t / a.R, r = t % a.R;
    const int seq = a.seqs.v[bi];
    const int L = s.kv_len[seq];
    const int N = a.R - 1;
    int nn = a.n_nodes ? a.n_nodes[bi] : N;
    __shared__ int sh_tok, sh_pos, sh_ok;
    if (threadIdx.x == 0) {
        uint32_t st = 0;
        if (nn < 0 || nn > N) { st |= MTAD_ST_BAD_COUNT; nn = 0; }
        if (L < 0 || (long long)L + nn + 1 > kv_capacity) st |= MTAD_ST_KV_OVERFLOW;
        const bool seq_ok = (st == 0);
        int tok = 0, depth = 0;
        uint32_t mask[MTAD_MASK_WORDS];
#pragma unroll
        for (int i = 0; i < MTAD_MASK_WORDS; ++i) mask[i] = 0;
        const bool active = seq_ok && r <= nn;
        if (active) {
            if (r == 0) {
                tok = s.root_tok[seq];
            } else {
                const int n = r - 1;
                tok = a.tok[bi * N + n];
                int cur = n, steps = 0;
                // walk to the root; valid trees have parent < child, so at most n + 1 steps
                while (cur >= 0 && steps <= N) {
                    mask[(cur + 1) >> 5] |= 1u << ((cur + 1) & 31);
                    const int p = a.parent ? a.parent[bi * N + cur] : cur - 1;
                    if (p < -1 || p >= cur) { st |= MTAD_ST_BAD_PARENT; break; }
                    cur = p;
                    ++depth;
                    ++steps;
                }
                if (depth > a.max_depth) st |= MTAD_ST_TOO_DEEP;
            }
            mask[0] |= 1u;
            if (tok < 0 || tok >= vocab) { st |= MTAD_ST_BAD_TOKEN; tok = 0; }
        }
        if (st) atomicOr(&status[bi], st);
        rm.tok[t] = tok;
        rm.depth[t] = depth;
        rm.pos[t] = L + depth;
        rm.slot[t] = active ? L + r : -1;
        rm.seq[t] = seq;
#pragma unroll
        for (int i = 0; i < MTAD_MASK_WORDS; ++i) rm.mask[(size_t)t * MTAD_MASK_WORDS + i] = mask[i];
        int pr = -1;
        if (active && r > 0 && !(st & MTAD_ST_BAD_PARENT)) {
            const int p0 = a.parent ? a.parent[bi * N + (r - 1)] : r - 2;
            pr = bi * a.R + p0 + 1;
        }
        rm.prow[t] = pr;
        if (r == 0) {
            rm.n_rows[bi] = seq_ok ? nn + 1 : 0;
            rm.n_spec[bi] = seq_ok ? nn + 1 : 0;
            rm.kv_base[bi] = L;
            rm.call_seq[bi] = seq;
        }
        sh_tok = tok;
        sh_pos = L + depth;
        sh_ok = active;
    }
    __syncthreads();
    const int tok = sh_tok;
    const bool ok = sh_ok;
    float ss = embed_row(embed + (size_t)tok * d, ok, d, hidden + (size_t)t * d, a.gain0,
                         a.x ? a.x + (size_t)t * a.terms * d : nullptr, a.terms);
    if (a.x) {
        __shared__ float red[32];
        ss = block_sum(ss, red);                     // (also orders the hidden row's stores before the loop below)
        if (threadIdx.x == 0) a.sumsq_out[t] = ss;
        if (a.x2)
            for (int i = threadIdx.x; i < d; i += blockDim.x)
                store_terms(hidden[(size_t)t * d + i] * __bfloat162float(a.gain0[i]),
                            a.x2 + (size_t)t * a.terms2 * d + i, d, a.terms2);
    }
    // rotary table: angle = pos * base^(-2i/hd)
    for (int i = threadIdx.x; i < hd / 2; i += blockDim.x) {
        float cs, sn;
        rope_cs((double)sh_pos, rinv.v[i], cs, sn);
        rope[((size_t)t * (hd / 2) + i) * 2 + 0] = cs;
        rope[((size_t)t * (hd / 2) + i) * 2 + 1] = sn;
    }
}

cudaError_t launch_prepare(const ModelView& m, const SeqState& s, const RowMeta& rm, const Scratch& sc,
                           const PrepareArgs& a, uint32_t* status, cudaStream_t st) {
    prepare_kernel<<<a.B * a.R, 128, 0, st>>>(static_cast<const __nv_bfloat16*>(m.d.embed), m.d.d_model, m.d.vocab,
                                              m.d.head_dim, rope_inv((double)m.d.rope_base, m.d.head_dim),
                                              (long long)m.d.kv_capacity, s, rm,
                                              sc.hidden, sc.rope, a, status);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// RMSNorm: y = x * rsqrt(mean(x^2) + eps) * gain
// ---------------------------------------------------------------------------------------------------------------

__global__ void rmsnorm_kernel(const float* __restrict__ x, const __nv_bfloat16* __restrict__ gain,
                               float* __restrict__ y, int d, float eps) {
    __shared__ float red[32];
    const float* xr = x + (size_t)blockIdx.x * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) ss += xr[i] * xr[i];
    ss = block_sum(ss, red);
    const float rstd = rsqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        y[(size_t)blockIdx.x * d + i] = xr[i] * rstd * __bfloat162float(gain[i]);
}

cudaError_t launch_rmsnorm(const float* x, const __nv_bfloat16* gain, float* y, int T, int d, float eps,
                           cudaStream_t st) {
    rmsnorm_kernel<<<T, 256, 0, st>>>(x, gain, y, d, eps);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// CUDA-core skinny GEMM: one warp owns NW output columns for a chunk of <= 8 rows; lanes split K in 8-element
// (16-byte) pieces; fp32 accumulation; butterfly reduction at the end.
// ---------------------------------------------------------------------------------------------------------------

template <int NW, int MODE>
__global__ void __launch_bounds__(256) gemm_rows_kernel(const float* __restrict__ x, int ldx,
                                                        const __nv_bfloat16* __restrict__ W,
                                                        const __nv_bfloat16* __restrict__ W2, float* __restrict__ y,
                                                        int ldy, int col0, int T, int N, int K) {
    constexpr int RC = MTAD_ROW_CHUNK;
    constexpr int NM = (MODE == 2) ? 2 : 1;          // matrices streamed together
    const int chunk = blockIdx.x;                    // row chunk varies fastest so that chunks share weights in L2
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = (blockIdx.y * 8 + warp) * NW;
    if (n0 >= N) return;
    const int t0 = chunk * RC;
    const int rows = min(RC, T - t0);
    float acc[NM][NW][RC];
#pragma unroll
    for (int a = 0; a < NM; ++a)
#pragma unroll
        for (int j = 0; j < NW; ++j)
#pragma unroll
            for (int r = 0; r < RC; ++r) acc[a][j][r] = 0.f;

    for (int k = lane * 8; k < K; k += 256) {
        uint4 wv[NM][NW];
#pragma unroll
        for (int j = 0; j < NW; ++j) {
            const int n = min(n0 + j, N - 1);
            wv[0][j] = __ldg(reinterpret_cast<const uint4*>(W + (size_t)n * K + k));
            if (NM == 2) wv[NM - 1][j] = __ldg(reinterpret_cast<const uint4*>(W2 + (size_t)n * K + k));
        }
#pragma unroll
        for (int r = 0; r < RC; ++r) {
            if (r < rows) {
                const float4 xa = *reinterpret_cast<const float4*>(x + (size_t)(t0 + r) * ldx + k);
                const float4 xb = *reinterpret_cast<const float4*>(x + (size_t)(t0 + r) * ldx + k + 4);
#pragma unroll
                for (int a = 0; a < NM; ++a)
#pragma unroll
                    for (int j = 0; j < NW; ++j) {
                        const uint4 w = wv[a][j];
                        float s = acc[a][j][r];
                        s = fmaf(xa.x, bf16_lo(w.x), s);
                        s = fmaf(xa.y, bf16_hi(w.x), s);
                        s = fmaf(xa.z, bf16_lo(w.y), s);
                        s = fmaf(xa.w, bf16_hi(w.y), s);
                        s = fmaf(xb.x, bf16_lo(w.z), s);
                        s = fmaf(xb.y, bf16_hi(w.z), s);
                        s = fmaf(xb.z, bf16_lo(w.w), s);
                        s = fmaf(xb.w, bf16_hi(w.w), s);
                        acc[a][j][r] = s;
                    }
            }
        }
    }
#pragma unroll
    for (int a = 0; a < NM; ++a)
#pragma unroll
        for (int j = 0; j < NW; ++j)
#pragma unroll
            for (int r = 0; r < RC; ++r) acc[a][j][r] = warp_sum(acc[a][j][r]);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < NW; ++j) {
            if (n0 + j < N) {
#pragma unroll
                for (int r = 0; r < RC; ++r) {
                    if (r < rows) {
                        float* dst = y + (size_t)(t0 + r) * ldy + col0 + n0 + j;
                        if (MODE == 0) {
                            *dst = acc[0][j][r];
                        } else if (MODE == 1) {
                            *dst += acc[0][j][r];
                        } else {
                            const float g = acc[0][j][r];
                            *dst = g / (1.f + expf(-g)) * acc[NM - 1][j][r];
                        }
                    }
                }
            }
        }
    }
}

cudaError_t launch_gemm_rows(const float* x, int ldx, const __nv_bfloat16* W, const __nv_bfloat16* W2, float* y,
                             int ldy, int col0, int T, int N, int K, int mode, cudaStream_t st) {
    // K is a multiple of 8 (16-byte weight pieces); checked when the context is created.
    const int chunks = (T + MTAD_ROW_CHUNK - 1) / MTAD_ROW_CHUNK;
    if (mode == 2) {
        constexpr int NW = 2;
        dim3 grid(chunks, (N + 8 * NW - 1) / (8 * NW));
        gemm_rows_kernel<NW, 2><<<grid, 256, 0, st>>>(x, ldx, W, W2, y, ldy, col0, T, N, K);
    } else {
        constexpr int NW = 4;
        dim3 grid(chunks, (N + 8 * NW - 1) / (8 * NW));
        if (mode == 0)
            gemm_rows_kernel<NW, 0><<<grid, 256, 0, st>>>(x, ldx, W, W2, y, ldy, col0, T, N, K);
        else
            gemm_rows_kernel<NW, 1><<<grid, 256, 0, st>>>(x, ldx, W, W2, y, ldy, col0, T, N, K);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// rotary embedding on q (in place, also scaled by 1/sqrt(hd)) and k; K, V rounded to bf16 into the cache
// ---------------------------------------------------------------------------------------------------------------

__global__ void rope_append_kernel(float* __restrict__ qkv, const float* __restrict__ rope,
                                   __nv_bfloat16* __restrict__ cache, const int32_t* __restrict__ slot,
                                   const int32_t* __restrict__ seq, int layer, int max_batch, int Hq, int Hkv, int hd,
                                   long long cap) {
    const int t = blockIdx.x;
    const int half = hd / 2;
    const int ldq = (Hq + 2 * Hkv) * hd;
    float* row = qkv + (size_t)t * ldq;
    const float* rt = rope + (size_t)t * half * 2;
    const int sl = slot[t];
    const float scale = rsqrtf((float)hd);
    for (int i = threadIdx.x; i < Hq * half; i += blockDim.x) {
        const int h = i / half, j = i % half;
        const float c = rt[j * 2], sn = rt[j * 2 + 1];
        const float a = row[h * hd + j], b = row[h * hd + j + half];
        row[h * hd + j] = (a * c - b * sn) * scale;
        row[h * hd + j + half] = (b * c + a * sn) * scale;
    }
    if (sl < 0 || sl >= cap || (unsigned)seq[t] >= (unsigned)max_batch) return;
    const size_t kbase = ((((size_t)layer * max_batch + seq[t]) * 2 + 0) * Hkv) * cap * hd;
    const size_t vbase = ((((size_t)layer * max_batch + seq[t]) * 2 + 1) * Hkv) * cap * hd;
    const float* kr = row + Hq * hd;
    const float* vr = kr + Hkv * hd;
    for (int i = threadIdx.x; i < Hkv * half; i += blockDim.x) {
        const int h = i / half, j = i % half;
        const float c = rt[j * 2], sn = rt[j * 2 + 1];
        const float a = kr[h * hd + j], b = kr[h * hd + j + half];
        __nv_bfloat16* dst = cache + kbase + ((size_t)h * cap + sl) * hd;
        dst[j] = __float2bfloat16_rn(a * c - b * sn);
        dst[j + half] = __float2bfloat16_rn(b * c + a * sn);
    }
    for (int i = threadIdx.x; i < Hkv * hd; i += blockDim.x) {
        const int h = i / hd, j = i % hd;
        cache[vbase + ((size_t)h * cap + sl) * hd + j] = __float2bfloat16_rn(vr[i]);
    }
}

cudaError_t launch_rope_append(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int T,
                               cudaStream_t st) {
    rope_append_kernel<<<T, 256, 0, st>>>(sc.qkv, sc.rope, static_cast<__nv_bfloat16*>(m.d.kv_cache), rm.slot, rm.seq,
                                          layer, m.max_batch, m.d.n_q_heads, m.d.n_kv_heads, m.d.head_dim,
                                          (long long)m.d.kv_capacity);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// LM-head reductions over a row of logits: log-sum-exp, Gumbel-argmax, and the gather of each node's token
// ---------------------------------------------------------------------------------------------------------------

struct Best {
    float v;
    int i;
};
__device__ __forceinline__ Best better(Best a, Best b) {   // larger value, then lower index
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

__global__ void __launch_bounds__(1024) lm_reduce_kernel(const float* __restrict__ logits, int V, int R,
                                                         const float* __restrict__ uni,
                                                         const int32_t* __restrict__ slot,
                                                         float* __restrict__ row_lse, int32_t* __restrict__ row_cand,
                                                         float* __restrict__ row_cand_lp, uint32_t* status) {
    const int t = blockIdx.x, bi = t / R;
    if (slot[t] < 0) {
        if (threadIdx.x == 0) { row_lse[t] = 0.f; row_cand[t] = 0; row_cand_lp[t] = 0.f; }
        return;
    }
    const float* z = logits + (size_t)t * V;
    const float* u = uni + (size_t)bi * V;
    float m = -CUDART_INF_F, s = 0.f;
    Best best{-CUDART_INF_F, 0x7fffffff};
    for (int j = threadIdx.x; j < V; j += blockDim.x) {
        const float zj = z[j];
        if (zj > m) { s *= expf(m - zj); m = zj; }
        s += expf(zj - m);
        const float g = -logf(-logf(u[j]));
        best = better(best, Best{zj + g, j});
    }
    __shared__ float sm[1024], ss[1024], sv[1024];
    __shared__ int si[1024];
    sm[threadIdx.x] = m; ss[threadIdx.x] = s; sv[threadIdx.x] = best.v; si[threadIdx.x] = best.i;
    __syncthreads();
    for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float m1 = sm[threadIdx.x], m2 = sm[threadIdx.x + o];
            const float mm = fmaxf(m1, m2);
            const float s1 = (m1 == -CUDART_INF_F) ? 0.f : ss[threadIdx.x] * expf(m1 - mm);
            const float s2 = (m2 == -CUDART_INF_F) ? 0.f : ss[threadIdx.x + o] * expf(m2 - mm);
            sm[threadIdx.x] = mm; ss[threadIdx.x] = s1 + s2;
            const Best b = better(Best{sv[threadIdx.x], si[threadIdx.x]},
                                  Best{sv[threadIdx.x + o], si[threadIdx.x + o]});
            sv[threadIdx.x] = b.v; si[threadIdx.x] = b.i;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float lse = sm[0] + logf(ss[0]);
        // a row of NaN logits wins no comparison and leaves no candidate: flag it instead of indexing with it
        const bool none = (unsigned)si[0] >= (unsigned)V;
        if (none || !isfinite(lse)) atomicOr(&status[bi], MTAD_ST_NONFINITE);
        const int c = none ? 0 : si[0];
        row_lse[t] = lse;
        row_cand[t] = c;
        row_cand_lp[t] = z[c] - lse;
    }
}

__global__ void node_lp_kernel(const float* __restrict__ logits, int V, int B, int R, const int32_t* __restrict__ tok,
                               const int32_t* __restrict__ parent, const int32_t* __restrict__ slot,
                               const float* __restrict__ row_lse, float* __restrict__ node_lp) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int N = R - 1;
    if (i >= B * N) return;
    const int bi = i / N, n = i % N;
    const int t = bi * R + n + 1;
    float v = 0.f;
    if (slot[t] >= 0) {
        const int p = parent ? parent[i] : n - 1;
        const int tk = tok[i];
        if (p >= -1 && p < n && tk >= 0 && tk < V) {
            const int pr = bi * R + p + 1;
            v = logits[(size_t)pr * V + tk] - row_lse[pr];
        }
    }
    node_lp[t] = v;
}

cudaError_t launch_lm_reduce(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R,
                             const float* bonus_uniform, const int32_t* tok, const int32_t* parent,
                             uint32_t* status, cudaStream_t st) {
    lm_reduce_kernel<<<B * R, 1024, 0, st>>>(sc.logits, m.d.vocab, R, bonus_uniform, rm.slot, sc.row_lse, sc.row_cand,
                                             sc.row_cand_lp, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (R > 1) {
        const int n = B * (R - 1);
        node_lp_kernel<<<(n + 127) / 128, 128, 0, st>>>(sc.logits, m.d.vocab, B, R, tok, parent, rm.slot, sc.row_lse,
                                                        sc.node_lp);
        e = cudaGetLastError();
    }
    return e;
}

// Merge of the LM-head kernel's per-(row, vocab tile) partials, in tile order: log-sum-exp, Gumbel-argmax candidate
// and its log-probability per row, then the log-probability of every node's token under its parent row.
__global__ void lm_merge_kernel(const float4* __restrict__ part, int n_tiles, int V, int R,
                                const float* __restrict__ uni, const int32_t* __restrict__ slot,
                                float* __restrict__ row_lse, int32_t* __restrict__ row_cand,
                                float* __restrict__ row_cand_lp, uint32_t* status) {
    const int t = blockIdx.x, bi = t / R;
    if (slot[t] < 0) {
        if (threadIdx.x == 0) { row_lse[t] = 0.f; row_cand[t] = 0; row_cand_lp[t] = 0.f; }
        return;
    }
    float m = -CUDART_INF_F, s = 0.f;
    Best best{-CUDART_INF_F, 0x7fffffff};
    for (int j = threadIdx.x; j < n_tiles; j += blockDim.x) {
        const float4 q = part[idx_lm_part(t, n_tiles, j)];
        const float mm = fmaxf(m, q.x);
        s = (m == -CUDART_INF_F ? 0.f : s * expf(m - mm)) + (q.x == -CUDART_INF_F ? 0.f : q.y * expf(q.x - mm));
        m = mm;
        best = better(best, Best{q.z, __float_as_int(q.w)});
    }
    __shared__ float sm[256], ss[256], sv[256];
    __shared__ int si[256];
    sm[threadIdx.x] = m; ss[threadIdx.x] = s; sv[threadIdx.x] = best.v; si[threadIdx.x] = best.i;
    __syncthreads();
    for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float m1 = sm[threadIdx.x], m2 = sm[threadIdx.x + o];
            const float mm = fmaxf(m1, m2);
            const float s1 = (m1 == -CUDART_INF_F) ? 0.f : ss[threadIdx.x] * expf(m1 - mm);
            const float s2 = (m2 == -CUDART_INF_F) ? 0.f : ss[threadIdx.x + o] * expf(m2 - mm);
            sm[threadIdx.x] = mm; ss[threadIdx.x] = s1 + s2;
            const Best b = better(Best{sv[threadIdx.x], si[threadIdx.x]},
                                  Best{sv[threadIdx.x + o], si[threadIdx.x + o]});
            sv[threadIdx.x] = b.v; si[threadIdx.x] = b.i;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float lse = sm[0] + logf(ss[0]);
        // a row of NaN logits wins no comparison and leaves no candidate: flag it instead of indexing with it
        const bool none = (unsigned)si[0] >= (unsigned)V;
        if (none || !isfinite(lse)) atomicOr(&status[bi], MTAD_ST_NONFINITE);
        const int c = none ? 0 : si[0];
        row_lse[t] = lse;
        row_cand[t] = c;
        // the partial keeps logit + noise; take the noise off again to get the candidate's logit
        const float g = -logf(-logf(uni[(size_t)bi * V + c]));
        row_cand_lp[t] = (sv[0] - g) - lse;
    }
}

__global__ void node_lp_from_z_kernel(const float* __restrict__ node_z, const int32_t* __restrict__ prow,
                                      const float* __restrict__ row_lse, float* __restrict__ node_lp, int T) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const int pr = prow[t];
    node_lp[t] = pr >= 0 ? node_z[t] - row_lse[pr] : 0.f;
}

cudaError_t launch_lm_merge(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int n_tiles,
                            const float* bonus_uniform, uint32_t* status, cudaStream_t st) {
    lm_merge_kernel<<<B * R, 256, 0, st>>>(sc.lm_part, n_tiles, m.d.vocab, R, bonus_uniform, rm.slot, sc.row_lse,
                                           sc.row_cand, sc.row_cand_lp, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    node_lp_from_z_kernel<<<(B * R + 127) / 128, 128, 0, st>>>(sc.node_z, rm.prow, sc.row_lse, sc.node_lp, B * R);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// accept / select: one warp per sequence
// ---------------------------------------------------------------------------------------------------------------

__global__ void accept_kernel(RowMeta rm, Scratch sc, AcceptArgs a, mtad_result out) {
    const int bi = blockIdx.x, lane = threadIdx.x;
    const int R = a.R, N = R - 1, D = a.max_depth;
    __shared__ float LP[MTAD_MAX_NODES + 1];
    const int nrows = rm.n_rows[bi];
    const bool bad = (out.status[bi] != 0) || nrows == 0;
    const int nn = bad ? 0 : nrows - 1;
    const int t0 = bi * R;
    // joint log-likelihood along each path: LP[n] = LP[parent(n)] + lp[n] in node order (fp32)
    if (lane == 0) {
        for (int n = 0; n < nn; ++n) {
            const int p = a.parent ? a.parent[bi * N + n] : n - 1;
            LP[n] = (p < 0 ? 0.f : LP[p]) + sc.node_lp[t0 + n + 1];
        }
    }
    __syncwarp();
    // test every node against the threshold; keep the best (depth, LP, lowest index)
    int bd = 0, bn = -1;
    float bl = -CUDART_INF_F;
    float m_acc = CUDART_INF_F;
    for (int n = lane; n < nn; n += 32) {
        const int dep = rm.depth[t0 + n + 1];
        const float gap = (LP[n] - a.logq_ref[bi * D + dep - 1]) - a.log_tau;
        if (isfinite(gap)) m_acc = fminf(m_acc, fabsf(gap));
        if (gap > 0.f && (dep > bd || (dep == bd && LP[n] > bl))) { bd = dep; bl = LP[n]; bn = n; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int od = __shfl_xor_sync(0xffffffffu, bd, o);
        const float ol = __shfl_xor_sync(0xffffffffu, bl, o);
        const int on = __shfl_xor_sync(0xffffffffu, bn, o);
        m_acc = fminf(m_acc, __shfl_xor_sync(0xffffffffu, m_acc, o));
        const bool take = on >= 0 && (bn < 0 || od > bd || (od == bd && (ol > bl || (ol == bl && on < bn))));
        if (take) { bd = od; bl = ol; bn = on; }
    }
    // runner-up gap at the winning depth
    float tie = CUDART_INF_F;
    for (int n = lane; n < nn; n += 32) {
        const int dep = rm.depth[t0 + n + 1];
        const float gap = (LP[n] - a.logq_ref[bi * D + dep - 1]) - a.log_tau;
        if (bn >= 0 && n != bn && dep == bd && gap > 0.f) tie = fminf(tie, bl - LP[n]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tie = fminf(tie, __shfl_xor_sync(0xffffffffu, tie, o));

    if (out.node_LP) for (int n = lane; n < N; n += 32) out.node_LP[bi * N + n] = n < nn ? LP[n] : 0.f;
    if (out.node_lp) for (int n = lane; n < N; n += 32) out.node_lp[bi * N + n] = n < nn ? sc.node_lp[t0 + n + 1] : 0.f;
    for (int r = lane; r < R; r += 32) {
        const bool v = !bad && r < nrows;
        if (out.row_lse) out.row_lse[bi * R + r] = v ? sc.row_lse[t0 + r] : 0.f;
        if (out.row_cand) out.row_cand[bi * R + r] = v ? sc.row_cand[t0 + r] : 0;
        if (out.row_cand_lp) out.row_cand_lp[bi * R + r] = v ? sc.row_cand_lp[t0 + r] : 0.f;
    }
    if (lane == 0) {
        if (bad) {
            out.eta[bi] = 0; out.winner[bi] = -1; out.n_out[bi] = 0;
            if (out.margin) { out.margin[bi * 2] = CUDART_INF_F; out.margin[bi * 2 + 1] = CUDART_INF_F; }
            return;
        }
        const int eta = bd;
        out.eta[bi] = eta;
        out.winner[bi] = bn;
        out.n_out[bi] = eta + 1;
        int cur = bn;
        for (int i = eta - 1; i >= 0 && cur >= 0; --i) {
            out.path[bi * D + i] = cur;
            out.out_tok[bi * (D + 1) + i] = a.tok[bi * N + cur];
            out.out_lp[bi * (D + 1) + i] = sc.node_lp[t0 + cur + 1];
            cur = a.parent ? a.parent[bi * N + cur] : cur - 1;
        }
        const int wrow = t0 + bn + 1;
        out.out_tok[bi * (D + 1) + eta] = sc.row_cand[wrow];
        out.out_lp[bi * (D + 1) + eta] = sc.row_cand_lp[wrow];
        if (out.margin) { out.margin[bi * 2] = m_acc; out.margin[bi * 2 + 1] = tie; }
    }
}

cudaError_t launch_accept(const RowMeta& rm, const Scratch& sc, const AcceptArgs& a, const mtad_result& out,
                          cudaStream_t st) {
    accept_kernel<<<a.B, 32, 0, st>>>(rm, sc, a, out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// KV commit: node path[i] (slot L + 1 + path[i]) moves to position L + 1 + i.  One block per (layer, K|V, kv head,
// sequence) reads all rows it moves before writing any (a destination may be a later move's source).
// ---------------------------------------------------------------------------------------------------------------

__global__ void kv_commit_kernel(__nv_bfloat16* __restrict__ cache, const int32_t* __restrict__ call_seq,
                                 const int32_t* __restrict__ kv_len, mtad_result res, int D, int max_batch, int Hkv,
                                 int hd, long long cap) {
    const int bi = blockIdx.y;
    if (res.status[bi] != 0) return;
    const int eta = res.eta[bi];
    if (eta <= 0) return;
    const int seq = call_seq[bi];
    if ((unsigned)seq >= (unsigned)max_batch) return;
    const int L = kv_len[seq];
    // every source and destination row inside the cache, or nothing moves (seq_advance_kernel flags the sequence)
    if (eta > D || L < 0 || (long long)L + 1 + eta > cap) return;
    for (int r = 0; r < eta; ++r) {
        const int pn = res.path[bi * D + r];
        if (pn < 0 || (long long)L + 1 + pn >= cap) return;
    }
    const int head = blockIdx.x % Hkv;
    const int kv = (blockIdx.x / Hkv) & 1;
    const int layer = blockIdx.x / (2 * Hkv);
    __nv_bfloat16* base = cache + idx_cache(layer, max_batch, seq, kv, Hkv, head, cap, 0, hd);
    extern __shared__ __nv_bfloat16 buf[];
    for (int i = threadIdx.x; i < eta * hd; i += blockDim.x) {
        const int r = i / hd, j = i % hd;
        buf[i] = base[(size_t)(L + 1 + res.path[bi * D + r]) * hd + j];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < eta * hd; i += blockDim.x) {
        const int r = i / hd, j = i % hd;
        base[(size_t)(L + 1 + r) * hd + j] = buf[i];
    }
}

__global__ void seq_advance_kernel(SeqState s, const int32_t* __restrict__ call_seq, mtad_result res, int D, int B,
                                   int max_batch, long long cap) {
    const int bi = blockIdx.x * blockDim.x + threadIdx.x;
    if (bi >= B || res.status[bi] != 0) return;
    const int seq = call_seq[bi];
    const int eta = res.eta[bi];
    bool ok = (unsigned)seq < (unsigned)max_batch && eta >= 0 && eta <= D;
    if (ok) {
        const long long L = s.kv_len[seq];
        ok = L >= 0 && L + 1 + eta <= cap;
        for (int r = 0; r < eta && ok; ++r) {
            const int pn = res.path[bi * D + r];
            ok = pn >= 0 && L + 1 + pn < cap;
        }
    }
    if (!ok) { atomicOr(&res.status[bi], MTAD_ST_RANGE); return; }
    s.kv_len[seq] += eta + 1;
    s.root_tok[seq] = res.out_tok[bi * (D + 1) + eta];
}

cudaError_t launch_kv_commit(const ModelView& m, const SeqState& s, int B, const int32_t* call_seq_dev,
                             const mtad_result& res, int max_depth, cudaStream_t st) {
    dim3 grid(m.d.layers * 2 * m.d.n_kv_heads, B);
    const size_t smem = (size_t)(max_depth > 0 ? max_depth : 1) * m.d.head_dim * sizeof(__nv_bfloat16);
    kv_commit_kernel<<<grid, 128, smem, st>>>(static_cast<__nv_bfloat16*>(m.d.kv_cache), call_seq_dev, s.kv_len, res,
                                              max_depth, m.max_batch, m.d.n_kv_heads, m.d.head_dim,
                                              (long long)m.d.kv_capacity);
    return cudaGetLastError();
}

cudaError_t launch_seq_advance(const SeqState& s, int B, const int32_t* call_seq_dev, const mtad_result& res,
                               int max_depth, int max_batch, long long cap, cudaStream_t st) {
    seq_advance_kernel<<<1, 64, 0, st>>>(s, call_seq_dev, res, max_depth, B, max_batch, cap);
    return cudaGetLastError();
}

}  // namespace mtad
