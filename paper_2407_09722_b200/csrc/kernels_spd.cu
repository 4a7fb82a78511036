// The rule of vanilla speculative decoding (Sec. 2.2 of the paper) as a second accept mode on the same verify
// forward: draft token i is accepted iff u_i < min(1, p_i(x_i) / q_i(x_i)); the first rejection ends the scan and
// its position is resampled from norm(max(0, p_i - q_i)); with every token accepted one more is drawn from the
// target's next row.  Works on the plain logits [rows, V] of the forward and the auxiliary model's normalised
// log-distributions at the draft positions (the caller's), one block per sequence.
#include <math_constants.h>

#include "common.cuh"

namespace mtad {

namespace {

struct Pick {
    float y;
    int v;
};
__device__ __forceinline__ bool ahead(const Pick& a, const Pick& b) { return a.y > b.y || (a.y == b.y && a.v < b.v); }

}  // namespace

__global__ void __launch_bounds__(1024) spd_accept_kernel(const float* __restrict__ logits, int V, RowMeta rm,
                                                          SpdArgs a, mtad_result out) {
    const int bi = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int R = a.R, g = R - 1, D = a.max_depth;
    __shared__ float s_red[32];
    __shared__ float s_lse[MTAD_MAX_DEPTH + 1];
    __shared__ int s_eta;
    __shared__ Pick s_p[1024];
    const int nrows = rm.n_rows[bi];
    if (out.status[bi] != 0 || nrows == 0) {
        if (tid == 0) { out.eta[bi] = 0; out.winner[bi] = -1; out.n_out[bi] = 0; }
        return;
    }
    const float* z0 = logits + (size_t)bi * R * V;
    // log-sum-exp of every row (fixed combination order)
    for (int r = 0; r < R; ++r) {
        const float* z = z0 + (size_t)r * V;
        float m = -CUDART_INF_F;
        for (int v = tid; v < V; v += blockDim.x) m = fmaxf(m, z[v]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) s_red[warp] = m;
        __syncthreads();
        m = s_red[0];
        for (int w = 1; w < 32; ++w) m = fmaxf(m, s_red[w]);
        __syncthreads();
        float sum = 0.f;
        for (int v = tid; v < V; v += blockDim.x) sum += expf(z[v] - m);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) s_red[warp] = sum;
        __syncthreads();
        if (tid == 0) {
            float acc = 0.f;
            for (int w = 0; w < 32; ++w) acc += s_red[w];
            s_lse[r] = m + logf(acc);
        }
        __syncthreads();
    }
    // rows of NaN logits: flag the sequence and accept nothing, as the other modes do
    bool finite = true;
    for (int r = 0; r < R; ++r) finite = finite && isfinite(s_lse[r]);
    if (!finite) {
        if (tid == 0) {
            atomicOr(&out.status[bi], MTAD_ST_NONFINITE);
            out.eta[bi] = 0; out.winner[bi] = -1; out.n_out[bi] = 0;
        }
        return;
    }
    // the accept scan: stops at the first rejection
    if (tid == 0) {
        int eta = g;
        float margin = CUDART_INF_F;
        for (int i = 0; i < g; ++i) {
            const int x = a.tok[bi * g + i];
            const float lp = z0[(size_t)i * V + x] - s_lse[i];
            const float ratio = fminf(0.f, lp - a.logq_rows[((size_t)bi * g + i) * V + x]);
            const float lu = logf(a.accept_uniform[bi * g + i]);
            margin = fminf(margin, fabsf(lu - ratio));
            if (!(lu < ratio)) { eta = i; break; }
            out.path[bi * D + i] = i;
            out.out_tok[bi * (D + 1) + i] = x;
            out.out_lp[bi * (D + 1) + i] = lp;
        }
        s_eta = eta;
        out.eta[bi] = eta;
        out.winner[bi] = eta - 1;
        out.n_out[bi] = eta + 1;
        if (out.margin) { out.margin[bi * 2] = margin; out.margin[bi * 2 + 1] = CUDART_INF_F; }
    }
    __syncthreads();
    // the last token: from the target's row after the chain, or from the positive part of p - q at the rejection
    const int eta = s_eta;
    const float* z = z0 + (size_t)eta * V;
    const float lse = s_lse[eta];
    const float* lq = eta < g ? a.logq_rows + ((size_t)bi * g + eta) * V : nullptr;
    const float* u = a.resample_uniform + (size_t)bi * V;
    Pick best{-CUDART_INF_F, 0x7fffffff};
    for (int v = tid; v < V; v += blockDim.x) {
        float s;
        if (lq) {
            const float w = expf(z[v] - lse) - expf(lq[v]);
            s = w > 0.f ? logf(w) : -CUDART_INF_F;
        } else {
            s = z[v] - lse;
        }
        if (s == -CUDART_INF_F) continue;
        const Pick c{s - logf(-logf(u[v])), v};
        if (ahead(c, best)) best = c;
    }
    s_p[tid] = best;
    __syncthreads();
    for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
        if (tid < o && ahead(s_p[tid + o], s_p[tid])) s_p[tid] = s_p[tid + o];
        __syncthreads();
    }
    if (tid == 0) {
        // (p == q everywhere leaves no residual mass; the ratio test cannot reject then, so a row is always found)
        const int t = s_p[0].v == 0x7fffffff ? 0 : s_p[0].v;
        out.out_tok[bi * (D + 1) + eta] = t;
        out.out_lp[bi * (D + 1) + eta] = z[t] - lse;
    }
    // optional per-row outputs of the result struct
    if (out.row_lse) for (int r = tid; r < R; r += blockDim.x) out.row_lse[bi * R + r] = r < nrows ? s_lse[r] : 0.f;
    if (out.node_lp) for (int n = tid; n < g; n += blockDim.x)
        out.node_lp[bi * g + n] = z0[(size_t)n * V + a.tok[bi * g + n]] - s_lse[n];
}

cudaError_t launch_spd_accept(const ModelView& m, const RowMeta& rm, const Scratch& sc, const SpdArgs& a,
                              const mtad_result& out, cudaStream_t st) {
    spd_accept_kernel<<<a.B, 1024, 0, st>>>(sc.logits, m.d.vocab, rm, a, out);
    return cudaGetLastError();
}

}  // namespace mtad
