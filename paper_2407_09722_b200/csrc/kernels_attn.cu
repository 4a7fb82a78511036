// Tree-masked attention of the draft rows against the KV cache: split-KV partial pass + deterministic combine.
// A row attends to the committed positions [0, L) of its sequence and to the cache slots L + s of the rows s that
// are its ancestors or itself (tree attention, Sec. 3.3 of the paper; the chain case is causal attention).
#include <math_constants.h>

#include "common.cuh"

namespace mtad {

template <int HD>
__global__ void __launch_bounds__(128) attn_partial_kernel(const float* __restrict__ qkv, int ldq,
                                                           const __nv_bfloat16* __restrict__ cache, RowMeta rm,
                                                           float* __restrict__ part, int layer, int max_batch, int Hq,
                                                           int Hkv, long long cap, int R, int nsplit, int chunk) {
    constexpr int TILE = MTAD_ATTN_TILE;           // 64 keys
    constexpr int PAD = HD + 8;                    // bf16 elements per staged row (16-byte pad against bank conflicts)
    constexpr int DPL = HD / 32;                   // output dims per lane
    __shared__ __align__(16) __nv_bfloat16 Ks[TILE * PAD];
    __shared__ __align__(16) __nv_bfloat16 Vs[TILE * PAD];
    __shared__ __align__(16) float qs[MTAD_ROW_CHUNK][HD];
    __shared__ float ps[4][TILE];

    const int h = blockIdx.x, sp = blockIdx.y, bi = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();          // q, the appended K/V rows and the row metadata come from the kernels before
    pdl_trigger();
    const int nrows = rm.n_rows[bi];
    if (nrows == 0) return;
    const int seq = rm.call_seq[bi];
    const int L = rm.kv_base[bi];
    const int nkeys = L + rm.n_spec[bi];
    const int c0 = sp * chunk;
    const int c1 = min(c0 + chunk, nkeys);
    const int g = h / (Hq / Hkv);
    const __nv_bfloat16* Kg = cache + idx_cache(layer, max_batch, seq, 0, Hkv, g, cap, 0, HD);
    const __nv_bfloat16* Vg = cache + idx_cache(layer, max_batch, seq, 1, Hkv, g, cap, 0, HD);

    for (int rc = 0; rc < nrows; rc += MTAD_ROW_CHUNK) {
        __syncthreads();
        for (int i = threadIdx.x; i < MTAD_ROW_CHUNK * HD; i += blockDim.x) {
            const int r = rc + i / HD;
            qs[i / HD][i % HD] = (r < nrows) ? qkv[(size_t)(bi * R + r) * ldq + h * HD + (i % HD)] : 0.f;
        }
        float m[2] = {-CUDART_INF_F, -CUDART_INF_F}, l[2] = {0.f, 0.f};
        float o[2][DPL];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int d = 0; d < DPL; ++d) o[a][d] = 0.f;

        for (int j0 = c0; j0 < c1; j0 += TILE) {
            __syncthreads();
            for (int i = threadIdx.x; i < TILE * (HD / 8); i += blockDim.x) {
                const int key = i / (HD / 8), piece = i % (HD / 8);
                uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
                if (j0 + key < c1) {
                    kv4 = *reinterpret_cast<const uint4*>(Kg + (size_t)(j0 + key) * HD + piece * 8);
                    vv4 = *reinterpret_cast<const uint4*>(Vg + (size_t)(j0 + key) * HD + piece * 8);
                }
                *reinterpret_cast<uint4*>(&Ks[key * PAD + piece * 8]) = kv4;
                *reinterpret_cast<uint4*>(&Vs[key * PAD + piece * 8]) = vv4;
            }
            __syncthreads();
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                const int rl = warp * 2 + a;                 // row within the chunk
                const int r = rc + rl;
                if (r >= nrows) continue;                    // warp-uniform
                const uint32_t* mk = rm.mask + (size_t)(bi * R + r) * MTAD_MASK_WORDS;
                float s[2];
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    const int key = lane + 32 * kk;
                    const int j = j0 + key;
                    float acc = 0.f;
#pragma unroll
                    for (int p = 0; p < HD / 8; ++p) {
                        const uint4 w = *reinterpret_cast<const uint4*>(&Ks[key * PAD + p * 8]);
                        const float4 qa = *reinterpret_cast<const float4*>(&qs[rl][p * 8]);
                        const float4 qb = *reinterpret_cast<const float4*>(&qs[rl][p * 8 + 4]);
                        acc = fmaf(qa.x, __uint_as_float(w.x << 16), acc);
                        acc = fmaf(qa.y, __uint_as_float(w.x & 0xffff0000u), acc);
                        acc = fmaf(qa.z, __uint_as_float(w.y << 16), acc);
                        acc = fmaf(qa.w, __uint_as_float(w.y & 0xffff0000u), acc);
                        acc = fmaf(qb.x, __uint_as_float(w.z << 16), acc);
                        acc = fmaf(qb.y, __uint_as_float(w.z & 0xffff0000u), acc);
                        acc = fmaf(qb.z, __uint_as_float(w.w << 16), acc);
                        acc = fmaf(qb.w, __uint_as_float(w.w & 0xffff0000u), acc);
                    }
                    bool vis = j < c1;
                    if (vis && j >= L) {
                        const int sr = j - L;
                        vis = (mk[sr >> 5] >> (sr & 31)) & 1u;
                    }
                    s[kk] = vis ? acc : -CUDART_INF_F;
                }
                float mx = fmaxf(s[0], s[1]);
#pragma unroll
                for (int ofs = 16; ofs > 0; ofs >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, ofs));
                const float mn = fmaxf(m[a], mx);
                float p0 = 0.f, p1 = 0.f, corr = 1.f;
                if (mn != -CUDART_INF_F) {
                    p0 = expf(s[0] - mn);
                    p1 = expf(s[1] - mn);
                    corr = expf(m[a] - mn);
                }
                float psum = p0 + p1;
#pragma unroll
                for (int ofs = 16; ofs > 0; ofs >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, ofs);
                l[a] = l[a] * corr + psum;
                m[a] = mn;
                __syncwarp();
                ps[warp][lane] = p0;
                ps[warp][lane + 32] = p1;
                __syncwarp();
#pragma unroll
                for (int d = 0; d < DPL; ++d) o[a][d] *= corr;
                for (int key = 0; key < TILE; ++key) {
                    const float p = ps[warp][key];
#pragma unroll
                    for (int d = 0; d < DPL; ++d)
                        o[a][d] = fmaf(p, __bfloat162float(Vs[key * PAD + lane * DPL + d]), o[a][d]);
                }
            }
        }
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int r = rc + warp * 2 + a;
            if (r >= nrows) continue;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            if (lane == 0) { dst[0] = m[a]; dst[1] = l[a]; }
#pragma unroll
            for (int d = 0; d < DPL; ++d) dst[2 + lane * DPL + d] = o[a][d];
        }
    }
}

// merge the split partials of one (row, head), in split order: the split weights exp(m_s - M) are computed once by
// the block, then every thread sums its output dimension over the splits with independent loads
template <int HD>
__global__ void attn_combine_kernel(const float* __restrict__ part, float* __restrict__ out, const int32_t* slot,
                                    int Hq, int nsplit, __nv_bfloat16* __restrict__ x, int terms) {
    const int t = blockIdx.x, h = blockIdx.y, d = threadIdx.x;
    pdl_wait();
    pdl_trigger();
    const size_t idx = ((size_t)t * Hq + h) * HD + d;
    const size_t xk = (size_t)Hq * HD;                          // operand rows of the O projection: see store_terms
    const size_t xidx = (size_t)t * terms * xk + (size_t)h * HD + d;
    float* dst = out + idx;
    if (slot[t] < 0) {
        *dst = 0.f;
        if (x) store_terms(0.f, x + xidx, xk, terms);
        return;
    }
    extern __shared__ float wsm[];                  // [nsplit] weights, then [1] the normaliser
    const float* p = part + idx_attn_part(t, Hq, h, nsplit, 0, HD);
    __shared__ float s_max;
    if (threadIdx.x < 32) {
        float M = -CUDART_INF_F;
        for (int s = threadIdx.x; s < nsplit; s += 32) M = fmaxf(M, p[(size_t)s * (HD + 2)]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        if (threadIdx.x == 0) s_max = M;
    }
    __syncthreads();
    const float M = s_max;
    for (int s = threadIdx.x; s < nsplit; s += blockDim.x) {
        const float ms = p[(size_t)s * (HD + 2)];
        wsm[s] = (ms == -CUDART_INF_F) ? 0.f : expf(ms - M);
    }
    __syncthreads();
    // A split without keys (a sequence shorter than its neighbours in the call) carries m = -inf, l = 0 and an
    // output part that nobody wrote: whatever an earlier call left there, possibly not finite, so it must not even be
    // multiplied by its zero weight.
    if (threadIdx.x == 0) {                          // fixed order: deterministic
        float lsum = 0.f;
        for (int s = 0; s < nsplit; ++s)
            if (wsm[s] != 0.f) lsum += p[(size_t)s * (HD + 2) + 1] * wsm[s];
        wsm[nsplit] = lsum;
    }
    float acc = 0.f;
#pragma unroll 8
    for (int s = 0; s < nsplit; ++s) {
        const float wgt = wsm[s];
        if (wgt != 0.f) acc += p[(size_t)s * (HD + 2) + 2 + d] * wgt;
    }
    __syncthreads();
    const float y = acc / wsm[nsplit];
    *dst = y;
    if (x) store_terms(y, x + xidx, xk, terms);
}

cudaError_t launch_attention(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int B, int R,
                             int nsplit, int chunk, bool emit_split, bool pdl, cudaStream_t st) {
    const int Hq = m.d.n_q_heads, Hkv = m.d.n_kv_heads, hd = m.d.head_dim;
    const int ldq = (Hq + 2 * Hkv) * hd;
    dim3 grid(Hq, nsplit, B);
    const __nv_bfloat16* cache = static_cast<const __nv_bfloat16*>(m.d.kv_cache);
    dim3 cgrid(B * R, Hq);
    cudaError_t e = cudaSuccess;
    __nv_bfloat16* xh = emit_split ? sc.xa : nullptr;
    const int xl = tc_terms(B * R);
    if (hd == 128) {
        e = launch_pdl(attn_partial_kernel<128>, grid, dim3(128), 0, st, pdl, sc.qkv, ldq, cache, rm, sc.attn_part, layer, m.max_batch, Hq,
                                                       Hkv, (long long)m.d.kv_capacity, R, nsplit, chunk);
        if (e == cudaSuccess)
            e = launch_pdl(attn_combine_kernel<128>, cgrid, dim3(128), (nsplit + 1) * sizeof(float), st, pdl, (const float*)sc.attn_part, sc.attn,
                           (const int32_t*)rm.slot, Hq, nsplit, xh, xl);
    } else if (hd == 64) {
        e = launch_pdl(attn_partial_kernel<64>, grid, dim3(128), 0, st, pdl, sc.qkv, ldq, cache, rm, sc.attn_part, layer, m.max_batch, Hq,
                                                      Hkv, (long long)m.d.kv_capacity, R, nsplit, chunk);
        if (e == cudaSuccess)
            e = launch_pdl(attn_combine_kernel<64>, cgrid, dim3(64), (nsplit + 1) * sizeof(float), st, pdl, (const float*)sc.attn_part, sc.attn,
                           (const int32_t*)rm.slot, Hq, nsplit, xh, xl);
    } else if (hd == 32) {
        e = launch_pdl(attn_partial_kernel<32>, grid, dim3(128), 0, st, pdl, sc.qkv, ldq, cache, rm, sc.attn_part, layer, m.max_batch, Hq,
                                                      Hkv, (long long)m.d.kv_capacity, R, nsplit, chunk);
        if (e == cudaSuccess)
            e = launch_pdl(attn_combine_kernel<32>, cgrid, dim3(32), (nsplit + 1) * sizeof(float), st, pdl, (const float*)sc.attn_part, sc.attn,
                           (const int32_t*)rm.slot, Hq, nsplit, xh, xl);
    } else {
        return cudaErrorInvalidValue;
    }
    return e;
}

cudaError_t launch_attention_combine(const ModelView& m, const RowMeta& rm, const Scratch& sc, int B, int R, int nsplit,
                                     bool emit_split, bool pdl, cudaStream_t st) {
    const int Hq = m.d.n_q_heads, hd = m.d.head_dim;
    dim3 cgrid(B * R, Hq);
    __nv_bfloat16* xh = emit_split ? sc.xa : nullptr;
    const int xl = tc_terms(B * R);
    if (hd == 128)
        return launch_pdl(attn_combine_kernel<128>, cgrid, dim3(128), (nsplit + 1) * sizeof(float), st, pdl, (const float*)sc.attn_part, sc.attn,
                          (const int32_t*)rm.slot, Hq, nsplit, xh, xl);
    if (hd == 64)
        return launch_pdl(attn_combine_kernel<64>, cgrid, dim3(64), (nsplit + 1) * sizeof(float), st, pdl, (const float*)sc.attn_part, sc.attn,
                          (const int32_t*)rm.slot, Hq, nsplit, xh, xl);
    return cudaErrorInvalidValue;
}

}  // namespace mtad
