// Tree-masked attention of the draft rows against the KV cache on tensor cores (warp-level mma.sync, bf16 x bf16
// -> fp32): the partial pass of the split-KV scheme.  One block owns (sequence, KV head, split of 64 keys): its K
// and V rows arrive in shared memory with cp.async (16-byte pieces, XOR-swizzled so that ldmatrix is conflict
// free) and every query row of the KV head's group - the draft rows of all its query heads, 16 per MMA tile - is
// run against them by one of the four warps.  fp32 queries and probabilities enter the tensor cores as bf16
// hi + lo pairs (two MMAs), so only the cache's own bf16 rounding remains.  A row sees the committed positions
// [0, L) and the draft rows among its ancestors and itself (Sec. 3.3 of the paper: tree attention).
#include <math_constants.h>

#include "common.cuh"

namespace mtad {
namespace {

constexpr int KT = 64;            // keys per block

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;                      // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma16816(float* d, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two fp32 values -> packed bf16 hi parts and packed bf16 lo parts (x = hi + lo up to ~2^-17 relative)
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 hx = __float2bfloat16_rn(x), hy = __float2bfloat16_rn(y);
    const __nv_bfloat16 lx = __float2bfloat16_rn(x - __bfloat162float(hx));
    const __nv_bfloat16 ly = __float2bfloat16_rn(y - __bfloat162float(hy));
    hi = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(lx) | ((uint32_t)__bfloat16_as_ushort(ly) << 16);
}

}  // namespace

// part[(t * Hq + h) * nsplit + split] = (running max m, sum l, unnormalised output o[HD]) of row t, head h over the
// keys of the split; attn_combine_kernel merges the splits in order.
template <int HD>
__global__ void __launch_bounds__(128) attn_mma_kernel(const float* __restrict__ qkv, int ldq,
                                                       const __nv_bfloat16* __restrict__ cache, RowMeta rm,
                                                       float* __restrict__ part, int layer, int max_batch, int Hq,
                                                       int Hkv, long long cap, int R, int nsplit) {
    constexpr int ROWB = HD * 2;          // bytes of one key row
    constexpr int CPR = HD / 8;           // 16-byte pieces per row
    constexpr int NDT = HD / 8;           // 8-wide output tiles over the head dim
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* Ks = smem;                               // [KT][HD] bf16, piece c of row k stored at piece c ^ (k & 7)
    uint8_t* Vs = smem + KT * ROWB;
    uint8_t* Qs = smem + 2 * KT * ROWB;               // per warp: [16][HD] hi then [16][HD] lo, same swizzle

    const int sp = blockIdx.x, g = blockIdx.y, bi = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();          // q, the appended K/V rows and the row metadata come from the kernels before
    pdl_trigger();
    const int nrows = rm.n_rows[bi];
    if (nrows == 0) return;
    const int L = rm.kv_base[bi];
    const int nkeys = L + nrows;
    const int k_begin = sp * KT;
    const int G = Hq / Hkv;
    if (k_begin >= nkeys) {
        // empty split: leave neutral partials so that the combine pass can read every split
        for (int i = threadIdx.x; i < G * nrows; i += blockDim.x) {
            const int h = g * G + i / nrows, r = i % nrows;
            float* dst = part + (((size_t)(bi * R + r) * Hq + h) * nsplit + sp) * (HD + 2);
            dst[0] = -CUDART_INF_F;
            dst[1] = 0.f;
        }
        return;
    }
    const int seq = rm.call_seq[bi];
    const __nv_bfloat16* Kg = cache + (((((size_t)layer * max_batch + seq) * 2 + 0) * Hkv + g) * cap) * HD;
    const __nv_bfloat16* Vg = cache + (((((size_t)layer * max_batch + seq) * 2 + 1) * Hkv + g) * cap) * HD;

    // ---- K and V rows of this split -> shared memory (zero-filled past the last key) ----
    for (int i = threadIdx.x; i < KT * CPR; i += blockDim.x) {
        const int key = i / CPR, c = i % CPR;
        const bool valid = k_begin + key < nkeys;
        const size_t goff = (size_t)(valid ? k_begin + key : 0) * HD + c * 8;
        const uint32_t soff = key * ROWB + ((c ^ (key & 7)) << 4);
        cp_async16(s_u32(Ks + soff), Kg + goff, valid);
        cp_async16(s_u32(Vs + soff), Vg + goff, valid);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");

    const int n_q = G * nrows;                        // query rows of this KV head: (head in group, draft row)
    const int n_mt = (n_q + 15) / 16;
    uint8_t* Qw = Qs + warp * (2 * 16 * ROWB);
    const int gq = lane >> 2, tq = lane & 3;          // fragment coordinates
    const bool spec = k_begin + KT > L;               // the split reaches into the draft rows: masks apply

    // 16 query rows of tile mt as bf16 hi / lo in this warp's slab
    auto stage_q = [&](int mt) {
        for (int i = lane; i < 16 * (HD / 2); i += 32) {
            const int row = i / (HD / 2), d2 = (i % (HD / 2)) * 2;
            const int qi = mt * 16 + row;
            float x = 0.f, y = 0.f;
            if (qi < n_q) {
                const int hg = qi / nrows, r = qi % nrows;
                const float2 v =
                    *reinterpret_cast<const float2*>(qkv + (size_t)(bi * R + r) * ldq + (g * G + hg) * HD + d2);
                x = v.x;
                y = v.y;
            }
            uint32_t hi, lo;
            split2(x, y, hi, lo);
            const uint32_t off = row * ROWB + (((d2 >> 3) ^ (row & 7)) << 4) + (d2 & 7) * 2;
            *reinterpret_cast<uint32_t*>(Qw + off) = hi;
            *reinterpret_cast<uint32_t*>(Qw + 16 * ROWB + off) = lo;
        }
    };
    if (warp < n_mt) stage_q(warp);                   // overlaps the K/V copies in flight
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();

    const uint32_t ks_base = s_u32(Ks), vs_base = s_u32(Vs), qh_base = s_u32(Qw), ql_base = s_u32(Qw + 16 * ROWB);
    const int lrow = lane & 7, lid = lane >> 3;       // ldmatrix: row within an 8x8 matrix, matrix id

    for (int mt = warp; mt < n_mt; mt += 4) {
        if (mt != warp) {
            __syncwarp();
            stage_q(mt);
        }
        __syncwarp();
        // ---- S = Q K^T over the 64 keys: 8 key tiles of 8, accumulated over HD in steps of 16 ----
        float sacc[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int c = 0; c < 4; ++c) sacc[n][c] = 0.f;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            uint32_t ah[4], al[4];
            {
                const int row = (lid & 1) * 8 + lrow, c = ks * 2 + (lid >> 1);
                const uint32_t off = row * ROWB + ((c ^ (row & 7)) << 4);
                ldsm4(qh_base + off, ah[0], ah[1], ah[2], ah[3]);
                ldsm4(ql_base + off, al[0], al[1], al[2], al[3]);
            }
#pragma unroll
            for (int n2 = 0; n2 < 4; ++n2) {
                const int key = n2 * 16 + (lid >> 1) * 8 + lrow, c = ks * 2 + (lid & 1);
                uint32_t b0, b1, b2, b3;
                ldsm4(ks_base + key * ROWB + ((c ^ (key & 7)) << 4), b0, b1, b2, b3);
                mma16816(sacc[2 * n2], ah, b0, b1);
                mma16816(sacc[2 * n2], al, b0, b1);
                mma16816(sacc[2 * n2 + 1], ah, b2, b3);
                mma16816(sacc[2 * n2 + 1], al, b2, b3);
            }
        }
        // ---- visibility: keys past the last one, and draft rows that are not ancestors-or-self ----
        // this thread holds rows gq and gq + 8 of the tile and, per key tile n, keys n * 8 + 2 * tq + {0, 1}
        const int qi0 = mt * 16 + gq, qi1 = qi0 + 8;
        const uint32_t* mk0 = nullptr;
        const uint32_t* mk1 = nullptr;
        if (spec) {
            if (qi0 < n_q) mk0 = rm.mask + (size_t)(bi * R + qi0 % nrows) * MTAD_MASK_WORDS;
            if (qi1 < n_q) mk1 = rm.mask + (size_t)(bi * R + qi1 % nrows) * MTAD_MASK_WORDS;
        }
        if (spec || k_begin + KT > nkeys) {
#pragma unroll
            for (int n = 0; n < 8; ++n)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int j = k_begin + n * 8 + 2 * tq + c;
                    bool v0 = j < nkeys, v1 = j < nkeys;
                    if (j >= L && j < nkeys) {
                        const int sr = j - L;
                        v0 = mk0 && ((mk0[sr >> 5] >> (sr & 31)) & 1u);
                        v1 = mk1 && ((mk1[sr >> 5] >> (sr & 31)) & 1u);
                    }
                    if (!v0) sacc[n][c] = -CUDART_INF_F;
                    if (!v1) sacc[n][2 + c] = -CUDART_INF_F;
                }
        }
        // ---- softmax numerators over this split ----
        float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            m0 = fmaxf(m0, fmaxf(sacc[n][0], sacc[n][1]));
            m1 = fmaxf(m1, fmaxf(sacc[n][2], sacc[n][3]));
        }
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
        float l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const float p0 = (m0 == -CUDART_INF_F) ? 0.f : expf(sacc[n][c] - m0);
                const float p1 = (m1 == -CUDART_INF_F) ? 0.f : expf(sacc[n][2 + c] - m1);
                sacc[n][c] = p0;
                sacc[n][2 + c] = p1;
                l0 += p0;
                l1 += p1;
            }
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        // ---- O = P V: P (hi + lo) straight from the score fragments, V through transposing ldmatrix ----
        float oacc[NDT][4];
#pragma unroll
        for (int n = 0; n < NDT; ++n)
#pragma unroll
            for (int c = 0; c < 4; ++c) oacc[n][c] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {
            uint32_t ph[4], pl[4];
            split2(sacc[2 * kk][0], sacc[2 * kk][1], ph[0], pl[0]);
            split2(sacc[2 * kk][2], sacc[2 * kk][3], ph[1], pl[1]);
            split2(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1], ph[2], pl[2]);
            split2(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3], ph[3], pl[3]);
#pragma unroll
            for (int d2 = 0; d2 < HD / 16; ++d2) {
                const int key = kk * 16 + (lid & 1) * 8 + lrow, c = d2 * 2 + (lid >> 1);
                uint32_t b0, b1, b2, b3;
                ldsm4t(vs_base + key * ROWB + ((c ^ (key & 7)) << 4), b0, b1, b2, b3);
                mma16816(oacc[2 * d2], ph, b0, b1);
                mma16816(oacc[2 * d2], pl, b0, b1);
                mma16816(oacc[2 * d2 + 1], ph, b2, b3);
                mma16816(oacc[2 * d2 + 1], pl, b2, b3);
            }
        }
        // ---- partials of the valid rows ----
        if (qi0 < n_q) {
            const int h = g * G + qi0 / nrows, r = qi0 % nrows;
            float* dst = part + (((size_t)(bi * R + r) * Hq + h) * nsplit + sp) * (HD + 2);
            if (tq == 0) { dst[0] = m0; dst[1] = l0; }
#pragma unroll
            for (int n = 0; n < NDT; ++n)
                *reinterpret_cast<float2*>(dst + 2 + n * 8 + 2 * tq) = make_float2(oacc[n][0], oacc[n][1]);
        }
        if (qi1 < n_q) {
            const int h = g * G + qi1 / nrows, r = qi1 % nrows;
            float* dst = part + (((size_t)(bi * R + r) * Hq + h) * nsplit + sp) * (HD + 2);
            if (tq == 0) { dst[0] = m1; dst[1] = l1; }
#pragma unroll
            for (int n = 0; n < NDT; ++n)
                *reinterpret_cast<float2*>(dst + 2 + n * 8 + 2 * tq) = make_float2(oacc[n][2], oacc[n][3]);
        }
    }
}

cudaError_t launch_attention_mma(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int B, int R,
                                 int nsplit, bool pdl, cudaStream_t st) {
    const int Hq = m.d.n_q_heads, Hkv = m.d.n_kv_heads, hd = m.d.head_dim;
    const int ldq = (Hq + 2 * Hkv) * hd;
    const __nv_bfloat16* cache = static_cast<const __nv_bfloat16*>(m.d.kv_cache);
    dim3 grid(nsplit, Hkv, B);
    if (hd == 128) {
        const size_t smem = 2 * KT * 256 + 4 * 2 * 16 * 256;       // K, V and one query slab per warp
        static bool set128 = false;
        if (!set128) {
            cudaError_t e = cudaFuncSetAttribute(attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 98304);
            if (e != cudaSuccess) return e;
            set128 = true;
        }
        return launch_pdl(attn_mma_kernel<128>, grid, dim3(128), smem, st, pdl, (const float*)sc.qkv, ldq, cache, rm,
                          sc.attn_part, layer, m.max_batch, Hq, Hkv, (long long)m.d.kv_capacity, R, nsplit);
    }
    if (hd == 64) {
        const size_t smem = 2 * KT * 128 + 4 * 2 * 16 * 128;
        return launch_pdl(attn_mma_kernel<64>, grid, dim3(128), smem, st, pdl, (const float*)sc.qkv, ldq, cache, rm,
                          sc.attn_part, layer, m.max_batch, Hq, Hkv, (long long)m.d.kv_capacity, R, nsplit);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mtad
