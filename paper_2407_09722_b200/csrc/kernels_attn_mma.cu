// Tree-masked attention of the draft rows against the KV cache on tensor cores (warp-level mma.sync, bf16 x bf16
// -> fp32): the partial pass of the split-KV scheme.  One block owns (sequence, KV head, run of 64-key tiles): its K
// and V rows arrive in shared memory by TMA (64 x 64 boxes of a map over the whole cache, 128-byte swizzle so that
// ldmatrix is conflict free; a block that walks several tiles keeps up to three in flight, and the tiles that hold
// only committed positions are requested before the block waits for the kernel in front of it), and every query
// row of the KV head's group - the draft rows of all its query heads, 16 per MMA tile - is run against them by one
// of the four warps.  fp32 queries and probabilities enter the tensor cores as bf16 hi + lo pairs (two MMAs, or one
// MMA tile that carries both when the group has at most eight query rows), so only the cache's own bf16 rounding
// remains.  A row sees the committed positions [0, L) and the draft rows among its ancestors and itself (Sec. 3.3
// of the paper: tree attention).  Waits on the tile barriers are bounded and end in MTAD_ST_TIMEOUT.
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

// ---- TMA + mbarrier (K/V tiles) ----
constexpr uint32_t ATTN_WAIT_LIMIT = 1u << 22;
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded: false when the limit ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < ATTN_WAIT_LIMIT; ++it) {
        if (mbar_test(bar, parity)) return true;
        if (it > 64) __nanosleep(32);
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
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
// keys of the split; attn_combine_kernel merges the splits in order.  q_hi / q_lo hold the query rows times
// log2(e) / sqrt(HD), so the softmax numerators are exp2(s - m); m is stored back in natural-log units.
template <int HD, int CNT, bool PACK>
__global__ void __launch_bounds__(CNT == 4 ? 192 : 128, CNT == 1 ? 4 : (CNT == 4 ? 2 : 3)) attn_mma_kernel(const __grid_constant__ CUtensorMap kvmap,
                                                          const __nv_bfloat16* __restrict__ q_hi,
                                                          const __nv_bfloat16* __restrict__ q_lo, RowMeta rm,
                                                          float* __restrict__ part, int layer, int max_batch, int Hq,
                                                          int Hkv, int R, int nsplit, int nslab, int nsp, int nb,
                                                          int early, uint32_t* status) {
    constexpr int ROWB = HD * 2;          // bytes of one key row
    constexpr int CPR = HD / 8;           // 16-byte pieces per row
    constexpr int NDT = HD / 8;           // 8-wide output tiles over the head dim
    constexpr int SLAB = 2 * 16 * ROWB;   // one query tile: 16 rows hi, then 16 rows lo
    constexpr int PARK = HD + 8;          // row stride (floats) of a parked output tile
    constexpr float LN2 = 0.6931471805599453f;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // nb K/V buffers, each K then V as TMA boxes of [KT keys][64 elements = 128 bytes] (two per tensor at head_dim
    // 128), 128-byte swizzle: 16-byte piece c of key k sits at piece c ^ (k & 7) of its row; then the query tiles
    uint8_t* Qs = smem + nb * 2 * KT * ROWB;          // nslab query tiles, [16 rows][HD], same XOR on the piece index
    float* ml = reinterpret_cast<float*>(Qs + nslab * SLAB);           // [4 warps][16 rows][m, l]
    uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(ml) + 1536);   // one barrier per buffer
    if (threadIdx.x == 0) {
        for (int b = 0; b < nb; ++b) mbar_init(s_u32(&full[b]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int sp = blockIdx.x, g = blockIdx.y, bi = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // q and the appended K/V rows come from the kernel before; with `early` the row metadata is older than that
    // (any layer but the first), so the committed part of the cache can be requested before waiting for it
    if (!early) { pdl_wait(); pdl_trigger(); }
    const int nrows = __ldcg(rm.n_rows + bi);         // past L1: these words are rewritten by every step
    if (nrows == 0) return;
    const int L = __ldcg(rm.kv_base + bi);
    const int nkeys = L + __ldcg(rm.n_spec + bi);
    const int n_tiles = (nkeys + KT - 1) / KT;        // 64-key tiles of this sequence
    const int tile_begin = sp * nsp, tile_end = min(tile_begin + nsp, n_tiles);
    const int G = Hq / Hkv;
    const int n_q = G * nrows;                        // query rows of this KV head: (head in group, draft row)
    if (tile_begin >= n_tiles) {
        // empty split: leave neutral partials so that the combine pass can read every split
        if (early) { pdl_wait(); pdl_trigger(); }
        for (int i = threadIdx.x; i < n_q; i += blockDim.x) {
            const int h = g * G + i / nrows, r = i % nrows;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            dst[0] = -CUDART_INF_F;
            dst[1] = 0.f;
        }
        return;
    }
    const int seq = __ldcg(rm.call_seq + bi);
    const int plane_k = ((layer * max_batch + seq) * 2 + 0) * Hkv + g, plane_v = plane_k + Hkv;
    const int n_mt = (n_q + 15) / 16;
    // With fewer than three query tiles the warps share a tile and split its 64 keys instead (kparts warps per
    // tile, merged through shared memory below); otherwise every warp runs whole tiles against all 64 keys.
    // (compile-time: the launch picks CNT from its largest sequence; with CNT = 1 the kernel needs 126 registers
    // instead of 168 and its unrolled loops carry no dead iterations)
    constexpr int cnt = CNT;                          // 16-key groups per task
    constexpr int kparts = 4 / CNT;
    // PACK (at most eight query rows per KV head in the whole launch): the hi parts take rows 0..7 of the 16-row MMA
    // tile and the lo parts rows 8..15, so one MMA multiplies both and a thread (which holds rows g and g + 8) adds
    // the two products of its query row: half the MMAs, one softmax row per thread
    constexpr bool packed = PACK;
    const int kt0 = (warp % kparts) * cnt;            // first 16-key group of this warp's tasks
    // whole-tile mode with a warp for every query tile: the warp keeps its tile's running softmax state and output in
    // registers over all key tiles of the block and writes one partial at the end; with more query tiles than warps
    // the block owns a single key tile (the launch sets nsp = 1) and every (query tile, key tile) is a partial
    const bool persist = kparts == 1 && n_mt <= (int)(blockDim.x >> 5);

    // query tile mt -> slab (16-byte async copies by `nthr` threads; rows past the last query are zero-filled)
    auto stage_q = [&](int mt, int slab, int tid, int nthr) {
        uint8_t* dst = Qs + slab * SLAB;
        for (int i = tid; i < 2 * 16 * CPR; i += nthr) {
            const int which = i / (16 * CPR), row = (i / CPR) % 16, c = i % CPR;
            const int qi = mt * 16 + row;
            const bool valid = qi < n_q;
            const int hg = valid ? qi / nrows : 0, r = valid ? qi % nrows : 0;
            const __nv_bfloat16* src = (which ? q_lo : q_hi) + ((size_t)(bi * R + r) * Hq + g * G + hg) * HD + c * 8;
            if (packed) {                             // query row `row` < 8: hi -> tile row `row`, lo -> tile row 8 + row
                if (row < 8)
                    cp_async16(s_u32(dst + (which * 8 + row) * ROWB + ((c ^ (row & 7)) << 4)), src, valid);
                continue;
            }
            cp_async16(s_u32(dst + which * 16 * ROWB + row * ROWB + ((c ^ (row & 7)) << 4)), src, valid);
        }
    };
    // K and V rows of one 64-key tile -> buffer `buf`, by TMA (one thread): positions past the cache capacity come
    // back as zeros, positions between the last key and the tile's end hold whatever the cache holds there
    constexpr uint32_t TILE_BYTES = 2 * KT * ROWB;
    auto load_kv = [&](int tile, int buf) {
        const uint32_t bar = s_u32(&full[buf]);
        const uint32_t dst = s_u32(smem + buf * TILE_BYTES);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the buffer's last readers were ldmatrix
        mbar_expect_tx(bar, TILE_BYTES);
#pragma unroll
        for (int h = 0; h < HD / 64; ++h) {
            tma_load_3d(dst + h * (KT * 128), &kvmap, bar, h * 64, tile * KT, plane_k);
            tma_load_3d(dst + KT * ROWB + h * (KT * 128), &kvmap, bar, h * 64, tile * KT, plane_v);
        }
    };
    // byte offset of 16-byte piece c of key `key` inside a K or V tile
    auto kv_off = [](int key, int c) -> uint32_t {
        return (uint32_t)((c >> 3) * (KT * 128) + key * 128 + (((c & 7) ^ (key & 7)) << 4));
    };
    int n_issued = 0;                                 // tiles requested so far (thread 0)
    // prologue: the first tiles of the block (one, or as many as the prefetch distance nb - 1)
    const int pd = nb - 1;
    const int n_pro = min(max(pd, 1), tile_end - tile_begin);
    uint32_t asked = 0;
    if (early) {
        if (threadIdx.x == 0)
            for (int j = 0; j < n_pro; ++j)
                if ((tile_begin + j + 1) * KT <= L) {      // committed positions only
                    load_kv(tile_begin + j, j);
                    asked |= 1u << j;
                }
        pdl_wait();
        pdl_trigger();
    }
    if (kparts > 1) {
        for (int mt = 0; mt < n_mt; ++mt) stage_q(mt, mt, threadIdx.x, blockDim.x);
    } else if (warp < n_mt) {
        stage_q(warp, warp, lane, 32);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int j = 0; j < n_pro; ++j)
            if (!((asked >> j) & 1u)) load_kv(tile_begin + j, j);
        n_issued = n_pro;
    }

    const int gq = lane >> 2, tq = lane & 3;          // fragment coordinates
    const int lrow = lane & 7, lid = lane >> 3;       // ldmatrix: row within an 8x8 matrix, matrix id
    // running softmax state of this thread's two rows (gq and gq + 8), in log2 units
    float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;
    float oacc[NDT][4];
#pragma unroll
    for (int n = 0; n < NDT; ++n)
#pragma unroll
        for (int c = 0; c < 4; ++c) oacc[n][c] = 0.f;

  for (int tile = tile_begin; tile < tile_end; ++tile) {
    const int t = tile - tile_begin, buf = t % nb;
    // request tile t + pd into the buffer that tile t - 1 has left (all warps passed the barrier that ends it)
    if (pd > 0 && tile + pd < tile_end && threadIdx.x == 0) {
        load_kv(tile + pd, (t + pd) % nb);
        n_issued = t + pd + 1;
    }
    if (pd == 0 && t > 0 && threadIdx.x == 0) {       // single buffer: the tile is requested when its turn comes
        load_kv(tile, 0);
        n_issued = t + 1;
    }
    if (t == 0) asm volatile("cp.async.wait_group 0;" ::: "memory");      // this thread's query pieces
    bool ok = mbar_wait(s_u32(&full[buf]), (uint32_t)(t / nb) & 1u);
    if (ok && tile * KT + KT > nkeys) {
        // rows past the last key: their scores are masked below, but 0 x (stale V) must not make a NaN
        const int first = max(nkeys - tile * KT, 0);
        uint8_t* Vs = smem + buf * TILE_BYTES + KT * ROWB;
        for (int i = threadIdx.x; i < (KT - first) * CPR; i += blockDim.x) {
            const int key = first + i / CPR, c = i % CPR;
            *reinterpret_cast<uint4*>(Vs + kv_off(key, c)) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    if (__syncthreads_or(ok ? 0 : 1)) {
        // a tile did not arrive within the limit: flag it, let the copies in flight land (bounded), leave neutral
        // partials so that the combine pass reads defined values
        if (threadIdx.x == 0) {
            if (status) atomicOr(status + bi, MTAD_ST_TIMEOUT);
            for (int tt = t; tt < n_issued; ++tt) mbar_wait(s_u32(&full[tt % nb]), (uint32_t)(tt / nb) & 1u);
        }
        for (int i = threadIdx.x; i < n_q; i += blockDim.x) {
            const int h = g * G + i / nrows, r = i % nrows;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            dst[0] = -CUDART_INF_F;
            dst[1] = 0.f;
        }
        __syncthreads();
        return;
    }
    const int k_begin = tile * KT;
    const bool spec = k_begin + KT > L;               // the tile reaches into the draft rows: masks apply
    const uint32_t ks_base = s_u32(smem + buf * TILE_BYTES), vs_base = ks_base + KT * ROWB;

    // (whole-tile mode: the block has four to six warps, one query tile per warp and round)
    const int mt_step = kparts > 1 ? 4 / kparts : (int)(blockDim.x >> 5);
    for (int mt = warp / kparts; mt < n_mt; mt += mt_step) {
        const int slab = kparts > 1 ? mt : warp;
        if (kparts == 1 && mt != warp) {
            __syncwarp();                             // the previous tile's fragments have been read
            stage_q(mt, slab, lane, 32);
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_all;" ::: "memory");
            __syncwarp();
        }
        if (kparts == 1 && (t == 0 || !persist)) {    // whole tiles: fresh state, unless this warp keeps its one query tile
            m0 = -CUDART_INF_F; m1 = -CUDART_INF_F; l0 = 0.f; l1 = 0.f;
#pragma unroll
            for (int n = 0; n < NDT; ++n)
#pragma unroll
                for (int c = 0; c < 4; ++c) oacc[n][c] = 0.f;
        }
        const uint32_t qh_base = s_u32(Qs + slab * SLAB), ql_base = qh_base + 16 * ROWB;
        // ---- S = Q K^T over this task's keys: key tiles of 8, accumulated over HD in steps of 16 ----
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
                if (!packed) ldsm4(ql_base + off, al[0], al[1], al[2], al[3]);
            }
#pragma unroll
            for (int n2 = 0; n2 < 4; ++n2) {
                if (n2 < cnt) {                       // sacc[2 * n2 ..] covers keys (kt0 + n2) * 16 ..
                    const int key = (kt0 + n2) * 16 + (lid >> 1) * 8 + lrow, c = ks * 2 + (lid & 1);
                    uint32_t b0, b1, b2, b3;
                    ldsm4(ks_base + kv_off(key, c), b0, b1, b2, b3);
                    mma16816(sacc[2 * n2], ah, b0, b1);
                    mma16816(sacc[2 * n2 + 1], ah, b2, b3);
                    if (!packed) {
                        mma16816(sacc[2 * n2], al, b0, b1);
                        mma16816(sacc[2 * n2 + 1], al, b2, b3);
                    }
                }
            }
        }
        if (packed) {
            // hi product (row g) + lo product (row g + 8) = the score of query row g; the second row is no query
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                sacc[n][0] += sacc[n][2];
                sacc[n][1] += sacc[n][3];
                sacc[n][2] = -CUDART_INF_F;
                sacc[n][3] = -CUDART_INF_F;
            }
        }
        // ---- visibility: keys past the last one, and draft rows that are not ancestors-or-self ----
        // this thread holds rows gq and gq + 8 of the tile and, per key tile n, keys n * 8 + 2 * tq + {0, 1}
        const int qi0 = mt * 16 + gq, qi1 = qi0 + 8;
        const int kfirst = k_begin + kt0 * 16;
        if (kfirst + cnt * 16 > min(L, nkeys)) {
            const uint32_t* mk0 = (spec && qi0 < n_q) ? rm.mask + (size_t)(bi * R + qi0 % nrows) * MTAD_MASK_WORDS : nullptr;
            const uint32_t* mk1 = (spec && qi1 < n_q) ? rm.mask + (size_t)(bi * R + qi1 % nrows) * MTAD_MASK_WORDS : nullptr;
#pragma unroll
            for (int n = 0; n < 8; ++n)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    if (n < 2 * cnt) {
                        const int j = kfirst + n * 8 + 2 * tq + c;
                        bool v0 = j < nkeys, v1 = v0;
                        if (v0 && j >= L) {
                            const int sr = j - L;
                            v0 = mk0 && ((mk0[sr >> 5] >> (sr & 31)) & 1u);
                            v1 = mk1 && ((mk1[sr >> 5] >> (sr & 31)) & 1u);
                        }
                        if (!v0) sacc[n][c] = -CUDART_INF_F;
                        if (!v1) sacc[n][2 + c] = -CUDART_INF_F;
                    }
                }
        }
        // ---- online softmax over this task's keys: new maximum, rescale the running sums, numerators ----
        float t0 = -CUDART_INF_F, t1 = -CUDART_INF_F;
#pragma unroll
        for (int n = 0; n < 8; ++n)
            if (n < 2 * cnt) {
                t0 = fmaxf(t0, fmaxf(sacc[n][0], sacc[n][1]));
                t1 = fmaxf(t1, fmaxf(sacc[n][2], sacc[n][3]));
            }
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1));
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
        const float n0 = fmaxf(m0, t0), n1 = fmaxf(m1, t1);
        const float c0 = (n0 == -CUDART_INF_F) ? 1.f : exp2f(m0 - n0);
        const float c1 = packed ? c0 : ((n1 == -CUDART_INF_F) ? 1.f : exp2f(m1 - n1));   // packed: both rows are one query
        const float s0 = (n0 == -CUDART_INF_F) ? 0.f : n0, s1 = (n1 == -CUDART_INF_F) ? 0.f : n1;
        m0 = n0; m1 = n1;
        float r0 = 0.f, r1 = 0.f;
#pragma unroll
        for (int n = 0; n < 8; ++n)
            if (n < 2 * cnt) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float p0 = exp2f(sacc[n][c] - s0), p1 = exp2f(sacc[n][2 + c] - s1);   // exp2(-inf) = 0
                    sacc[n][c] = p0;
                    sacc[n][2 + c] = p1;
                    r0 += p0;
                    r1 += p1;
                }
            }
        r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
        r0 += __shfl_xor_sync(0xffffffffu, r0, 2);
        r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
        r1 += __shfl_xor_sync(0xffffffffu, r1, 2);
        l0 = l0 * c0 + r0;
        l1 = l1 * c1 + r1;
#pragma unroll
        for (int n = 0; n < NDT; ++n) {
            oacc[n][0] *= c0; oacc[n][1] *= c0;
            oacc[n][2] *= c1; oacc[n][3] *= c1;
        }
        // ---- O += P V: P (hi + lo) straight from the score fragments, V through transposing ldmatrix ----
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {
            if (kk < cnt) {
                uint32_t ph[4], pl[4];
                split2(sacc[2 * kk][0], sacc[2 * kk][1], ph[0], pl[0]);
                split2(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1], ph[2], pl[2]);
                if (packed) {                         // rows 8..15 of the probability tile carry the lo parts
                    ph[1] = pl[0];
                    ph[3] = pl[2];
                } else {
                    split2(sacc[2 * kk][2], sacc[2 * kk][3], ph[1], pl[1]);
                    split2(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3], ph[3], pl[3]);
                }
#pragma unroll
                for (int d2 = 0; d2 < HD / 16; ++d2) {
                    const int key = (kt0 + kk) * 16 + (lid & 1) * 8 + lrow, c = d2 * 2 + (lid >> 1);
                    uint32_t b0, b1, b2, b3;
                    ldsm4t(vs_base + kv_off(key, c), b0, b1, b2, b3);
                    mma16816(oacc[2 * d2], ph, b0, b1);
                    mma16816(oacc[2 * d2 + 1], ph, b2, b3);
                    if (!packed) {
                        mma16816(oacc[2 * d2], pl, b0, b1);
                        mma16816(oacc[2 * d2 + 1], pl, b2, b3);
                    }
                }
            }
        }
        if (kparts > 1) break;                        // one task per warp: merged below
        if (persist && tile + 1 < tile_end) break;    // the warp's query tile goes on to the block's next key tile
        // ---- partials of the valid rows ----
        if (qi0 < n_q) {
            const int h = g * G + qi0 / nrows, r = qi0 % nrows;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            if (tq == 0) { dst[0] = m0 * LN2; dst[1] = l0; }
#pragma unroll
            for (int n = 0; n < NDT; ++n)
                *reinterpret_cast<float2*>(dst + 2 + n * 8 + 2 * tq) = make_float2(oacc[n][0], oacc[n][1]);
        }
        if (qi1 < n_q) {
            const int h = g * G + qi1 / nrows, r = qi1 % nrows;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            if (tq == 0) { dst[0] = m1 * LN2; dst[1] = l1; }
#pragma unroll
            for (int n = 0; n < NDT; ++n)
                *reinterpret_cast<float2*>(dst + 2 + n * 8 + 2 * tq) = make_float2(oacc[n][2], oacc[n][3]);
        }
    }
    __syncthreads();                                  // this tile's buffer is refilled by the next iteration's request
  }
    if (kparts > 1) {
        // ---- key-split tiles: park each warp's (m, l, o) over the K/V/Q area, then merge the parts in key order --
        float* ow = reinterpret_cast<float*>(smem) + warp * 16 * PARK;
        if (tq == 0) {
            ml[(warp * 16 + gq) * 2] = m0;     ml[(warp * 16 + gq) * 2 + 1] = l0;
            ml[(warp * 16 + gq + 8) * 2] = m1; ml[(warp * 16 + gq + 8) * 2 + 1] = l1;
        }
#pragma unroll
        for (int n = 0; n < NDT; ++n) {
            if (packed) {                             // hi-part sums (row g) + lo-part sums (row g + 8)
                *reinterpret_cast<float2*>(ow + gq * PARK + n * 8 + 2 * tq) =
                    make_float2(oacc[n][0] + oacc[n][2], oacc[n][1] + oacc[n][3]);
                continue;
            }
            *reinterpret_cast<float2*>(ow + gq * PARK + n * 8 + 2 * tq) = make_float2(oacc[n][0], oacc[n][1]);
            *reinterpret_cast<float2*>(ow + (gq + 8) * PARK + n * 8 + 2 * tq) = make_float2(oacc[n][2], oacc[n][3]);
        }
        __syncthreads();
        // per (row, part) weight exp2(m_part - M) and the row's sum first, then the outputs of the valid rows only
        float* wq = ml + 4 * 16 * 2;                  // [32 rows][4 parts] weights, then [32] maxima and [32] sums
        float* wM = wq + 2 * 16 * 4;
        float* wl = wM + 2 * 16;
        for (int qi = threadIdx.x; qi < n_q; qi += blockDim.x) {
            const int w0 = (qi >> 4) * kparts, row = qi & 15;
            float M = -CUDART_INF_F;
            for (int q = 0; q < kparts; ++q) M = fmaxf(M, ml[((w0 + q) * 16 + row) * 2]);
            float lsum = 0.f;
            for (int q = 0; q < kparts; ++q) {                       // key order: deterministic
                const float mq = ml[((w0 + q) * 16 + row) * 2];
                const float wgt = (mq == -CUDART_INF_F) ? 0.f : exp2f(mq - M);
                wq[qi * 4 + q] = wgt;
                lsum += ml[((w0 + q) * 16 + row) * 2 + 1] * wgt;
            }
            wM[qi] = M;
            wl[qi] = lsum;
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < n_q * HD; idx += blockDim.x) {
            const int qi = idx / HD, d = idx % HD;
            const int w0 = (qi >> 4) * kparts, row = qi & 15;
            float acc = 0.f;
            for (int q = 0; q < kparts; ++q)
                acc += (reinterpret_cast<const float*>(smem) + (w0 + q) * 16 * PARK)[row * PARK + d] * wq[qi * 4 + q];
            const int h = g * G + qi / nrows, r = qi % nrows;
            float* dst = part + idx_attn_part(bi * R + r, Hq, h, nsplit, sp, HD);
            dst[2 + d] = acc;
            if (d == 0) { dst[0] = wM[qi] * LN2; dst[1] = wl[qi]; }
        }
    }
}

namespace {
size_t attn_smem(int hd, int nslab, int nb) {
    // K/V ring, query tiles, merge scratch and barriers, and room to align the ring to 1024 bytes (TMA swizzle)
    return (size_t)nb * 2 * KT * hd * 2 + (size_t)nslab * 2 * 16 * hd * 2 + 2048 + 1024;
}
// K/V buffers of a block that walks several tiles: three (two tiles in flight behind the one being computed) when
// two such blocks fit an SM, else two
// With many (sequence, KV head) pairs - a batch - more resident warps are worth more than the third buffer: two
// buffers, three blocks per SM (13B batch: attention 6.0 -> 5.4 ms per step; the single 7B chain loses 1 % that way).
int attn_ring(int hd, int nslab, long long pairs) {
    return (pairs <= 148 && 2 * (attn_smem(hd, nslab, 3) + 1024) <= 228 * 1024) ? 3 : 2;
}
}  // namespace

int attention_mma_tiles_per_block(const ModelView& m, int B, int R, long long keys) {
    // with at most two query tiles per KV head a block walks several 64-key tiles, all blocks resident in a single
    // wave (two per SM with a ring of three buffers at head_dim 128, else three); larger trees take one tile per block
    const int n_mt_max = ((m.d.n_q_heads / m.d.n_kv_heads) * R + 15) / 16;
    if (n_mt_max > 6) return 1;
    if (n_mt_max > 2) {
        // three to six query tiles: a warp per tile, two K/V buffers, two blocks per SM, all blocks in one wave
        const long long tiles = (keys + KT - 1) / KT * m.d.n_kv_heads * B;
        const long long nsp = (tiles + 2 * 148 - 1) / (2 * 148);
        return (int)(nsp < 1 ? 1 : (nsp > 64 ? 64 : nsp));
    }
    const int ring = attn_ring(m.d.head_dim, n_mt_max, (long long)m.d.n_kv_heads * B);
    const int per_sm = (ring == 3 && m.d.head_dim == 128) ? 2 : 3;
    const long long tiles = (keys + KT - 1) / KT * m.d.n_kv_heads * B;
    const long long nsp = (tiles + per_sm * 148 - 1) / (per_sm * 148);
    return (int)(nsp < 1 ? 1 : (nsp > 64 ? 64 : nsp));
}

cudaError_t launch_attention_mma(const ModelView& m, int layer, const RowMeta& rm, const Scratch& sc, int B, int R,
                                 int nsplit, int nsp, uint32_t* status, bool pdl, cudaStream_t st) {
    const int Hq = m.d.n_q_heads, Hkv = m.d.n_kv_heads, hd = m.d.head_dim;
    if (!m.kv_map_ok) return cudaErrorInvalidValue;
    // query tiles kept in shared memory: all of them (at most two) when the warps split keys, else one per warp
    const int n_mt_max = ((Hq / Hkv) * R + 15) / 16;
    // whole-tile mode with five or six query tiles per KV head: one warp per tile instead of four warps in two rounds
    // (a 64-node tree plus its root is five tiles)
    const int n_warps = (n_mt_max == 5 || n_mt_max == 6) ? n_mt_max : 4;
    const int nslab = n_mt_max <= 2 ? n_mt_max : n_warps;
    if (n_mt_max > n_warps && nsp != 1) return cudaErrorInvalidValue;     // query tiles in rounds: one key tile per block
    const int ring = n_mt_max > 2 ? 2 : attn_ring(hd, nslab, (long long)Hkv * B);
    const int nb = nsp == 1 ? 1 : (nsp == 2 ? 2 : ring);
    const size_t smem = attn_smem(hd, nslab, nb);
    const int early = layer > 0 ? 1 : 0;              // the row metadata was final before the previous kernel started
    dim3 grid(nsplit, Hkv, B);
    const int cnt = n_mt_max >= 3 ? 4 : (n_mt_max == 2 ? 2 : 1);     // 16-key groups per warp task (template parameter)
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 116 * 1024);
        if (e != cudaSuccess) return e;
        return launch_pdl(kernel, grid, dim3(32 * n_warps), smem, st, pdl, m.kv_map, (const __nv_bfloat16*)sc.q_hi,
                          (const __nv_bfloat16*)sc.q_lo, rm, sc.attn_part, layer, m.max_batch, Hq, Hkv, R, nsplit,
                          nslab, nsp, nb, early, status);
    };
    const bool pack = (Hq / Hkv) * R <= 8;            // every sequence of the launch has at most eight query rows per KV head
    if (hd == 128)
        return cnt == 1 ? (pack ? go(attn_mma_kernel<128, 1, true>) : go(attn_mma_kernel<128, 1, false>))
                        : (cnt == 2 ? go(attn_mma_kernel<128, 2, false>) : go(attn_mma_kernel<128, 4, false>));
    if (hd == 64)
        return cnt == 1 ? (pack ? go(attn_mma_kernel<64, 1, true>) : go(attn_mma_kernel<64, 1, false>))
                        : (cnt == 2 ? go(attn_mma_kernel<64, 2, false>) : go(attn_mma_kernel<64, 4, false>));
    return cudaErrorInvalidValue;
}

}  // namespace mtad
