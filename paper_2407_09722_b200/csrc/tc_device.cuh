// Device-side building blocks shared by the tensor-core GEMM kernels: bounded mbarrier waits, TMA loads, tcgen05
// wrappers, the shared-memory descriptor of a K-major 128-byte-swizzled tile, and the fused epilogues.
#pragma once

#include <math_constants.h>

#include "tc_gemm.cuh"

namespace mtad {
namespace tcdev {

constexpr uint32_t WAIT_LIMIT = 1u << 22;
constexpr int MAX_STAGES = 12;
constexpr int EPI_THREADS = 128;
constexpr int EPI_ROWS = 8;                       // draft rows finished per epilogue pass
constexpr int MAX_HALVES = 4;                     // 128-row weight halves per stage, one MMA-issuing warp each
constexpr int TC_THREADS = 32 * (2 + MAX_HALVES + 4);
constexpr uint64_t HINT_STREAM = 0x12F0000000000000ull;   // evict-first: weights are read once
constexpr uint64_t HINT_KEEP = 0x14F0000000000000ull;     // evict-last: activation operands are re-read by every CTA

// MTAD_TRACE builds stamp the global timer at fixed points of every CTA's life (slot k of the launch's trace rows)
#ifdef MTAD_TRACE
__device__ __forceinline__ void trace_stamp(unsigned long long* trace, int k) {
    if (trace) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        trace[(size_t)blockIdx.x * 8 + k] = t;
    }
}
#else
__device__ __forceinline__ void trace_stamp(unsigned long long*, int) {}
#endif

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Bounded wait.  Returns false when the limit ran out here or another role already gave up.  abort_flag[0] is the
// CTA's give-up flag, abort_flag[1] the iteration limit of every wait of this launch.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const uint32_t limit = (uint32_t)abort_flag[1];
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_test(bar, parity)) return true;
        if (it > 64) __nanosleep(32);
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

// Bounded wait until the arrival count of a tile (low 16 bits of its counter) reaches `want` (acquire at gpu scope).
__device__ __forceinline__ bool arrivals_wait(const int* counter, int want, volatile int* abort_flag) {
    const uint32_t limit = (uint32_t)abort_flag[1];
    for (uint32_t it = 0; it < limit; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if ((v & 0xFFFF) >= want) return true;
        __nanosleep(64);
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

// Bounded wait until a counter written by other CTAs of this launch reaches `want` (acquire at gpu scope).
__device__ __forceinline__ bool flag_wait(const int* flag, int want, volatile int* abort_flag) {
    const uint32_t limit = (uint32_t)abort_flag[1];
    for (uint32_t it = 0; it < limit; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v >= want) return true;
        __nanosleep(64);
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                            uint64_t hint) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(hint)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 operands, fp32 accumulate, M = 128.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; start address advances 32 bytes per 16-element k step.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15},"
        " [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 consecutive columns of this warp's TMEM lanes
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ---- thread-block clusters ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive_release() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// fp32 store into the shared memory of CTA `rank` of this cluster, at the address that `local_addr` has in this CTA
__device__ __forceinline__ void st_cluster_f32(uint32_t local_addr, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// barrier of one group of 128 epilogue threads (id 1, or 1 and 2 where a kernel has two groups)
__device__ __forceinline__ void epi_bar(int id = 1) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// two-term split of the query rows for the tensor-core attention
__device__ __forceinline__ void split_store(float y, __nv_bfloat16* hi, __nv_bfloat16* lo) {
    const __nv_bfloat16 h = __float2bfloat16_rn(y);
    *hi = h;
    *lo = __float2bfloat16_rn(y - __bfloat162float(h));
}

// Weight boxes of one stage: how many, and for box b of a tile which map (0..2), which row coordinate and which
// row offset inside the stage.  SwiGLU tiles take their first half from the gate matrix and their second half
// from the up matrix; QKV tiles lie in the q, k or v matrix; a 512-row tile is fetched as two 256-row boxes.
__device__ __forceinline__ int a_boxes(int mode, int mh) { return (mode == TC_SWIGLU || mh == 4) ? 2 : 1; }
__device__ __forceinline__ void a_box(int mode, int mh, int seg_k, int seg_v, int tile, int b, int& which, int& y,
                                      int& row_off) {
    if (mode == TC_SWIGLU) {
        const int rows = 64 * mh;
        which = b;
        y = tile * rows;
        row_off = b * rows;
    } else if (mode == TC_QKV) {
        const int t128 = tile * mh;
        which = t128 < seg_k ? 0 : (t128 < seg_v ? 1 : 2);
        y = (t128 < seg_k ? t128 : (t128 < seg_v ? t128 - seg_k : t128 - seg_v)) * TC_TILE_N + b * 256;
        row_off = b * 256;
    } else {
        which = 0;
        y = tile * mh * TC_TILE_N + b * 256;
        row_off = b * 256;
    }
}

struct Smem {
    uint8_t* ring;
    float (*epi)[EPI_ROWS][TC_TILE_N + 1];   // [half][row][feature]
    float* rstd;
    float* red;            // [4][EPI_ROWS] floats, also reused as [4][EPI_ROWS] float4 via red4
    float4* red4;
    uint64_t* full;
    uint64_t* empty;
    uint64_t* tfull;
    uint64_t* tempty;
    uint32_t* tmem_ptr;
    int* abort_flag;
    int* flags;            // [0] last-arriver flag, [1..4] epilogue warp wait results
};

__device__ __forceinline__ Smem carve(uint8_t* base, int stages, int stage_bytes) {
    Smem s;
    s.ring = base;
    uint8_t* p = base + (size_t)stages * stage_bytes;
    s.epi = reinterpret_cast<float(*)[EPI_ROWS][TC_TILE_N + 1]>(p);
    p += sizeof(float) * MAX_HALVES * EPI_ROWS * (TC_TILE_N + 1);
    s.rstd = reinterpret_cast<float*>(p);
    p += sizeof(float) * TC_MAX_ROWS;
    p = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 15) & ~uintptr_t(15));
    s.red4 = reinterpret_cast<float4*>(p);
    s.red = reinterpret_cast<float*>(p);
    p += sizeof(float4) * 4 * EPI_ROWS * 2;
    s.full = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.empty = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.tfull = reinterpret_cast<uint64_t*>(p);
    p += 16;
    s.tempty = reinterpret_cast<uint64_t*>(p);
    p += 16;
    s.tmem_ptr = reinterpret_cast<uint32_t*>(p);
    p += 8;
    s.abort_flag = reinterpret_cast<int*>(p);
    p += 8;
    s.flags = reinterpret_cast<int*>(p);
    return s;
}

constexpr size_t SMEM_TAIL = sizeof(float) * MAX_HALVES * EPI_ROWS * (TC_TILE_N + 1) + sizeof(float) * TC_MAX_ROWS + 16 +
                             sizeof(float4) * 4 * EPI_ROWS * 2 + 8 * MAX_STAGES * 2 + 16 + 16 + 8 + 8 + 32;

// ---------------------------------------------------------------------------------------------------------------
// epilogues: called by the 128 epilogue threads for a block of ROWS finished rows (a template parameter: 8, or 16 where
// shared memory allows and there are many rows) of one 128-feature tile held in epi[j][i] (j: row r0 + j, i: feature
// tile * 128 + i).  e = epilogue thread index 0..127.
typedef float (*EpiTile)[TC_TILE_N + 1];
// ---------------------------------------------------------------------------------------------------------------

template <int ROWS>
__device__ __forceinline__ void epi_plain(const TcGemmParams& p, EpiTile epi, int tile, int r0, int t_end, int e) {
    const int n = tile * TC_TILE_N + e;
    if (n >= p.N) return;
    for (int j = 0; j < ROWS && r0 + j < t_end; ++j) p.out[(size_t)(r0 + j) * p.ldo + n] = epi[j][e];
}

// The epilogues below first issue the global loads of all ROWS rows, then compute: a finished tile is the end of
// a dependency chain (the next kernel waits for it), so one L2 round trip per pass instead of one per row matters.
template <int ROWS>
__device__ __forceinline__ void epi_qkv(const TcGemmParams& p, EpiTile epi, int tile, int r0, int t_end, int e) {
    const int hd = p.hd, half = hd >> 1;
    int seg, tin;
    if (tile < p.seg_k_tile) { seg = 0; tin = tile; }
    else if (tile < p.seg_v_tile) { seg = 1; tin = tile - p.seg_k_tile; }
    else { seg = 2; tin = tile - p.seg_v_tile; }
    const int f = tin * TC_TILE_N + e;
    const int head = f / hd, jin = f % hd;
    const int heads = seg == 0 ? p.Hq : p.Hkv;
    if (head >= heads) return;
    const int ldq = (p.Hq + 2 * p.Hkv) * hd;
    const float scale = rsqrtf((float)hd);
    const bool rot = seg != 2 && jin < half;          // this thread rotates the pair (jin, jin + half)
    if (seg != 2 && !rot) return;
    int sl[ROWS], sq[ROWS];
    float2 cs[ROWS];
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
        const int t = r0 + j;
        const bool valid = t < t_end;
        sl[j] = (valid && seg != 0) ? p.slot[t] : (valid ? 0 : -1);
        sq[j] = (valid && seg != 0) ? p.seq[t] : 0;
        cs[j] = (valid && rot) ? *reinterpret_cast<const float2*>(p.rope + ((size_t)t * half + jin) * 2)
                               : make_float2(1.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
        const int t = r0 + j;
        if (sl[j] < 0) continue;                      // row beyond T, or an inactive row (no cache slot)
        if (seg != 0 && (sl[j] >= p.cap || (unsigned)sq[j] >= (unsigned)p.max_batch)) continue;   // never past the cache
        if (seg == 2) {
            const size_t base = idx_cache(p.layer, p.max_batch, sq[j], 1, p.Hkv, head, p.cap, sl[j], hd);
            p.cache[base + jin] = __float2bfloat16_rn(epi[j][e]);
            continue;
        }
        const float c = cs[j].x, sn = cs[j].y;
        const float a = epi[j][e], b = epi[j][e + half];
        const float ra = a * c - b * sn, rb = b * c + a * sn;
        if (seg == 0) {
            float* q = p.q_out + (size_t)t * ldq + head * hd;
            q[jin] = ra * scale;
            q[jin + half] = rb * scale;
            if (p.q_hi) {
                // tensor-core attention operands: q * log2(e) / sqrt(hd) as bf16 hi + lo (softmax runs on exp2)
                const size_t o = (size_t)t * p.Hq * hd + head * hd;
                split_store(ra * scale * 1.4426950408889634f, p.q_hi + o + jin, p.q_lo + o + jin);
                split_store(rb * scale * 1.4426950408889634f, p.q_hi + o + jin + half, p.q_lo + o + jin + half);
            }
        } else {
            const size_t base = idx_cache(p.layer, p.max_batch, sq[j], 0, p.Hkv, head, p.cap, sl[j], hd);
            p.cache[base + jin] = __float2bfloat16_rn(ra);
            p.cache[base + jin + half] = __float2bfloat16_rn(rb);
        }
    }
}

template <int ROWS>
__device__ __forceinline__ void epi_resid(const TcGemmParams& p, float* red, EpiTile epi, int tile, int r0,
                                          int t_end, int e, int bar = 1) {
    const int n = tile * TC_TILE_N + e;
    const bool ok = n < p.N;
    const float g = ok ? __bfloat162float(p.gain[n]) : 0.f;
    const int warp = e >> 5, lane = e & 31;
    float y[ROWS];
#pragma unroll
    for (int j = 0; j < ROWS; ++j)
        y[j] = (ok && r0 + j < t_end) ? __ldcg(p.hidden + (size_t)(r0 + j) * p.N + n) : 0.f;
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
        const int t = r0 + j;
        if (ok && t < t_end) {
            y[j] += epi[j][e];
            p.hidden[(size_t)t * p.N + n] = y[j];
            store_terms(y[j] * g, p.x_out + (size_t)t * p.out_terms * p.xk + n, p.xk, p.out_terms);
            if (p.x_out2) store_terms(y[j] * g, p.x_out2 + (size_t)t * p.out_terms2 * p.xk + n, p.xk, p.out_terms2);
        }
        y[j] *= y[j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int j = 0; j < ROWS; ++j) y[j] += __shfl_xor_sync(0xffffffffu, y[j], o);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < ROWS; ++j) red[warp * ROWS + j] = y[j];
    }
    epi_bar(bar);
    if (e < ROWS && r0 + e < t_end)
        p.sumsq_out[(size_t)tile * TC_X_ROWS + r0 + e] =
            (red[e] + red[ROWS + e]) + (red[2 * ROWS + e] + red[3 * ROWS + e]);
    epi_bar(bar);       // the scratch is reused by the next tile half
}

template <int ROWS>
__device__ __forceinline__ void epi_swiglu(const TcGemmParams& p, float (*epi)[ROWS][TC_TILE_N + 1], int tile, int r0, int t_end,
                                           int e) {
    // the first half of a tile's weight rows are gate rows, the second half the matching up rows
    if (p.mh == 1) {
        if (e >= 64) return;
        const int f = tile * 64 + e;
        if (f >= p.N) return;
        for (int j = 0; j < ROWS && r0 + j < t_end; ++j) {
            const float g = epi[0][j][e], u = epi[0][j][e + 64];
            store_terms(g / (1.f + expf(-g)) * u, p.x_out + (size_t)(r0 + j) * p.out_terms * p.xk + f, p.xk, p.out_terms);
        }
        return;
    }
    const int hh = p.mh / 2;
    for (int h = 0; h < hh; ++h) {
        const int f = tile * 64 * p.mh + h * TC_TILE_N + e;
        if (f >= p.N) break;
        for (int j = 0; j < ROWS && r0 + j < t_end; ++j) {
            const float g = epi[h][j][e], u = epi[h + hh][j][e];
            store_terms(g / (1.f + expf(-g)) * u, p.x_out + (size_t)(r0 + j) * p.out_terms * p.xk + f, p.xk, p.out_terms);
        }
    }
}

template <int ROWS>
__device__ __forceinline__ void epi_lmhead(const TcGemmParams& p, float4* red4, EpiTile epi, int tile, int r0,
                                           int t_end, int e, int bar = 1) {
    const int v = tile * TC_TILE_N + e;
    const bool ok = v < p.N;
    const int warp = e >> 5, lane = e & 31;
    // Gumbel noise of this token: one draw per sequence, shared by all its rows
    float u[ROWS];
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
        const int t = r0 + j;
        const bool fresh = j == 0 || t / p.R != (t - 1) / p.R;
        u[j] = (ok && t < t_end && fresh) ? p.uniforms[(size_t)(t / p.R) * p.N + v] : -1.f;
    }
    float m[ROWS], sum[ROWS], bv[ROWS];
    int bi[ROWS];
    float gum = 0.f;
#pragma unroll
    for (int j = 0; j < ROWS; ++j) {
        if (u[j] >= 0.f) gum = -logf(-logf(u[j]));
        const bool valid = ok && r0 + j < t_end;
        m[j] = valid ? epi[j][e] : -CUDART_INF_F;
        bv[j] = valid ? m[j] + gum : -CUDART_INF_F;
        bi[j] = valid ? v : 0x7fffffff;
        sum[j] = m[j];                                // this thread's logit, kept for the sum below
    }
    // per row: maximum over the warp, then one exponential per thread and a sum; arg-max of the perturbed logits
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int j = 0; j < ROWS; ++j) {
            m[j] = fmaxf(m[j], __shfl_xor_sync(0xffffffffu, m[j], o));
            const float v2 = __shfl_xor_sync(0xffffffffu, bv[j], o);
            const int i2 = __shfl_xor_sync(0xffffffffu, bi[j], o);
            if (v2 > bv[j] || (v2 == bv[j] && i2 < bi[j])) { bv[j] = v2; bi[j] = i2; }
        }
#pragma unroll
    for (int j = 0; j < ROWS; ++j) sum[j] = (sum[j] == -CUDART_INF_F) ? 0.f : expf(sum[j] - m[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int j = 0; j < ROWS; ++j) sum[j] += __shfl_xor_sync(0xffffffffu, sum[j], o);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < ROWS; ++j) red4[warp * ROWS + j] = make_float4(m[j], sum[j], bv[j], __int_as_float(bi[j]));
    }
    epi_bar(bar);
    if (e < ROWS && r0 + e < t_end) {
        float4 a = red4[e];
        for (int w = 1; w < 4; ++w) {
            const float4 b = red4[w * ROWS + e];
            const float mm = fmaxf(a.x, b.x);
            const float sa = a.x == -CUDART_INF_F ? 0.f : a.y * expf(a.x - mm);
            const float sb = b.x == -CUDART_INF_F ? 0.f : b.y * expf(b.x - mm);
            a.x = mm;
            a.y = sa + sb;
            if (b.z > a.z || (b.z == a.z && __float_as_int(b.w) < __float_as_int(a.w))) { a.z = b.z; a.w = b.w; }
        }
        p.lm_part[idx_lm_part(r0 + e, p.n_tiles128, tile)] = a;
    }
    // gather: logit of each node's token under its parent row, when both fall into this block of rows and this tile
    const int n0 = tile * TC_TILE_N;
    for (int t = e; t < p.T; t += EPI_THREADS) {
        const int pr = p.prow[t];
        if (pr < r0 || pr >= t_end) continue;
        const int tk = p.tok[t] - n0;
        if (tk >= 0 && tk < TC_TILE_N) p.node_z[t] = epi[pr - r0][tk];
    }
    epi_bar(bar);       // the scratch is reused by the next tile half
}

}  // namespace tcdev
}  // namespace mtad
