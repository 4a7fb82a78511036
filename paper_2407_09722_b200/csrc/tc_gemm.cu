// Tensor-core weight-streaming GEMM for the skinny projections of the verification step.
//
//   acc[n, r] = sum_k W[n, k] * (x_0[r, k] + x_1[r, k] (+ x_2[r, k]))      n: output feature, r: draft row
//
// The weight matrix is the 128-row MMA operand (A), the draft rows are the MMA N dimension (B), both K-major bf16
// tiles of 64 elements (one 128-byte swizzled row) brought in by TMA; fp32 accumulators live in tensor memory.
// The fp32 activations arrive split into two or three bf16 terms (x_0 = bf16(x), x_1 = bf16(x - x_0), ...): with
// three (up to 32 rows) the tensor cores see the fp32 value itself, with two ~2^-17 relative.  Every term is a row of the MMA's N dimension with an fp32 accumulator column
// of its own; the drain adds a row's columns.  Work is cut into (tile, k-block) units dealt out
// evenly to the CTAs; a tile whose k-range spans several CTAs is completed by whichever of them arrives last, which
// sums the partial tiles in CTA order (deterministic) and runs the fused epilogue - with more than eight rows by all
// the contributors whose run ends in the tile, each taking every n-th pass of eight rows.  With few rows
// two CTAs share an SM (half the shared-memory ring and at most half the tensor memory each): while one drains its
// accumulator, waits for a fix-up or runs an epilogue, the other keeps the weight stream going.
//
// Warp roles: 0 = weight producer (TMA), 1 = operand-row producer (TMA, waits for the rows to exist), 2..5 = MMA
// issuers (one per 128-row half of a stage; a single thread cannot issue the many small MMAs of a skinny problem
// fast enough), 6..9 = epilogue (one TMEM lane quadrant each).
// Every wait on an mbarrier or on another CTA's counter is bounded; on a time-out the kernel raises MTAD_ST_TIMEOUT, waits (bounded) for its
// own copies in flight, frees its tensor memory and returns.
#include <math_constants.h>

#include <algorithm>
#include <type_traits>
#include <stdlib.h>

#include "tc_device.cuh"

namespace mtad {
using namespace tcdev;
namespace {


// ---------------------------------------------------------------------------------------------------------------
// kernel
// ---------------------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(TC_THREADS, 2) tc_gemm_kernel(const __grid_constant__ TcChain ch) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const TcGemmParams& p0 = ch.p[0];
    const int mh = p0.mh;                              // 128-row weight halves per stage (1, 2 or 4), the same for the whole launch
    const int a_bytes = mh * TC_TILE_N * 128;
    const int terms = p0.terms;
    const int acc_cols = terms * p0.rpad;              // one column per operand row: the terms of a draft row are neighbours
    const int n_bbox = p0.n_bbox;                      // TMA boxes (and MMAs per k step and half) that cover the operand rows
    const int bbox_rows = acc_cols / n_bbox;
    const int stage_bytes = a_bytes + acc_cols * 128;
    const int stages = p0.stages, nbuf = p0.nbuf, T = p0.T;
    const Smem s = carve(smem_base, stages, stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&ch.maps[0].a0)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&ch.maps[0].x)) : "memory");
    }
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < nbuf * mh * acc_cols) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < stages; ++i) {
            mbar_init(smem_u32(&s.full[i]), 1);
            mbar_init(smem_u32(&s.empty[i]), mh);        // one commit per MMA-issuing warp
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&s.tfull[i]), mh);
            mbar_init(smem_u32(&s.tempty[i]), 4);
        }
        s.abort_flag[0] = 0;
        s.abort_flag[1] = (int)(p0.wait_limit ? p0.wait_limit : WAIT_LIMIT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s.tmem_ptr)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s.tmem_ptr;
    // let the next kernel in the stream start its own prologue (it waits for this grid before it reads our output)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) trace_stamp(p0.trace, 0);
    volatile int* abort_flag = s.abort_flag;
    // this CTA's share of the launch: units [first, first + count)
    auto share = [&](const TcGemmParams& p, int& first, int& count) {
        first = (int)blockIdx.x * p.units_per_cta;
        count = max(min(first + p.units_per_cta, p.total_units) - first, 0);
    };

    if (warp == 0) {
        // ---------------- weight producer (one thread) -------------------------------------------------------------
        // Weights never depend on an earlier step: their copies go out as soon as a stage is free.  The operand rows of the same stage are brought by the next warp once they exist.
        if (lane == 0) {
            int g = 0;
            bool ok = true;
            {
                const TcGemmParams& p = ch.p[0];
                const TcMaps& mp = ch.maps[0];
                int first, n_units;
                share(p, first, n_units);
                const int nb = a_boxes(p.mode, mh);
                int tile = n_units > 0 ? first / p.k_blocks : 0, kb = n_units > 0 ? first % p.k_blocks : 0;
                for (int i = 0; i < n_units; ++i, ++g) {
                    const int st = g % stages;
                    if (g >= stages) {
                        ok = mbar_wait(smem_u32(&s.empty[st]), (((uint32_t)(g / stages)) & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                    }
                    const uint32_t bar = smem_u32(&s.full[st]);
                    const uint32_t base = smem_u32(s.ring + (size_t)st * stage_bytes);
                    mbar_expect_tx(bar, (uint32_t)stage_bytes);
                    for (int b = 0; b < nb; ++b) {
                        int which, y, row_off;
                        a_box(p.mode, mh, p.seg_k_tile, p.seg_v_tile, tile, b, which, y, row_off);
                        const CUtensorMap* m = which == 0 ? &mp.a0 : (which == 1 ? &mp.a1 : &mp.a2);
                        tma_load_2d(base + row_off * 128, m, bar, kb * TC_TILE_K, y, HINT_STREAM);
                    }
                    if (++kb == p.k_blocks) { kb = 0; ++tile; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- operand-row producer (one thread) --------------------------------------------------------
        // The rows of a k-block exist once the previous kernel is finished.
        if (lane == 0) {
            int g = 0;
            bool ok = true;
            {
                const TcGemmParams& p = ch.p[0];
                int first, n_units;
                share(p, first, n_units);
                asm volatile("griddepcontrol.wait;" ::: "memory");
                trace_stamp(p0.trace, 1);
                int kb = n_units > 0 ? first % p.k_blocks : 0;
                for (int i = 0; i < n_units && ok; ++i, ++g) {
                    const int st = g % stages;
                    if (g >= stages) {
                        ok = mbar_wait(smem_u32(&s.empty[st]), (((uint32_t)(g / stages)) & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                    }
                    const uint32_t bar = smem_u32(&s.full[st]);
                    const uint32_t base = smem_u32(s.ring + (size_t)st * stage_bytes) + a_bytes;
                    for (int b = 0; b < n_bbox && !p0.debug_no_operands; ++b)
                        tma_load_2d(base + b * bbox_rows * 128, &ch.maps[0].x, bar, kb * TC_TILE_K, b * bbox_rows,
                                    HINT_KEEP);
                    if (++kb == p.k_blocks) kb = 0;
                }
            }
            if (*abort_flag) {
                // give the copies in flight a bounded chance to land before the CTA exits
                for (int i = max(0, g - stages); i < g; ++i) {
                    const uint32_t bar = smem_u32(&s.full[i % stages]);
                    const uint32_t phs = (uint32_t)(i / stages) & 1u;
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_test(bar, phs); ++it) __nanosleep(64);
                }
            }
        }
    } else if (warp < 2 + MAX_HALVES) {
        // ---------------- MMA issuers: warp 2 + h owns the 128-row half h of every stage and its accumulator --------
        const int h = warp - 2;
        if (lane == 0 && h < mh) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bbox_rows >> 3) << 17) |
                                   ((uint32_t)(TC_TILE_N >> 4) << 24);
            int g = 0, seg = 0;                        // running unit and segment counters
            bool ok = true;
            {
                const TcGemmParams& p = ch.p[0];
                int first, n_units;
                share(p, first, n_units);
                const int KB = p.k_blocks;
                int i = 0;
                while (i < n_units && ok) {
                    const int kb0 = (first + i) % KB;
                    // (only tiles of the K and V rows are accumulated in capped pieces: Q is never rounded to bf16)
                    const int cap = ((first + i) / KB) * mh < p.seg_k_tile ? (1 << 20) : p.seg_cap;
                    const int len = min(min(KB - kb0, n_units - i), cap);
                    const int buf = seg % nbuf;
                    const uint32_t aph = (uint32_t)(seg / nbuf) & 1u;
                    ok = mbar_wait(smem_u32(&s.tempty[buf]), aph ^ 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * mh * acc_cols);
                    for (int k = 0; k < len && ok; ++k, ++i, ++g) {
                        const int st = g % stages;
                        const uint32_t sph = (uint32_t)(g / stages) & 1u;
                        ok = mbar_wait(smem_u32(&s.full[st]), sph, abort_flag);
                        if (!ok) break;
                        if (g == 0 && h == 0) trace_stamp(p0.trace, 2);
                        tc_fence_after();
                        const uint32_t a_addr = smem_u32(s.ring + (size_t)st * stage_bytes);
                        const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
                        for (int k4 = 0; k4 < TC_TILE_K / 16; ++k4) {
                            const uint32_t acc = (k > 0 || k4 > 0) ? 1u : 0u;
                            const uint64_t ad = smem_desc(a_addr + h * TC_TILE_N * 128 + k4 * 32);
                            for (int b = 0; b < n_bbox; ++b)
                                tc_mma(d_tmem + (uint32_t)(h * acc_cols + b * bbox_rows), ad,
                                       smem_desc(b_addr + b * bbox_rows * 128 + k4 * 32), idesc, acc);
                        }
                        tc_commit(smem_u32(&s.empty[st]));      // frees the smem stage once these MMAs have read it
                    }
                    if (ok) tc_commit(smem_u32(&s.tfull[buf]));  // accumulator of this segment complete
                    if (h == 0 && i == n_units) trace_stamp(p0.trace, 3);
                    ++seg;
                }
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int e = threadIdx.x - 32 * (2 + MAX_HALVES);   // 0..127
        const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
        const int feat = quad * 32 + lane;              // feature (TMEM lane) within a 128-row half
        const size_t half_floats = (size_t)p0.rpad * TC_TILE_N;
        const size_t part_floats = (size_t)mh * half_floats;
        int seg = 0;
        {
            const TcGemmParams& p = ch.p[0];
            int first, n_units;
            share(p, first, n_units);
            const int KB = p.k_blocks;
            // everything read here besides the operand rows (row statistics, the residual stream) is final once the
            // previous kernel has finished
            asm volatile("griddepcontrol.wait;" ::: "memory");
            // deferred RMSNorm scale of every row
            for (int r = e; r < TC_MAX_ROWS; r += EPI_THREADS) {
                float v = 1.f;
                if (r < T && p.sumsq_in_parts > 0) {
                    float acc = 0.f;
                    for (int q = 0; q < p.sumsq_in_parts; ++q) acc += __ldcg(p.sumsq_in + (size_t)q * TC_X_ROWS + r);
                    v = rsqrtf(acc * p.inv_dim + p.eps);
                }
                s.rstd[r] = v;
            }
            epi_bar();
            int i = 0;
            while (i < n_units) {
                const int u = first + i;
                const int tile = u / KB, kb0 = u % KB;
                // A run of this CTA inside one tile of K or V rows is accumulated in pieces of at most seg_cap k-blocks:
                // the tensor cores truncate every partial sum, so a long chain drifts (about -6e-8 relative per
                // k-block); the pieces are added up in fp32 in this CTA's partial tile
                const int len_all = min(KB - kb0, n_units - i);
                const int len = min(len_all, tile * mh < p.seg_k_tile ? (1 << 20) : p.seg_cap);
                const bool first_piece = (i == 0 || kb0 == 0), last_piece = (len == len_all);
                const int buf = seg % nbuf;
                const uint32_t aph = (uint32_t)(seg / nbuf) & 1u;
                bool ok = true;
                if (lane == 0) ok = mbar_wait(smem_u32(&s.tfull[buf]), aph, abort_flag);
                if (lane == 0) s.flags[1 + (warp - 2 - MAX_HALVES)] = ok ? 1 : 0;
                epi_bar();
                if (e == 0 && i + len == n_units) trace_stamp(p0.trace, 4);
                if (!(s.flags[1] && s.flags[2] && s.flags[3] && s.flags[4])) break;
                tc_fence_after();
                // contributors of this tile, in CTA order
                const int c_first = (tile * KB) / p.units_per_cta;
                const int c_last = ((tile + 1) * KB - 1) / p.units_per_cta;
                const int n_contrib = c_last - c_first + 1;
                const int slot_idx = (int)blockIdx.x - c_first;
                float* part = p.ws + idx_tc_ws(tile, p.max_contrib, slot_idx, part_floats);
                // (two copies of the loops, chosen once per piece: a per-element choice between storing and adding
                // would make every store wait for a load)
                auto drain = [&](auto accumulate) {
                    constexpr bool ADD = decltype(accumulate)::value;
                    for (int h = 0; h < mh; ++h) {
                        const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16) +
                                               (uint32_t)(buf * mh * acc_cols + h * acc_cols);
                        float* dst = part + h * half_floats + feat;
                        if (terms == 3) {
                            for (int rb = 0; rb < T; rb += 16) {           // 16 rows = 48 accumulator columns
                                float v[48];
                                tc_ld16(t_acc + 3 * rb, v);
                                tc_ld16(t_acc + 3 * rb + 16, v + 16);
                                tc_ld16(t_acc + 3 * rb + 32, v + 32);
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    if (rb + j < T) {
                                        const float y = v[3 * j] + (v[3 * j + 1] + v[3 * j + 2]);
                                        float* q = dst + (size_t)(rb + j) * TC_TILE_N;
                                        if (ADD) *q += y; else *q = y;
                                    }
                            }
                        } else {
                            for (int c0 = 0; c0 < 2 * T; c0 += 16) {
                                float v[16];
                                tc_ld16(t_acc + c0, v);
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    const int r = (c0 >> 1) + j;
                                    if (r < T) {
                                        const float y = v[2 * j] + v[2 * j + 1];
                                        float* q = dst + (size_t)r * TC_TILE_N;
                                        if (ADD) *q += y; else *q = y;
                                    }
                                }
                            }
                        }
                    }
                };
                if (first_piece) drain(std::false_type{});
                else drain(std::true_type{});
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s.tempty[buf]));   // MMA may reuse this accumulator
                if (!last_piece) {                                      // more of this run in this tile to come
                    i += len;
                    ++seg;
                    continue;
                }
                __threadfence();
                epi_bar();
                // Who finishes the tile.  Few rows (one pass): whoever arrives last.  More rows: the contributors for
                // which this tile is the last of their run - all of them but, possibly, the last in CTA order, which
                // met the tile at the start of its run - arrive within microseconds of one another at the end of the
                // launch; each waits for the full count and takes every n_late-th pass of eight rows, so the passes
                // (each a chain of L2 round trips) run side by side on several SMs.  Counter: arrivals in the low
                // 16 bits, finished late contributors in the high 16.
                const int run_end = min(((int)blockIdx.x + 1) * p.units_per_cta, p.total_units);
                const bool c_last_late = min((c_last + 1) * p.units_per_cta, p.total_units) == (tile + 1) * KB;
                const int n_late = (c_last - c_first) + (c_last_late ? 1 : 0);
                const bool sliced = p.sliced && n_contrib > 1;
                const bool late = u + len == run_end;          // (last piece: u + len is the end of the run in this tile)
                int pass0 = 0, pass_step = 1;
                if (e == 0) {
                    const int old = atomicAdd(&p.counters[tile], 1);
                    int fin = (old + 1 == n_contrib) ? 1 : 0;
                    if (sliced) fin = !late ? 0 : (arrivals_wait(&p.counters[tile], n_contrib, abort_flag) ? 1 : 2);
                    s.flags[0] = fin;
                }
                epi_bar();
                const int fin = s.flags[0];
                epi_bar();                                  // flags[0] is rewritten by the next segment
                if (fin == 2) break;
                if (sliced) { pass0 = slot_idx; pass_step = n_late; }
                if (e == 0 && i + len == n_units) trace_stamp(p0.trace, fin == 1 ? 6 : 5);
                if (fin == 1) {
                    __threadfence();
                    const float* tile_ws = p.ws + idx_tc_ws(tile, p.max_contrib, 0, part_floats);
                    for (int r0 = pass0 * EPI_ROWS; r0 < T; r0 += pass_step * EPI_ROWS) {
                        for (int h = 0; h < mh; ++h) {
                            float acc[EPI_ROWS];
#pragma unroll
                            for (int j = 0; j < EPI_ROWS; ++j) acc[j] = 0.f;
                            // partials are added in CTA order (deterministic); four contributors' loads are issued
                            // together so that the L2 latency is paid once per group, not once per contributor
                            for (int c = 0; c < n_contrib; c += 4) {
                                float v[4][EPI_ROWS];
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const float* src = tile_ws + (size_t)(c + q) * part_floats + h * half_floats + e;
#pragma unroll
                                    for (int j = 0; j < EPI_ROWS; ++j)
                                        v[q][j] = (c + q < n_contrib && r0 + j < T)
                                                      ? __ldcg(src + (size_t)(r0 + j) * TC_TILE_N) : 0.f;
                                }
#pragma unroll
                                for (int q = 0; q < 4; ++q)
#pragma unroll
                                    for (int j = 0; j < EPI_ROWS; ++j) acc[j] += v[q][j];
                            }
#pragma unroll
                            for (int j = 0; j < EPI_ROWS; ++j) s.epi[h][j][e] = (r0 + j < T) ? acc[j] * s.rstd[r0 + j] : 0.f;
                        }
                        epi_bar();
                        const int t_end = min(T, r0 + EPI_ROWS);
                        if (p.mode == TC_SWIGLU) {
                            epi_swiglu<EPI_ROWS>(p, s.epi, tile, r0, t_end, e);
                        } else {
                            for (int h = 0; h < mh; ++h) {
                                const int t128 = tile * mh + h;
                                if (t128 * TC_TILE_N >= p.n_rows_total) break;      // half beyond the last weight row
                                switch (p.mode) {
                                    case TC_PLAIN: epi_plain<EPI_ROWS>(p, s.epi[h], t128, r0, t_end, e); break;
                                    case TC_QKV: epi_qkv<EPI_ROWS>(p, s.epi[h], t128, r0, t_end, e); break;
                                    case TC_RESID: epi_resid<EPI_ROWS>(p, s.red, s.epi[h], t128, r0, t_end, e); break;
                                    default: epi_lmhead<EPI_ROWS>(p, s.red4, s.epi[h], t128, r0, t_end, e); break;
                                }
                            }
                        }
                        epi_bar();
                    }
                    bool closer = true;                         // the one that leaves the tile's counter at zero
                    if (sliced) {
                        __threadfence();
                        epi_bar();
                        if (e == 0) {
                            const int old = atomicAdd(&p.counters[tile], 0x10000);
                            s.flags[0] = ((old >> 16) + 1 == n_late) ? 1 : 0;
                        }
                        epi_bar();
                        closer = s.flags[0] != 0;
                        epi_bar();
                    }
                    if (e == 0 && closer) p.counters[tile] = 0;          // ready for the next launch
                }
                i += len;
                ++seg;
            }
        }
    }
    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) trace_stamp(p0.trace, 7);
    if (warp == 2) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag && p0.status) {
        // every sequence of the call carries the bit: the rows of all of them went through this launch
        const int nseq = p0.R > 0 ? (T + p0.R - 1) / p0.R : 1;
        for (int b = 0; b < nseq; ++b) atomicOr(p0.status + b, MTAD_ST_TIMEOUT);
    }
}

__global__ void split_rows_kernel(const float* __restrict__ x, int ldx_in, __nv_bfloat16* __restrict__ out, int terms,
                                  int K) {
    const int t = blockIdx.x;
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        store_terms(x[(size_t)t * ldx_in + k], out + (size_t)t * terms * K + k, K, terms);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    }
    return fn;
}

}  // namespace


int tc_make_map(CUtensorMap* out, const void* base, long long rows, long long cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return -1;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_TILE_K, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

int tc_make_kv_map(CUtensorMap* out, const void* cache, int hd, long long cap, long long planes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || (hd != 64 && hd != 128) || cap < 1 || planes < 1) return -1;
    const cuuint64_t dims[3] = {(cuuint64_t)hd, (cuuint64_t)cap, (cuuint64_t)planes};
    const cuuint64_t strides[2] = {(cuuint64_t)hd * 2, (cuuint64_t)cap * hd * 2};
    const cuuint32_t box[3] = {64, 64, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(cache), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

int tc_boxes(int acc_cols) {
    for (int n = 1; n <= 3; ++n)
        if (acc_cols % n == 0 && acc_cols / n <= 256 && (acc_cols / n) % 16 == 0) return n;
    return 0;
}

int tc_qkv_terms(int T) {
    const int rpad = (T + 15) / 16 * 16;
    return 3 * rpad <= 512 ? 3 : tc_terms(T);
}

void tc_decompose(TcGemmParams& p, int n_tiles, int K, int T, int sms, int per_sm, int terms) {
    p.per_sm = per_sm > 0 ? per_sm : tc_ctas_per_sm(T);
    const int ctas = sms * p.per_sm;
    p.n_tiles = n_tiles;
    p.k_blocks = (K + TC_TILE_K - 1) / TC_TILE_K;
    p.total_units = n_tiles * p.k_blocks;
    p.units_per_cta = (p.total_units + ctas - 1) / ctas;
    // small matrices (the auxiliary model's): fewer CTAs with longer runs, so that a tile is not cut into one
    // contributor per k-block whose partial tiles the last arriver has to add up
    if (p.units_per_cta < 2) p.units_per_cta = 2;
    p.max_contrib = (p.k_blocks + p.units_per_cta - 1) / p.units_per_cta + 1;
    p.T = T;
    p.rpad = (T + 15) / 16 * 16;
    p.terms = terms > 0 ? terms : tc_terms(T);
    p.out_terms = p.terms;
    p.n_bbox = tc_boxes(p.terms * p.rpad);
    // more than one pass of eight rows: the passes of a tile are shared out among its contributors, which wait for
    // one another - every CTA of the launch must be resident, i.e. at most one per SM slot
    p.sliced = (T > EPI_ROWS && sms <= 148) ? 1 : 0;
    p.seg_cap = 1 << 20;
}

int tc_terms(int T) {
    // Three terms up to 32 rows, where the third costs nothing measurable; two beyond.  With more rows the operand
    // rows (terms * rows * 128 B per k-block, re-read from L2 by every CTA) outweigh the 16 KB of weights they meet,
    // two terms leave room in tensor memory for two weight halves per stage up to 64 rows, and at the level of the
    // whole model the third term changes nothing (the error there is set by bf16 K/V rounding).
    const int rpad = (T + 15) / 16 * 16;
    return rpad <= 32 ? 3 : 2;
}

int tc_ctas_per_sm(int T) {
    // two CTAs need: 16 KB of weights + terms * rpad operand rows per stage, at least two stages in 112 KB less the
    // epilogue scratch, and one accumulator buffer of terms * rpad columns within 256 columns
    const int rpad = (T + 15) / 16 * 16, cols = tc_terms(T) * rpad;
    if (cols > 240) return 1;
    return rpad <= 32 ? 2 : 1;
}

int tc_halves(int T) {
    if (tc_ctas_per_sm(T) == 2) return 1;
    // TMEM holds buffers x halves x terms * rpad columns <= 512.  Two halves (two MMA-issuing warps, 32 KB of weights
    // per stage against the same operand rows) are worth more than a second accumulator buffer: with 129..256
    // columns a stage has two halves and the launch a single buffer (7B tree 8.7 -> 8.0 ms).  Four halves fit the
    // smallest row counts but fill and drain slower than two.
    const int cap = 2;
    const int cols = tc_terms(T) * ((T + 15) / 16 * 16);
    const int fit = cols <= 64 ? 4 : (cols <= 256 ? 2 : 1);
    return fit < cap ? fit : cap;
}

size_t tc_workspace_floats(int n_tiles_max, int max_contrib_max, int rpad_max) {
    return (size_t)n_tiles_max * max_contrib_max * rpad_max * TC_TILE_N;
}

cudaError_t launch_tc_chain(const TcChain& chain_in, bool pdl, cudaStream_t st) {
    TcChain ch = chain_in;
    const TcGemmParams& f = ch.p[0];
    if (f.mh != 1 && f.mh != 2 && f.mh != 4) return cudaErrorInvalidValue;
    if (f.terms != 2 && f.terms != 3) return cudaErrorInvalidValue;
    if (f.per_sm != 1 && f.per_sm != 2) return cudaErrorInvalidValue;
    const int acc_cols = f.terms * f.rpad;
    const int tmem_budget = 512 / f.per_sm;           // the CTAs of an SM allocate tensor memory side by side
    if (f.mh * acc_cols > tmem_budget || f.n_bbox < 1 || f.n_bbox != tc_boxes(acc_cols)) return cudaErrorInvalidValue;
    const int nbuf = (2 * f.mh * acc_cols <= tmem_budget) ? 2 : 1;
    const int stage_bytes = f.mh * TC_TILE_N * 128 + acc_cols * 128;
    const size_t budget = f.per_sm == 2 ? (size_t)112 * 1024 : (size_t)226 * 1024;
    int stages = (int)((budget - SMEM_TAIL - 1024) / stage_bytes);
    stages = stages > MAX_STAGES ? MAX_STAGES : stages;
    if (stages < 2) return cudaErrorInvalidValue;
    int grid = 1;
    {
        TcGemmParams& p = ch.p[0];
        if (p.mh != f.mh || p.rpad != f.rpad || p.T != f.T || p.terms != f.terms || p.per_sm != f.per_sm ||
            p.n_bbox != f.n_bbox)
            return cudaErrorInvalidValue;                  // one ring, one TMEM layout
        p.nbuf = nbuf;
        p.stages = stages;
        grid = std::max(grid, (p.total_units + p.units_per_cta - 1) / p.units_per_cta);
    }
    const size_t smem = (size_t)stages * stage_bytes + SMEM_TAIL + 1024;
    static bool attr_set[64] = {};                     // per device
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_gemm_kernel, ch);
}

cudaError_t launch_tc_gemm(const TcMaps& maps, const TcGemmParams& p, int ctas, bool pdl, cudaStream_t st) {
    (void)ctas;
    TcChain ch{};
    ch.maps[0] = maps;
    ch.p[0] = p;
    return launch_tc_chain(ch, pdl, st);
}

cudaError_t launch_split_rows(const float* x, int ldx_in, __nv_bfloat16* out, int terms, int T, int K, cudaStream_t st) {
    split_rows_kernel<<<T, 256, 0, st>>>(x, ldx_in, out, terms, K);
    return cudaGetLastError();
}

}  // namespace mtad
