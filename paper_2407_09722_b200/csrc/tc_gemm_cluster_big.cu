// Cluster split-K GEMM for calls of more than 32 draft rows (a draft tree, a batch of chains): the many-row sibling of
// tc_gemm_cluster.cu.  Same idea - a cluster of `csize` CTAs owns one tile, CTA `rank` streams its share of the
// k-blocks into tensor memory, the partial rows meet in the shared memory of the rows' owners - with what many rows
// change:
//   - one CTA per SM (the operand rows of a stage take as much shared memory as the weights), and a tile of two
//     128-feature halves that meet the same operand rows, one MMA-issuing warp and one accumulator each;
//   - the partial tile (65 rows x 256 features are 66 KB) does not travel as single stores: it is drained into a
//     staging area, rows in order, and the rows of a pass - one contiguous piece - go to the pass's owner as one bulk
//     copy over distributed shared memory, counted on an mbarrier of the owner;
//   - receive slots and staging area lie over the copy ring, which is idle by then: the first cluster barrier is
//     passed only when every CTA of the cluster has all its MMAs behind it;
//   - two groups of four epilogue warps.  An epilogue is a chain of dependent loads and stores with a single warp on
//     each scheduler of the SM, so its pace is set by latency, not by work; the second group doubles what is in
//     flight.  The groups share out the (pass, half) pairs of the CTA.
//
// Warps: 0 weight producer (TMA), 1 operand-row producer (TMA), 2..3 MMA issuers (warp 2 owns the tensor-memory
// allocation), 4..7 and 8..11 epilogue groups (a warp reads the TMEM lane quadrant warp % 4).
// Every mbarrier wait is bounded; a time-out raises MTAD_ST_TIMEOUT for every sequence of the call, and the CTA still
// takes part in both cluster barriers so that its neighbours never wait for it.
#include <algorithm>

#include "tc_device.cuh"

namespace mtad {
using namespace tcdev;
namespace {

constexpr int BG_MH = 2;                          // halves of a tile (at most)
constexpr int BG_GROUPS = 2;                      // epilogue groups of 128 threads (three: 7B tree 6.05 -> 6.59 ms, four: 6.43)
constexpr int BG_EPI_WARP0 = 2 + BG_MH;
constexpr int BG_THREADS = 32 * (BG_EPI_WARP0 + 4 * BG_GROUPS);
constexpr int BG_ROWS = EPI_ROWS;                 // rows of an epilogue pass
constexpr size_t BG_BUDGET = (size_t)225 * 1024;  // dynamic shared memory of the CTA

__device__ __forceinline__ void both_bar() {         // all epilogue groups
    asm volatile("bar.sync 15, %0;" ::"n"(128 * BG_GROUPS) : "memory");
}

// Bulk copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) from this CTA's shared memory into the
// shared memory of CTA `rank` of the cluster, at the address that `local_dst` has in this CTA; the bytes are counted
// on the mbarrier that `local_bar` names in the destination CTA.
__device__ __forceinline__ void bulk_copy_to_rank(uint32_t local_dst, uint32_t src, uint32_t bytes, uint32_t local_bar,
                                                  uint32_t rank) {
    uint32_t dst, bar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(local_dst), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(local_bar), "r"(rank));
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "r"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

struct BgSmem {
    uint8_t* ring;                 // the copy ring; later [receive slots][staging area]
    float* epi;                    // [group][half][BG_ROWS][129]: the rows of the pass a group is finishing
    float* rstd;                   // [TC_MAX_ROWS]
    float4* red4;                  // [group][4][BG_ROWS] float4 epilogue scratch (also used as floats)
    uint64_t* full;
    uint64_t* empty;
    uint64_t* tfull;
    uint64_t* rfull;               // counts the bytes of the partial rows that the cluster copies into the receive slots
    uint32_t* tmem_ptr;
    int* abort_flag;
    int* flags;
};

constexpr size_t BG_EPI_BYTES = (sizeof(float) * BG_MH * BG_ROWS * (TC_TILE_N + 1) + 15) / 16 * 16;      // one group
constexpr size_t BG_TAIL = BG_GROUPS * BG_EPI_BYTES + sizeof(float) * TC_MAX_ROWS +
                           sizeof(float4) * BG_GROUPS * 4 * BG_ROWS + 8 * (2 * MAX_STAGES + 2) + 8 + 8 + 32;

__device__ __forceinline__ BgSmem bg_carve(uint8_t* base, int ring_bytes) {
    BgSmem s;
    s.ring = base;
    uint8_t* p = base + ring_bytes;
    s.epi = reinterpret_cast<float*>(p);
    p += BG_GROUPS * BG_EPI_BYTES;
    s.rstd = reinterpret_cast<float*>(p);
    p += sizeof(float) * TC_MAX_ROWS;
    s.red4 = reinterpret_cast<float4*>(p);
    p += sizeof(float4) * BG_GROUPS * 4 * BG_ROWS;
    s.full = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.empty = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.tfull = reinterpret_cast<uint64_t*>(p);
    p += 8;
    s.rfull = reinterpret_cast<uint64_t*>(p);
    p += 8;
    s.tmem_ptr = reinterpret_cast<uint32_t*>(p);
    p += 8;
    s.abort_flag = reinterpret_cast<int*>(p);
    p += 8;
    s.flags = reinterpret_cast<int*>(p);
    return s;
}

// receive slots of one CTA: passes it owns x source ranks x rows per pass x halves x 128 features
__host__ __device__ inline int bg_recv_floats(int T, int rpr, int csize, int mh) {
    const int n_pass = (T + rpr - 1) / rpr;
    const int own = (n_pass + csize - 1) / csize;
    return own * csize * rpr * mh * TC_TILE_N;
}

__global__ void __launch_bounds__(BG_THREADS, 1) tc_gemm_cluster_big_kernel(const __grid_constant__ TcMaps mp,
                                                                           const __grid_constant__ TcGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // every CTA of the cluster must carve identically: the copies into another CTA use this CTA's own offsets
    uint8_t* smem_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int terms = p.terms, T = p.T, mh = p.mh;
    const int acc_cols = terms * p.rpad;               // one accumulator column per operand row
    const int a_bytes = mh * TC_TILE_N * 128;
    const int stage_bytes = a_bytes + acc_cols * 128;
    const int stages = p.stages;
    const int csize = p.csize, rpr = p.rpr;
    const BgSmem s = bg_carve(smem_base, p.ring_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const int tile = p.tile_base + (int)blockIdx.x / csize;
    const int kb0 = (int)(((long long)rank * p.k_blocks) / csize);
    const int kb1 = (int)(((long long)(rank + 1) * p.k_blocks) / csize);
    const int n_kb = kb1 - kb0;
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mp.a0)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mp.x)) : "memory");
        for (int i = 0; i < stages; ++i) {
            mbar_init(smem_u32(&s.full[i]), 1);
            mbar_init(smem_u32(&s.empty[i]), mh);      // one commit per MMA-issuing warp
        }
        mbar_init(smem_u32(s.tfull), mh);
        mbar_init(smem_u32(s.rfull), 1);
        s.abort_flag[0] = 0;
        s.abort_flag[1] = (int)(p.wait_limit ? p.wait_limit : WAIT_LIMIT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < mh * acc_cols) tmem_cols <<= 1;
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
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) trace_stamp(p.trace, 0);
    volatile int* abort_flag = s.abort_flag;

    if (warp == 0) {
        // ---------------- weight producer: copies go out as soon as a stage is free, before the previous kernel ends
        if (lane == 0) {
            const int nb = a_boxes(p.mode, mh);
            for (int i = 0; i < n_kb; ++i) {
                const int st = i % stages;
                if (i >= stages && !mbar_wait(smem_u32(&s.empty[st]), (((uint32_t)(i / stages)) & 1u) ^ 1u, abort_flag))
                    break;
                const uint32_t bar = smem_u32(&s.full[st]);
                const uint32_t base = smem_u32(s.ring + (size_t)st * stage_bytes);
                mbar_expect_tx(bar, (uint32_t)stage_bytes);
                for (int b = 0; b < nb; ++b) {
                    int which, y, row_off;
                    a_box(p.mode, mh, p.seg_k_tile, p.seg_v_tile, tile, b, which, y, row_off);
                    const CUtensorMap* m = which == 0 ? &mp.a0 : (which == 1 ? &mp.a1 : &mp.a2);
                    tma_load_2d(base + row_off * 128, m, bar, (kb0 + i) * TC_TILE_K, y, HINT_STREAM);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- operand-row producer: the rows exist once the previous kernel has finished
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            trace_stamp(p.trace, 1);
            int i = 0;
            for (; i < n_kb; ++i) {
                const int st = i % stages;
                if (i >= stages && !mbar_wait(smem_u32(&s.empty[st]), (((uint32_t)(i / stages)) & 1u) ^ 1u, abort_flag))
                    break;
                const uint32_t bar = smem_u32(&s.full[st]);
                const uint32_t base = smem_u32(s.ring + (size_t)st * stage_bytes) + a_bytes;
                if (!p.debug_no_operands) tma_load_2d(base, &mp.x, bar, (kb0 + i) * TC_TILE_K, 0, HINT_KEEP);
            }
            if (*abort_flag) {
                // give the copies in flight a bounded chance to land before the CTA exits
                for (int j = max(0, i - stages); j < i; ++j) {
                    const uint32_t bar = smem_u32(&s.full[j % stages]);
                    const uint32_t phs = (uint32_t)(j / stages) & 1u;
                    for (uint32_t it = 0; it < (1u << 16) && !mbar_test(bar, phs); ++it) __nanosleep(64);
                }
            }
        }
    } else if (warp < BG_EPI_WARP0) {
        // ---------------- MMA issuers: warp 2 + h owns the 128-feature half h of every stage and its accumulator
        const int h = warp - 2;
        if (lane == 0 && h < mh) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(acc_cols >> 3) << 17) |
                                   ((uint32_t)(TC_TILE_N >> 4) << 24);
            const uint32_t d_tmem = tmem_base + (uint32_t)(h * acc_cols);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int st = i % stages;
                ok = mbar_wait(smem_u32(&s.full[st]), (uint32_t)(i / stages) & 1u, abort_flag);
                if (!ok) break;
                if (i == 0 && h == 0) trace_stamp(p.trace, 2);
                tc_fence_after();
                const uint32_t a_addr = smem_u32(s.ring + (size_t)st * stage_bytes) + h * TC_TILE_N * 128;
                const uint32_t b_addr = smem_u32(s.ring + (size_t)st * stage_bytes) + a_bytes;
#pragma unroll
                for (int k4 = 0; k4 < TC_TILE_K / 16; ++k4)
                    tc_mma(d_tmem, smem_desc(a_addr + k4 * 32), smem_desc(b_addr + k4 * 32), idesc,
                           (i > 0 || k4 > 0) ? 1u : 0u);
                tc_commit(smem_u32(&s.empty[st]));
            }
            if (ok) tc_commit(smem_u32(s.tfull));
            if (h == 0) trace_stamp(p.trace, 3);
        }
    } else {
        // ---------------- epilogue: two groups of 128 threads
        const int grp = (warp - BG_EPI_WARP0) >> 2;       // 0 .. BG_GROUPS - 1
        const int e = (threadIdx.x - 32 * BG_EPI_WARP0) & 127;   // index within the group
        const int e2 = threadIdx.x - 32 * BG_EPI_WARP0;   // index over all groups
        const int quad = warp & 3;                        // TMEM lane quadrant this warp may read
        const int feat = quad * 32 + lane;                // feature (TMEM lane) this thread drains
        const int bar_id = 1 + grp;
        const int n_pass = (T + rpr - 1) / rpr;
        // everything read below besides the accumulator (row statistics, residual stream, row metadata) is final
        // once the previous kernel has finished
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int r = e2; r < T; r += 128 * BG_GROUPS) {
            float v = 1.f;
            if (p.sumsq_in_parts > 0) {
                float acc = 0.f;
                for (int q = 0; q < p.sumsq_in_parts; ++q) acc += __ldcg(p.sumsq_in + (size_t)q * TC_X_ROWS + r);
                v = rsqrtf(acc * p.inv_dim + p.eps);
            }
            s.rstd[r] = v;
        }
        if (e2 == 0) {
            s.flags[0] = (n_kb == 0 || mbar_wait(smem_u32(s.tfull), 0u, abort_flag)) ? 1 : 0;
            // the bytes this CTA is to receive: every rank's partial rows of the passes it owns
            uint32_t rows = 0;
            for (int pass = rank; pass < n_pass; pass += csize) rows += (uint32_t)(min(T, pass * rpr + rpr) - pass * rpr);
            mbar_expect_tx(smem_u32(s.rfull), rows * (uint32_t)(csize * mh * TC_TILE_N * 4));
        }
        both_bar();                                       // also publishes rstd
        if (e2 == 0) trace_stamp(p.trace, 4);
        const bool have = s.flags[0] != 0;
        tc_fence_after();
        // first cluster barrier: every CTA of the cluster has its MMAs behind it (or gave up), no ring is read any more
        cluster_arrive_release();
        cluster_wait_acquire();
        // This CTA's partial tile goes to the staging area behind the receive slots, rows in order, [row][half][128]:
        // the rows of a pass are one contiguous piece, which one bulk copy takes to the pass's owner.
        float* recv = reinterpret_cast<float*>(s.ring);
        float* stage_out = recv + bg_recv_floats(T, rpr, csize, mh);
        const int nblk = (T + 15) / 16;
        // 16 rows of half h: tensor memory -> staging area
        auto stage_block = [&](int h, int rb) {
            const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(h * acc_cols);
            float v[16];
            if (n_kb == 0) {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0.f;
            } else if (terms == 3) {
                float w[48];
                tc_ld16(t_acc + 3 * rb, w);
                tc_ld32(t_acc + 3 * rb + 16, w + 16);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = w[3 * j] + (w[3 * j + 1] + w[3 * j + 2]);
            } else {
                float w[32];
                tc_ld32(t_acc + 2 * rb, w);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = w[2 * j] + w[2 * j + 1];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (rb + j < T) stage_out[((size_t)(rb + j) * mh + h) * TC_TILE_N + feat] = v[j];
        };
        auto send_pass = [&](int pass) {
            const int r0 = pass * rpr, rows = min(T, r0 + rpr) - r0;
            const int owner = pass % csize, own = pass / csize;
            const uint32_t dst = smem_u32(recv) + (uint32_t)((own * csize + rank) * rpr * mh * TC_TILE_N) * 4u;
            bulk_copy_to_rank(dst, smem_u32(stage_out + (size_t)r0 * mh * TC_TILE_N), (uint32_t)(rows * mh * TC_TILE_N * 4),
                              smem_u32(s.rfull), (uint32_t)owner);
        };
        if (rpr == 8) {
            // Passes of eight rows sit inside the 16-row blocks: a group stages whole blocks (both halves) and sends a
            // block's two passes as soon as the block is in the staging area, so that the transfers run while the rest
            // is still being drained.
            for (int b = grp; b < nblk; b += BG_GROUPS) {
                if (have)
                    for (int h = 0; h < mh; ++h) stage_block(h, b * 16);
                tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the copies read what was just written
                epi_bar(bar_id);
                if (have && e < 2 && 2 * b + e < n_pass) send_pass(2 * b + e);
            }
            if (e2 == 0) trace_stamp(p.trace, 5);
        } else {
            // the groups share out the (half, 16 rows) blocks; the copies go out when everything is staged
            if (have)
                for (int it = grp; it < mh * nblk; it += BG_GROUPS) stage_block(it / nblk, (it % nblk) * 16);
            tc_fence_before();
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            both_bar();
            if (e2 == 0) trace_stamp(p.trace, 5);
            if (have && e2 < n_pass) send_pass(e2);
        }
        if (e2 == 0) s.flags[0] = (have && mbar_wait(smem_u32(s.rfull), 0u, abort_flag)) ? 1 : 0;
        both_bar();
        const bool got = s.flags[0] != 0;
        // second cluster barrier, waited for at the very end: nobody leaves while a copy still reads its staging area
        // or writes its slots (every CTA arrives once all its own rows are in, or it gave up waiting)
        cluster_arrive_release();
        if (e2 == 0) trace_stamp(p.trace, 6);
        if (got && !*abort_flag) {
            // The (pass, half) pairs of this CTA, shared out between the groups (SwiGLU pairs the two halves, so there a
            // whole pass is one piece of work): the sum of the csize partial rows in rank order (deterministic), times
            // the row's deferred RMSNorm scale, then the fused epilogue.
            float(*epi)[BG_ROWS][TC_TILE_N + 1] =
                reinterpret_cast<float(*)[BG_ROWS][TC_TILE_N + 1]>(s.epi + (size_t)grp * (BG_EPI_BYTES / sizeof(float)));
            float4* red4 = s.red4 + grp * 4 * BG_ROWS;
            const bool paired = p.mode == TC_SWIGLU;
            const int per_pass = paired ? 1 : mh;
            int idx = 0;
            for (int own = 0, pass = rank; pass < n_pass; ++own, pass += csize) {
                const int r0 = pass * rpr, t_end = min(T, r0 + rpr);
                for (int w = 0; w < per_pass; ++w, ++idx) {
                    if (idx % BG_GROUPS != grp) continue;
                    const int h0 = paired ? 0 : w, h1 = paired ? mh : w + 1;
                    for (int h = h0; h < h1; ++h) {
                        float acc[BG_ROWS];
#pragma unroll
                        for (int j = 0; j < BG_ROWS; ++j) acc[j] = 0.f;
                        // all BG_ROWS rows are read whatever rpr is (what lies behind a slot is the next slot or the
                        // staging area): unconditional loads can be issued together, guarded ones come one by one
                        const float* q0 = recv + (((size_t)(own * csize) * rpr) * mh + h) * TC_TILE_N + e;
                        const size_t src_stride = (size_t)rpr * mh * TC_TILE_N, row_stride = (size_t)mh * TC_TILE_N;
                        int src = 0;
                        for (; src + 2 <= csize; src += 2) {
                            float v0[BG_ROWS], v1[BG_ROWS];
#pragma unroll
                            for (int j = 0; j < BG_ROWS; ++j) {
                                v0[j] = q0[src * src_stride + j * row_stride];
                                v1[j] = q0[(src + 1) * src_stride + j * row_stride];
                            }
#pragma unroll
                            for (int j = 0; j < BG_ROWS; ++j) acc[j] = (acc[j] + v0[j]) + v1[j];
                        }
                        if (src < csize) {
#pragma unroll
                            for (int j = 0; j < BG_ROWS; ++j) acc[j] += q0[src * src_stride + j * row_stride];
                        }
#pragma unroll
                        for (int j = 0; j < BG_ROWS; ++j)
                            epi[paired ? h : 0][j][e] = (r0 + j < t_end) ? acc[j] * s.rstd[r0 + j] : 0.f;
                    }
                    epi_bar(bar_id);
                    const int t128 = tile * mh + w;
                    if (paired) {
                        epi_swiglu<BG_ROWS>(p, epi, tile, r0, t_end, e);
                    } else if (t128 * TC_TILE_N < p.n_rows_total) {     // (a half beyond the last weight row: nothing)
                        switch (p.mode) {
                            case TC_PLAIN: epi_plain<BG_ROWS>(p, epi[0], t128, r0, t_end, e); break;
                            case TC_QKV: epi_qkv<BG_ROWS>(p, epi[0], t128, r0, t_end, e); break;
                            case TC_RESID:
                                epi_resid<BG_ROWS>(p, reinterpret_cast<float*>(red4), epi[0], t128, r0, t_end, e, bar_id);
                                break;
                            default: epi_lmhead<BG_ROWS>(p, red4, epi[0], t128, r0, t_end, e, bar_id); break;
                        }
                    }
                    epi_bar(bar_id);
                }
            }
        }
        cluster_wait_acquire();                           // second barrier (see above)
    }
    // ---------------- teardown: the roles that took no part in the exchange pass both cluster barriers here ----------
    if (warp < BG_EPI_WARP0) {
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) trace_stamp(p.trace, 7);
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag && p.status) {
        const int nseq = p.R > 0 ? (T + p.R - 1) / p.R : 1;
        for (int b = 0; b < nseq; ++b) atomicOr(p.status + b, MTAD_ST_TIMEOUT);
    }
}

cudaError_t bg_set_attributes() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!done[dev]) {
        e = cudaFuncSetAttribute(tc_gemm_cluster_big_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}

// Stand-in for the occupancy query below (the runtime's occupancy calculator does not count kernels that allocate
// tensor memory the way the hardware places them; this kernel has the same block size and no tensor memory).
__global__ void __launch_bounds__(BG_THREADS, 1) bg_occupancy_probe_kernel(int* p) {
    extern __shared__ uint8_t probe_smem[];
    if (p) p[0] = probe_smem[0];
}

// Clusters of `csize` CTAs, one CTA per SM, that can be resident at once (a cluster must fit one GPC, so this is less
// than sms / csize).  Asked once per device and size; without a device the plain quotient.
int bg_max_active_clusters(int csize, int sms) {
    static int cache[64][9] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || csize < 1 || csize > 8) return sms / csize;
    if (cache[dev][csize] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(csize * 148);
        cfg.blockDim = dim3(BG_THREADS);
        cfg.dynamicSmemBytes = BG_BUDGET;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = csize;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(bg_occupancy_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, bg_occupancy_probe_kernel, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = -1;
        }
        cache[dev][csize] = n;
    }
    return cache[dev][csize] > 0 ? cache[dev][csize] : sms / csize;
}

// Shared memory of a launch below the fixed tail: the copy ring; the receive slots and the staging area of the CTA's
// own partial tile lie over it.
struct BgLayout { size_t region, stage_bytes, exchange; int stages; };
BgLayout bg_layout(int T, int rpad, int terms, int mh, int rpr, int csize) {
    BgLayout l{};
    const size_t fixed = BG_TAIL + 1024;
    l.stage_bytes = (size_t)mh * TC_TILE_N * 128 + (size_t)terms * rpad * 128;
    l.region = (BG_BUDGET - fixed) / 1024 * 1024;
    l.exchange = ((size_t)bg_recv_floats(T, rpr, csize, mh) + (size_t)T * mh * TC_TILE_N) * sizeof(float) +
                 (size_t)BG_ROWS * mh * TC_TILE_N * sizeof(float);      // (the last slot is read BG_ROWS rows deep)
    l.stages = (int)std::min<size_t>(l.region / l.stage_bytes, MAX_STAGES);
    return l;
}

}  // namespace

bool tc_cluster_plan_big(TcGemmParams& p, int n_tiles128, int K, int T, int sms) {
    p.k_blocks = (K + TC_TILE_K - 1) / TC_TILE_K;
    p.T = T;
    p.rpad = (T + 15) / 16 * 16;
    p.terms = tc_terms(T);
    p.out_terms = p.terms;
    p.n_bbox = 1;
    p.nbuf = 1;
    p.sliced = 0;
    p.per_sm = 1;
    p.recv_alias = 1;
    p.tile_base = 0;
    const int cols = p.terms * p.rpad;
    if (n_tiles128 < 1 || cols > 256) return false;
    // two halves of weights against the same operand rows where tensor memory (512 columns) and the exchange area
    // allow, else one; the largest cluster whose tiles are all resident in one wave and whose exchange fits
    for (int mh = 2 * cols <= 512 ? 2 : 1; mh >= 1; --mh) {
        if (p.mode == TC_QKV && (p.seg_k_tile % mh || p.seg_v_tile % mh || n_tiles128 % mh)) continue;   // no tile straddles q | k | v
        const int n_tiles = (n_tiles128 + mh - 1) / mh;
        int c = std::min(std::min(sms / n_tiles, 8), p.k_blocks);          // (8: portable cluster size)
        while (c >= 1 && bg_max_active_clusters(c, sms) < n_tiles) --c;
        for (; c >= 1; --c) {
            const int rpr = std::max(1, std::min((T + c - 1) / c, BG_ROWS));
            const BgLayout l = bg_layout(T, p.rpad, p.terms, mh, rpr, c);
            if (l.stages < 2 || l.exchange > l.region) continue;
            p.mh = mh;
            p.n_tiles = n_tiles;
            p.total_units = n_tiles * p.k_blocks;
            p.csize = c;
            p.units_per_cta = (p.k_blocks + c - 1) / c;
            p.max_contrib = c;
            p.rpr = rpr;
            return true;
        }
    }
    return false;                      // more tiles than SMs (a second wave would start late), or no room for the exchange
}

// A matrix with more tiles than half the SMs (a single launch would leave every CTA a whole tile) as two launches over two ranges of its tiles: the first fills the SMs with small
// clusters, the second spreads the remaining tiles over large ones (its weights are requested while the first one
// finishes).  Both read the same operand rows; neither depends on the other.
bool tc_cluster_plan_big_split(TcGemmParams& a, TcGemmParams& b, int n_tiles128, int K, int T, int sms) {
    TcGemmParams p = a;
    p.k_blocks = (K + TC_TILE_K - 1) / TC_TILE_K;
    p.T = T;
    p.rpad = (T + 15) / 16 * 16;
    p.terms = tc_terms(T);
    p.out_terms = p.terms;
    p.n_bbox = 1;
    p.nbuf = 1;
    p.sliced = 0;
    p.per_sm = 1;
    p.recv_alias = 1;
    const int cols = p.terms * p.rpad;
    if (n_tiles128 < 1 || cols > 256 || p.mode == TC_QKV) return false;
    const int mh = 2 * cols <= 512 ? 2 : 1;
    p.mh = mh;
    const int n_tiles = (n_tiles128 + mh - 1) / mh;
    if (2 * n_tiles <= sms || n_tiles >= 2 * sms) return false;    // (up to sms / 2 tiles: one launch of clusters of two or more)
    int best_a = 0, best_b = 0, best_n = 0;
    double best_cost = 1e30;
    for (int ca = 2; ca <= 4 && ca <= p.k_blocks; ++ca) {
        const int na = std::min(n_tiles - 1, bg_max_active_clusters(ca, sms));
        const int rest = n_tiles - na;
        int cb = std::min(std::min(8, sms / rest), p.k_blocks);
        while (cb >= 1 && bg_max_active_clusters(cb, sms) < rest) --cb;
        if (na < 1 || cb < 1) continue;
        const double cost = (double)p.k_blocks / ca + (double)p.k_blocks / cb;      // k-blocks a CTA streams, both launches
        if (cost < best_cost) { best_cost = cost; best_a = ca; best_b = cb; best_n = na; }
    }
    if (!best_a) return false;
    auto fill = [&](TcGemmParams& q, int tiles, int base, int c) -> bool {
        q = p;
        q.n_tiles = tiles;
        q.tile_base = base;
        q.total_units = tiles * q.k_blocks;
        q.csize = c;
        q.units_per_cta = (q.k_blocks + c - 1) / c;
        q.max_contrib = c;
        q.rpr = std::max(1, std::min((T + c - 1) / c, BG_ROWS));
        const BgLayout l = bg_layout(T, q.rpad, q.terms, mh, q.rpr, c);
        return l.stages >= 2 && l.exchange <= l.region;
    };
    return fill(a, best_n, 0, best_a) && fill(b, n_tiles - best_n, best_n, best_b);
}

cudaError_t launch_tc_cluster_big(const TcMaps& maps, const TcGemmParams& p_in, bool pdl, cudaStream_t st) {
    TcGemmParams p = p_in;
    if ((p.mh != 1 && p.mh != 2) || p.csize < 1 || p.csize > 8 || p.per_sm != 1 || p.rpr < 1 || p.rpr > BG_ROWS)
        return cudaErrorInvalidValue;
    const int acc_cols = p.terms * p.rpad;
    if (acc_cols > 256 || acc_cols % 16 || p.mh * acc_cols > 512 || p.T > 128 * BG_GROUPS) return cudaErrorInvalidValue;
    const BgLayout l = bg_layout(p.T, p.rpad, p.terms, p.mh, p.rpr, p.csize);
    if (l.stages < 2 || l.exchange > l.region) return cudaErrorInvalidValue;
    p.stages = l.stages;
    p.ring_bytes = (int)l.region;
    const size_t smem = l.region + BG_TAIL + 1024;
    cudaError_t e = bg_set_attributes();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.n_tiles * p.csize);
    cfg.blockDim = dim3(BG_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = p.csize;
    at[1].val.clusterDim.y = 1;
    at[1].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, tc_gemm_cluster_big_kernel, maps, p);
}

// The cluster variant for a call of T rows: the small kernel next to a second CTA (up to 32 rows), the big one beyond.
bool tc_cluster_plan(TcGemmParams& p, int n_tiles128, int K, int T, int sms) {
    if (tc_ctas_per_sm(T) == 2) return tc_cluster_plan_small(p, n_tiles128, K, T, 2 * sms);
    return tc_cluster_plan_big(p, n_tiles128, K, T, sms);
}

cudaError_t launch_tc_cluster(const TcMaps& maps, const TcGemmParams& p, bool pdl, cudaStream_t st) {
    return p.per_sm == 2 ? launch_tc_cluster_small(maps, p, pdl, st) : launch_tc_cluster_big(maps, p, pdl, st);
}

}  // namespace mtad
