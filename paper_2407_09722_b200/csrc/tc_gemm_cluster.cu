// Tensor-core weight-streaming GEMM with the split-K reduction inside a thread-block cluster.
//
// Same contraction, operands, tiles and fused epilogues as tc_gemm.cu; what differs is how a tile's k-range is
// shared out and how the partial sums meet.  A cluster of `csize` CTAs owns one 128-feature tile; CTA `rank` of the
// cluster streams the k-blocks [rank * KB / csize, (rank + 1) * KB / csize) into one accumulator in tensor memory.
// The draft rows are cut into passes of `rpr` (at most eight) rows; pass q belongs to rank q % csize.  When its
// accumulator is complete a CTA drains it and stores every row straight into the shared memory of the row's owner
// (distributed shared memory, st.shared::cluster), one slot per source rank; a cluster barrier later each owner adds
// the csize slots of its rows in rank order (deterministic) and runs the fused epilogue on them.  No partial tile
// goes through global memory, no counter is polled, and the epilogue passes of a tile run side by side on several
// SMs.  With csize = 1 (LM head: more tiles than CTA slots) the same code is a plain one-tile-per-CTA GEMM.
//
// Warps: 0 weight producer (TMA), 1 operand-row producer (TMA; the only role besides the epilogue that waits for the
// previous kernel), 2 MMA issuer (owns the tensor-memory allocation), 3..6 epilogue (one TMEM lane quadrant each).
// Every mbarrier wait is bounded; a time-out raises MTAD_ST_TIMEOUT for every sequence of the call, and the CTA
// still takes part in both cluster barriers (they are hardware barriers over co-scheduled CTAs, not polls) so that
// its neighbours never wait for it, waits (bounded) for its copies in flight, frees its tensor memory and returns.
#include <algorithm>

#include "tc_device.cuh"

namespace mtad {
using namespace tcdev;
namespace {

constexpr int CL_THREADS = 32 * 7;
constexpr int CL_EPI_WARP0 = 3;

struct ClSmem {
    uint8_t* ring;
    float (*epi)[TC_TILE_N + 1];   // [EPI_ROWS][feature]: the rows of the pass being finished
    float* recv;                   // [own pass][source rank][rpr][128]
    float* rstd;                   // [TC_MAX_ROWS]
    float4* red4;                  // [4][EPI_ROWS] float4 epilogue scratch (also used as floats)
    uint64_t* full;
    uint64_t* empty;
    uint64_t* tfull;
    uint32_t* tmem_ptr;
    int* abort_flag;
    int* flags;
};

constexpr size_t CL_EPI_BYTES = (sizeof(float) * EPI_ROWS * (TC_TILE_N + 1) + 15) / 16 * 16;
constexpr size_t CL_TAIL = CL_EPI_BYTES + sizeof(float) * TC_MAX_ROWS + sizeof(float4) * 4 * EPI_ROWS +
                           8 * (2 * MAX_STAGES + 1) + 8 + 8 + 32;

__device__ __forceinline__ ClSmem cl_carve(uint8_t* base, int stages, int stage_bytes, int recv_bytes) {
    ClSmem s;
    s.ring = base;
    uint8_t* p = base + (size_t)stages * stage_bytes;
    s.epi = reinterpret_cast<float(*)[TC_TILE_N + 1]>(p);
    p += CL_EPI_BYTES;
    s.recv = reinterpret_cast<float*>(p);
    p += recv_bytes;
    s.rstd = reinterpret_cast<float*>(p);
    p += sizeof(float) * TC_MAX_ROWS;
    s.red4 = reinterpret_cast<float4*>(p);
    p += sizeof(float4) * 4 * EPI_ROWS;
    s.full = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.empty = reinterpret_cast<uint64_t*>(p);
    p += 8 * MAX_STAGES;
    s.tfull = reinterpret_cast<uint64_t*>(p);
    p += 8;
    s.tmem_ptr = reinterpret_cast<uint32_t*>(p);
    p += 8;
    s.abort_flag = reinterpret_cast<int*>(p);
    p += 8;
    s.flags = reinterpret_cast<int*>(p);
    return s;
}

// receive slots of one CTA: passes it owns x source ranks x rows per pass x 128 features
__host__ __device__ inline int cl_recv_floats(int T, int rpr, int csize) {
    const int n_pass = (T + rpr - 1) / rpr;
    const int own = (n_pass + csize - 1) / csize;
    return own * csize * rpr * TC_TILE_N;
}

__global__ void __launch_bounds__(CL_THREADS, 2) tc_gemm_cluster_kernel(const __grid_constant__ TcMaps mp,
                                                                       const __grid_constant__ TcGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // every CTA of the cluster must carve identically: the remote stores use this CTA's own offsets
    uint8_t* smem_base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int terms = p.terms, T = p.T;
    const int acc_cols = terms * p.rpad;               // one accumulator column per operand row
    const int a_bytes = TC_TILE_N * 128;
    const int stage_bytes = a_bytes + acc_cols * 128;
    const int stages = p.stages;
    const int csize = p.csize, rpr = p.rpr;
    const ClSmem s = cl_carve(smem_base, stages, stage_bytes, cl_recv_floats(T, rpr, csize) * (int)sizeof(float));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const int tile = (int)blockIdx.x / csize;
    const int kb0 = (int)(((long long)rank * p.k_blocks) / csize);
    const int kb1 = (int)(((long long)(rank + 1) * p.k_blocks) / csize);
    const int n_kb = kb1 - kb0;
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mp.a0)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mp.x)) : "memory");
        for (int i = 0; i < stages; ++i) {
            mbar_init(smem_u32(&s.full[i]), 1);
            mbar_init(smem_u32(&s.empty[i]), 1);
        }
        mbar_init(smem_u32(s.tfull), 1);
        s.abort_flag[0] = 0;
        s.abort_flag[1] = (int)(p.wait_limit ? p.wait_limit : WAIT_LIMIT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < acc_cols) tmem_cols <<= 1;
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
    // first cluster barrier: every CTA of the cluster is running (its shared memory may be written from now on);
    // the arrival costs nothing here, the matching wait comes right before the first remote store
    cluster_arrive_release();
    volatile int* abort_flag = s.abort_flag;

    if (warp == 0) {
        // ---------------- weight producer: copies go out as soon as a stage is free, before the previous kernel ends
        if (lane == 0) {
            const int nb = a_boxes(p.mode, 1);
            for (int i = 0; i < n_kb; ++i) {
                const int st = i % stages;
                if (i >= stages && !mbar_wait(smem_u32(&s.empty[st]), (((uint32_t)(i / stages)) & 1u) ^ 1u, abort_flag))
                    break;
                const uint32_t bar = smem_u32(&s.full[st]);
                const uint32_t base = smem_u32(s.ring + (size_t)st * stage_bytes);
                mbar_expect_tx(bar, (uint32_t)stage_bytes);
                for (int b = 0; b < nb; ++b) {
                    int which, y, row_off;
                    a_box(p.mode, 1, p.seg_k_tile, p.seg_v_tile, tile, b, which, y, row_off);
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
    } else if (warp == 2) {
        // ---------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(acc_cols >> 3) << 17) |
                                   ((uint32_t)(TC_TILE_N >> 4) << 24);
            bool ok = true;
            for (int i = 0; i < n_kb && ok; ++i) {
                const int st = i % stages;
                ok = mbar_wait(smem_u32(&s.full[st]), (uint32_t)(i / stages) & 1u, abort_flag);
                if (!ok) break;
                if (i == 0) trace_stamp(p.trace, 2);
                tc_fence_after();
                const uint32_t a_addr = smem_u32(s.ring + (size_t)st * stage_bytes);
                const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
                for (int k4 = 0; k4 < TC_TILE_K / 16; ++k4)
                    tc_mma(tmem_base, smem_desc(a_addr + k4 * 32), smem_desc(b_addr + k4 * 32), idesc,
                           (i > 0 || k4 > 0) ? 1u : 0u);
                tc_commit(smem_u32(&s.empty[st]));
            }
            if (ok) tc_commit(smem_u32(s.tfull));
            trace_stamp(p.trace, 3);
        }
    } else {
        // ---------------- epilogue
        const int e = threadIdx.x - 32 * CL_EPI_WARP0;   // 0..127
        const int quad = warp & 3;                        // TMEM lane quadrant this warp may read
        const int feat = quad * 32 + lane;                // feature (TMEM lane) this thread drains
        // everything read below besides the accumulator (row statistics, residual stream, row metadata) is final
        // once the previous kernel has finished
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int r = e; r < T; r += EPI_THREADS) {
            float v = 1.f;
            if (p.sumsq_in_parts > 0) {
                float acc = 0.f;
                for (int q = 0; q < p.sumsq_in_parts; ++q) acc += __ldcg(p.sumsq_in + (size_t)q * TC_X_ROWS + r);
                v = rsqrtf(acc * p.inv_dim + p.eps);
            }
            s.rstd[r] = v;
        }
        if (e == 0) s.flags[0] = (n_kb == 0 || mbar_wait(smem_u32(s.tfull), 0u, abort_flag)) ? 1 : 0;
        epi_bar();                                        // also publishes rstd
        if (e == 0) trace_stamp(p.trace, 4);
        const bool have = s.flags[0] != 0;
        tc_fence_after();
        cluster_wait_acquire();                           // first barrier: the owners' shared memory is live
        if (have) {
            // drain: row r of this CTA's partial tile goes to slot [own pass of r][this rank] of the row's owner
            const uint32_t t_acc = tmem_base + ((uint32_t)(quad * 32) << 16);
            const uint32_t recv0 = smem_u32(s.recv);
            for (int rb = 0; rb < T; rb += 16) {
                float v[16];
                if (n_kb == 0) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
                } else if (terms == 3) {
                    float w[48];
                    tc_ld16(t_acc + 3 * rb, w);
                    tc_ld16(t_acc + 3 * rb + 16, w + 16);
                    tc_ld16(t_acc + 3 * rb + 32, w + 32);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = w[3 * j] + (w[3 * j + 1] + w[3 * j + 2]);
                } else {
                    float w[32];
                    tc_ld16(t_acc + 2 * rb, w);
                    tc_ld16(t_acc + 2 * rb + 16, w + 16);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = w[2 * j] + w[2 * j + 1];
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int r = rb + j;
                    if (r < T) {
                        const int pass = r / rpr, jr = r - pass * rpr;
                        const int owner = pass % csize, own = pass / csize;
                        const uint32_t off = (uint32_t)(((own * csize + rank) * rpr + jr) * TC_TILE_N + feat) * 4u;
                        st_cluster_f32(recv0 + off, (uint32_t)owner, v[j]);
                    }
                }
            }
        }
        tc_fence_before();
        if (e == 0) trace_stamp(p.trace, 5);
        cluster_arrive_release();                         // second barrier: this CTA's partial rows are on their way
        cluster_wait_acquire();                           // ... and everybody else's have landed here
        if (e == 0) trace_stamp(p.trace, 6);
        const bool all_ok = have && !*abort_flag;
        const int n_pass = (T + rpr - 1) / rpr;
        for (int own = 0, pass = rank; pass < n_pass && all_ok; ++own, pass += csize) {
            const int r0 = pass * rpr, t_end = min(T, r0 + rpr);
            float acc[EPI_ROWS];
#pragma unroll
            for (int j = 0; j < EPI_ROWS; ++j) acc[j] = 0.f;
            for (int src = 0; src < csize; ++src) {       // rank order: deterministic
                const float* q = s.recv + ((size_t)(own * csize + src) * rpr) * TC_TILE_N + e;
#pragma unroll
                for (int j = 0; j < EPI_ROWS; ++j)
                    if (j < rpr) acc[j] += q[j * TC_TILE_N];
            }
#pragma unroll
            for (int j = 0; j < EPI_ROWS; ++j) s.epi[j][e] = (r0 + j < t_end) ? acc[j] * s.rstd[r0 + j] : 0.f;
            epi_bar();
            if (tile * TC_TILE_N < p.n_rows_total || p.mode == TC_SWIGLU) {
                switch (p.mode) {
                    case TC_PLAIN: epi_plain<EPI_ROWS>(p, s.epi, tile, r0, t_end, e); break;
                    case TC_QKV: epi_qkv<EPI_ROWS>(p, s.epi, tile, r0, t_end, e); break;
                    case TC_RESID: epi_resid<EPI_ROWS>(p, reinterpret_cast<float*>(s.red4), s.epi, tile, r0, t_end, e); break;
                    case TC_SWIGLU:
                        epi_swiglu<EPI_ROWS>(p, reinterpret_cast<float(*)[EPI_ROWS][TC_TILE_N + 1]>(s.epi), tile, r0, t_end, e);
                        break;
                    default: epi_lmhead<EPI_ROWS>(p, s.red4, s.epi, tile, r0, t_end, e); break;
                }
            }
            epi_bar();
        }
    }
    // ---------------- teardown: the roles that took no part in the exchange pass both cluster barriers here ----------
    if (warp < CL_EPI_WARP0) {
        __syncwarp();
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

}  // namespace

namespace {
// The kernel may use the whole shared memory of an SM (two CTAs of up to 112 KB share it); once per device.
cudaError_t cl_set_attributes() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!done[dev]) {
        e = cudaFuncSetAttribute(tc_gemm_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(tc_gemm_cluster_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}

// Stand-in for the occupancy query below: same block size and launch bounds, no tensor memory.  The runtime's
// occupancy calculator counts a kernel that allocates tensor memory as one CTA per SM although two CTAs that ask for
// at most 256 columns each do run side by side; asked about this kernel it reports what the hardware does.
__global__ void __launch_bounds__(CL_THREADS, 2) cl_occupancy_probe_kernel(int* p) {
    extern __shared__ uint8_t probe_smem[];
    if (p) p[0] = probe_smem[0];
}

// Clusters of `csize` CTAs of the kernel that can be resident at once (two CTAs per SM; a cluster must fit one GPC, so
// this is less than slots / csize).  Asked once per device and size; without a device the plain quotient.
int max_active_clusters(int csize, int slots) {
    static int cache[64][9] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || csize < 1 || csize > 8) return slots / csize;
    if (cache[dev][csize] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(csize * 296);
        cfg.blockDim = dim3(CL_THREADS);
        cfg.dynamicSmemBytes = 112 * 1024;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = csize;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
if (cudaFuncSetAttribute(cl_occupancy_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, cl_occupancy_probe_kernel, &cfg) != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = -1;
        }
        cache[dev][csize] = n;
    }
    return cache[dev][csize] > 0 ? cache[dev][csize] : slots / csize;
}
}  // namespace

bool tc_cluster_plan_small(TcGemmParams& p, int n_tiles, int K, int T, int slots) {
    p.n_tiles = n_tiles;
    p.k_blocks = (K + TC_TILE_K - 1) / TC_TILE_K;
    p.T = T;
    p.rpad = (T + 15) / 16 * 16;
    p.terms = tc_terms(T);
    p.out_terms = p.terms;
    p.n_bbox = 1;
    p.mh = 1;
    p.per_sm = 2;
    p.nbuf = 1;
    p.sliced = 0;
    p.total_units = n_tiles * p.k_blocks;
    if (n_tiles < 1 || p.terms * p.rpad > 256 || tc_ctas_per_sm(T) != 2) return false;
    int c = slots / n_tiles;
    c = std::min(c, 8);                // portable cluster size
    c = std::min(c, p.k_blocks);
    while (c >= 1 && max_active_clusters(c, slots) < n_tiles) --c;     // every cluster resident in one wave
    if (c < 1) return false;           // more tiles than CTA slots: a second wave would start late
    p.csize = c;
    p.units_per_cta = (p.k_blocks + c - 1) / c;
    p.max_contrib = c;
    int rpr = (T + c - 1) / c;
    p.rpr = std::max(1, std::min(rpr, EPI_ROWS));
    return true;
}

cudaError_t launch_tc_cluster_small(const TcMaps& maps, const TcGemmParams& p_in, bool pdl, cudaStream_t st) {
    TcGemmParams p = p_in;
    if (p.mh != 1 || p.csize < 1 || p.csize > 8 || p.rpr < 1 || p.rpr > EPI_ROWS) return cudaErrorInvalidValue;
    const int acc_cols = p.terms * p.rpad;
    if (acc_cols > 256 || acc_cols % 16) return cudaErrorInvalidValue;
    const int stage_bytes = TC_TILE_N * 128 + acc_cols * 128;
    const size_t recv_bytes = (size_t)cl_recv_floats(p.T, p.rpr, p.csize) * sizeof(float);
    const size_t budget = (size_t)112 * 1024;
    if (CL_TAIL + recv_bytes + 1024 + 2 * (size_t)stage_bytes > budget) return cudaErrorInvalidValue;
    int stages = (int)((budget - CL_TAIL - recv_bytes - 1024) / stage_bytes);
    stages = std::min(stages, MAX_STAGES);
    p.stages = stages;
    const size_t smem = (size_t)stages * stage_bytes + CL_TAIL + recv_bytes + 1024;
    cudaError_t e = cl_set_attributes();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.n_tiles * p.csize);
    cfg.blockDim = dim3(CL_THREADS);
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
    return cudaLaunchKernelEx(&cfg, tc_gemm_cluster_kernel, maps, p);
}

}  // namespace mtad
