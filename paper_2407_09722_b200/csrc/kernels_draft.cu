// Beam-sampling draft with the auxiliary model (Sec. 2.1 of the paper, the p_beam equation; every intermediate
// beam becomes a node of the candidate tree, Sec. 3.3): row bookkeeping of each draft step, the Gumbel-top-b
// selection over (beam, token) pairs, and the roll-forward of the auxiliary KV cache after a verification.
//
// Virtual rows of one draft: the P pending tokens (not yet in the auxiliary cache, the last one is the root) are
// rows 0 .. P-1, node n is row P + n; row v lives in cache slot aux_len + v.
#include <math_constants.h>

#include "common.cuh"

namespace mtad {

namespace {

__device__ __forceinline__ float wsum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct Cand {
    float y;      // perturbed joint score
    int flat;     // beam * V + token
};
__device__ __forceinline__ bool before(const Cand& a, const Cand& b) {     // a ranks ahead of b
    return a.y > b.y || (a.y == b.y && a.flat < b.flat);
}

// The best candidate of a block of 256 threads, returned to every thread: butterfly inside each warp, then the eight
// warp winners through shared memory (two barriers a call; s_w is free again on return).
__device__ __forceinline__ Cand block_best(Cand c, Cand* s_w, int tid) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const Cand c2{__shfl_xor_sync(0xffffffffu, c.y, o), __shfl_xor_sync(0xffffffffu, c.flat, o)};
        if (before(c2, c)) c = c2;
    }
    if ((tid & 31) == 0) s_w[tid >> 5] = c;
    __syncthreads();
    Cand best = s_w[0];
#pragma unroll
    for (int w = 1; w < 8; ++w)
        if (before(s_w[w], best)) best = s_w[w];
    __syncthreads();
    return best;
}

}  // namespace

// ---------------------------------------------------------------------------------------------------------------
// rows of one draft step: step 0 runs the pending tokens as a causal chain, step s >= 1 the nodes of layer s
// ---------------------------------------------------------------------------------------------------------------

__global__ void draft_prepare_kernel(const __nv_bfloat16* __restrict__ embed, int d, int vocab, int hd,
                                     RopeInv rinv, long long kv_capacity, SeqState s, DraftState ds, RowMeta rm,
                                     float* __restrict__ hidden, float* __restrict__ rope, SeqList seqs, int R, int step,
                                     int beam, const __nv_bfloat16* __restrict__ gain0, __nv_bfloat16* x, int terms,
                                     float* sumsq_out, __nv_bfloat16* __restrict__ cache, int layers, int max_batch,
                                     int Hkv) {
    const int t = blockIdx.x, bi = t / R, r = t % R;
    const int seq = seqs.v[bi];
    __shared__ int sh_tok, sh_pos, sh_ok, sh_hole;
    pdl_wait();               // the sequence and draft state, and every buffer written here, belong to earlier kernels
    pdl_trigger();
    if (threadIdx.x == 0) {
        const int L = step == 0 ? s.aux_len[seq] : ds.base_len[seq];
        const int P = step == 0 ? s.aux_npend[seq] : ds.npend[seq];
        if (step == 0 && r == 0) { ds.base_len[seq] = L; ds.npend[seq] = P; }
        uint32_t mask[MTAD_MASK_WORDS];
#pragma unroll
        for (int i = 0; i < MTAD_MASK_WORDS; ++i) mask[i] = 0;
        int tok = 0, pos = L, vrow = 0, hole = -1;
        bool active;
        if (step == 0) {
            active = r < P;
            if (active) {
                tok = s.aux_pend[seq * (MTAD_MAX_DEPTH + 1) + r];
                vrow = r;
                pos = L + r;
                for (int i = 0; i <= r; ++i) mask[i >> 5] |= 1u << (i & 31);        // causal over the pending rows
            }
        } else {
            // the beams the step before kept: the beam width, or fewer on warped rows
            const int nbp = min(max(ds.nb[seq * MTAD_MAX_DEPTH + step - 1], 0), beam);
            active = r < nbp;
            // A beam slot of the layer before that no beam took is a cache row nobody wrote.  This step's rows never
            // look at it (their masks name ancestors only), but a masked key still meets its value row with weight 0, and
            // 0 x (whatever the memory held) must stay 0: the row is cleared (cache != null: only then can slots be empty).
            hole = (cache && !active && r < beam) ? L + P + (step - 1) * beam + r : -1;
            if (active) {
                const int n = (step - 1) * beam + r;
                tok = ds.node_tok[seq * MTAD_DRAFT_NODES + n];
                vrow = P + n;
                pos = L + P - 1 + step;
#pragma unroll
                for (int i = 0; i < MTAD_MASK_WORDS; ++i)
                    mask[i] = ds.node_mask[((size_t)seq * MTAD_DRAFT_NODES + n) * MTAD_MASK_WORDS + i];
            }
        }
        if (tok < 0 || tok >= vocab) tok = 0;
        rm.tok[t] = tok;
        rm.depth[t] = step;
        rm.pos[t] = pos;
        if (L < 0 || P < 1 || P > MTAD_MAX_DEPTH + 1 || (long long)L + vrow >= kv_capacity) active = false;
        rm.slot[t] = active ? L + vrow : -1;
        rm.seq[t] = seq;
        rm.prow[t] = -1;
        // the mask is indexed by cache slot minus L: virtual rows
#pragma unroll
        for (int i = 0; i < MTAD_MASK_WORDS; ++i) rm.mask[(size_t)t * MTAD_MASK_WORDS + i] = mask[i];
        if (r == 0) {
            const bool state_ok = L >= 0 && P >= 1 && P <= MTAD_MAX_DEPTH + 1 && P <= (step == 0 ? R : MTAD_MAX_DEPTH + 1) &&
                                  (long long)L + P + (long long)step * beam <= kv_capacity;
            const int nbp = step == 0 ? 0 : min(max(ds.nb[seq * MTAD_MAX_DEPTH + step - 1], 0), beam);
            rm.n_rows[bi] = !state_ok ? 0 : (step == 0 ? P : nbp);
            rm.n_spec[bi] = !state_ok ? 0 : (step == 0 ? P : P + step * beam);
            rm.kv_base[bi] = L;
            rm.call_seq[bi] = seq;
        }
        sh_tok = tok;
        sh_pos = pos;
        sh_ok = active;
        sh_hole = (hole >= 0 && L >= 0 && (long long)hole < kv_capacity) ? hole : -1;
    }
    __syncthreads();
    if (sh_hole >= 0) {
        for (int i = threadIdx.x; i < layers * 2 * Hkv * hd; i += blockDim.x) {
            const int j = i % hd, head = (i / hd) % Hkv, kv = (i / (hd * Hkv)) & 1, layer = i / (2 * hd * Hkv);
            cache[idx_cache(layer, max_batch, seq, kv, Hkv, head, kv_capacity, sh_hole, hd) + j] = __float2bfloat16_rn(0.f);
        }
    }
    const int tok = sh_tok;
    const bool ok = sh_ok;
    float ss = embed_row(embed + (size_t)tok * d, ok, d, hidden + (size_t)t * d, gain0,
                         x ? x + (size_t)t * terms * d : nullptr, terms);
    if (x) {
        __shared__ float red[32];
        ss = wsum(ss);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) {
            float a = 0.f;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) a += red[w];
            sumsq_out[t] = a;
        }
    }
    for (int i = threadIdx.x; i < hd / 2; i += blockDim.x) {
        float cs, sn;
        rope_cs((double)sh_pos, rinv.v[i], cs, sn);
        rope[((size_t)t * (hd / 2) + i) * 2 + 0] = cs;
        rope[((size_t)t * (hd / 2) + i) * 2 + 1] = sn;
    }
}

cudaError_t launch_draft_prepare(const ModelView& m, const SeqState& s, const DraftState& ds, const RowMeta& rm,
                                 const Scratch& sc, const SeqList& seqs, int B, int R, int step, int beam, bool tc,
                                 bool warped, bool pdl, cudaStream_t st) {
    return launch_pdl(draft_prepare_kernel, dim3(B * R), dim3(128), 0, st, pdl,
                      static_cast<const __nv_bfloat16*>(m.d.embed), m.d.d_model, m.d.vocab, m.d.head_dim,
                      rope_inv((double)m.d.rope_base, m.d.head_dim), (long long)m.d.kv_capacity, s, ds, rm, sc.hidden,
                      sc.rope, seqs, R, step, beam,
                      tc ? m.w(0, 0) : (const __nv_bfloat16*)nullptr, tc ? sc.xd : (__nv_bfloat16*)nullptr,
                      tc_terms(B * R), sc.sumsq_a,
                      warped ? static_cast<__nv_bfloat16*>(m.d.kv_cache) : (__nv_bfloat16*)nullptr, m.d.layers, m.max_batch,
                      m.d.n_kv_heads);
}

// ---------------------------------------------------------------------------------------------------------------
// selection: the `beam` largest of log q(beam) + log q(token | beam) + Gumbel noise over all (beam, token) pairs
//
// Two passes.  draft_scan_kernel, one block per (chunk of the vocabulary, beam row, sequence): the chunk's share of
// the row's log-sum-exp (running maximum and sum) and its `beam` largest perturbed logits t = z - log(-log u).  The
// joint score of a pair is t + (log q(beam) - lse(row)), a per-row constant added in fp32 (monotone), so a pair
// among the overall `beam` largest is among the `beam` largest of its chunk.  draft_pick_kernel, one block per
// sequence: merges the chunks of every row in chunk order, scores the surviving pairs and takes the `beam` largest
// (ties to the lower flat index beam * V + token), then writes the new layer of the tree.
// ---------------------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(256) draft_scan_kernel(const float* __restrict__ logits, int V, int R, int step,
                                                         int gamma, int beam, int kpb, const float* __restrict__ uni,
                                                         DraftState ds, SeqList seqs, DraftPart* __restrict__ part,
                                                         int nch) {
    // kpb: perturbed logits of this chunk to hand on (the beam width, or with all candidates kept the candidates
    // recorded per beam: beam * beam of the single beam of step 0, beam afterwards)
    const int c = blockIdx.x, j = blockIdx.y, bi = blockIdx.z, seq = seqs.v[bi];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_wait();               // the logits come from the kernel before
    pdl_trigger();
    const int P = min(max(ds.npend[seq], 1), step == 0 ? R : MTAD_MAX_DEPTH + 1);   // in range whatever the state holds
    const int row = step == 0 ? P - 1 : j;
    const float* z = logits + (size_t)(bi * R + row) * V;
    const float* ub = uni + (((size_t)bi * gamma + step) * beam + j) * V;
    const int len = (V + nch - 1) / nch, v0 = c * len, v1 = min(V, v0 + len);
    __shared__ float s_m[8], s_s[8];
    __shared__ Cand s_w[8];
    float m = -CUDART_INF_F, sum = 0.f;
    // a thread sees at most MTAD_MAX_BEAM tokens of the chunk (the host keeps chunks within 256 * MTAD_MAX_BEAM), so
    // its sorted list holds all of them and the rounds below find the chunk's exact order
    Cand loc[MTAD_MAX_BEAM];
#pragma unroll
    for (int k = 0; k < MTAD_MAX_BEAM; ++k) loc[k] = Cand{-CUDART_INF_F, 0x7fffffff};
    for (int v = v0 + tid; v < v1; v += 256) {
        const float zv = z[v];
        if (zv > m) { sum = sum * expf(m - zv) + 1.f; m = zv; }
        else sum += expf(zv - m);
        const Cand cd{zv - logf(-logf(ub[v])), v};
        if (before(cd, loc[MTAD_MAX_BEAM - 1])) {
            loc[MTAD_MAX_BEAM - 1] = cd;
#pragma unroll
            for (int k = MTAD_MAX_BEAM - 1; k > 0; --k)
                if (before(loc[k], loc[k - 1])) { const Cand tmp = loc[k]; loc[k] = loc[k - 1]; loc[k - 1] = tmp; }
        }
    }
    // the chunk's maximum and sum of exponentials (fixed combination order: butterfly, then warps in order)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, sum, o);
        const float M = fmaxf(m, m2);
        sum = (M == -CUDART_INF_F) ? 0.f : sum * expf(m - M) + s2 * expf(m2 - M);
        m = M;
    }
    if (lane == 0) { s_m[warp] = m; s_s[warp] = sum; }
    DraftPart* dst = part + ((size_t)(bi * MTAD_MAX_BEAM + j)) * nch + c;
    // kpb rounds: the block's best head-of-list wins, its owner advances
    int head = 0;
    for (int k = 0; k < kpb; ++k) {
        Cand cd{-CUDART_INF_F, 0x7fffffff};
#pragma unroll
        for (int q = 0; q < MTAD_MAX_BEAM; ++q)
            if (q == head) cd = loc[q];
        const Cand win = block_best(cd, s_w, tid);
        if (cd.flat == win.flat && win.flat != 0x7fffffff) ++head;      // the owner of the winner (tokens are unique)
        if (tid == 0) {
            dst->t[k] = win.y;
            dst->v[k] = win.flat == 0x7fffffff ? -1 : win.flat;
        }
    }
    if (tid == 0) {
        float M = -CUDART_INF_F;
        for (int w = 0; w < 8; ++w) M = fmaxf(M, s_m[w]);
        float a = 0.f;
        for (int w = 0; w < 8; ++w) a += (s_m[w] == -CUDART_INF_F) ? 0.f : s_s[w] * expf(s_m[w] - M);
        dst->m = M;
        dst->s = a;
    }
}

__global__ void __launch_bounds__(256) draft_pick_kernel(const float* __restrict__ logits, int V, int R, int step,
                                                         int gamma, int beam, int keep_all, int kpb, DraftState ds,
                                                         SeqList seqs, const DraftPart* __restrict__ part, int nch,
                                                         DraftOut out) {
    const int bi = blockIdx.x, seq = seqs.v[bi];
    const int tid = threadIdx.x;
    pdl_wait();               // the chunk results come from the kernel before
    pdl_trigger();
    const int P = min(max(ds.npend[seq], 1), step == 0 ? R : MTAD_MAX_DEPTH + 1);   // in range whatever the state holds
    const int n_beams = step == 0 ? 1 : beam;
    const int per_layer = keep_all ? beam * beam : beam;          // nodes of a layer of the caller's tree
    const int N = gamma * per_layer;
    __shared__ float s_lse[MTAD_MAX_BEAM], s_lq[MTAD_MAX_BEAM];
    __shared__ int s_slot[MTAD_MAX_BEAM], s_tree[MTAD_MAX_BEAM];   // the current beams: beam slot and tree id (-1: the context)
    __shared__ float s_y[MTAD_MAX_BEAM * MTAD_DRAFT_CHUNKS * MTAD_MAX_BEAM];
    __shared__ int s_flat[MTAD_MAX_BEAM * MTAD_DRAFT_CHUNKS * MTAD_MAX_BEAM];
    __shared__ Cand s_w[8];
    __shared__ float l_y[MTAD_MAX_CAND];                           // the layer's nodes: perturbed score, flat pair,
    __shared__ int l_flat[MTAD_MAX_CAND], l_rank[MTAD_MAX_CAND];   // rank among the kept beams (-1: not kept)
    const DraftPart* pp = part + (size_t)bi * MTAD_MAX_BEAM * nch;
    if (tid < n_beams) {
        // log-sum-exp of beam row tid: chunks in order
        const DraftPart* pj = pp + (size_t)tid * nch;
        float M = -CUDART_INF_F;
        for (int c = 0; c < nch; ++c) M = fmaxf(M, pj[c].m);
        float a = 0.f;
        for (int c = 0; c < nch; ++c) a += (pj[c].m == -CUDART_INF_F) ? 0.f : pj[c].s * expf(pj[c].m - M);
        s_lse[tid] = M + logf(a);
        const int slot = step == 0 ? -1 : (step - 1) * beam + tid;
        s_slot[tid] = slot;
        s_tree[tid] = slot < 0 ? -1 : ds.tree_id[seq * MTAD_DRAFT_NODES + slot];
        s_lq[tid] = slot < 0 ? 0.f : ds.node_logq[seq * MTAD_DRAFT_NODES + slot];
    }
    __syncthreads();
    const int per_beam = nch * kpb;                                // candidates of one beam row
    const int n_cand = n_beams * per_beam;
    for (int i = tid; i < n_cand; i += 256) {
        const int j = i / per_beam, c = (i / kpb) % nch, k = i % kpb;
        const DraftPart& d = pp[(size_t)j * nch + c];
        const bool ok = d.v[k] >= 0;
        s_y[i] = ok ? d.t[k] + (s_lq[j] - s_lse[j]) : -CUDART_INF_F;
        s_flat[i] = ok ? j * V + d.v[k] : 0x7fffffff;
    }
    __syncthreads();
    // The layer's nodes.  Plain tree: the `beam` best pairs of all, best first.  All candidates kept: beam by beam its
    // kpb best pairs, best first.  Every round is a block-wide arg-max over a range of the candidates; the winner is
    // struck out.
    const int n_groups = keep_all ? n_beams : 1, rounds = keep_all ? kpb : beam;
    for (int gidx = 0; gidx < n_groups; ++gidx) {
        const int lo = keep_all ? gidx * per_beam : 0, hi = keep_all ? lo + per_beam : n_cand;
        for (int k = 0; k < rounds; ++k) {
            Cand best{-CUDART_INF_F, 0x7fffffff};
            int bidx = -1;
            for (int i = lo + tid; i < hi; i += 256) {
                const Cand cd{s_y[i], s_flat[i]};
                if (cd.flat != 0x7fffffff && before(cd, best)) { best = cd; bidx = i; }
            }
            const Cand win = block_best(best, s_w, tid);
            const bool found = win.flat != 0x7fffffff;
            if (found && bidx >= 0 && best.flat == win.flat) {       // the owner strikes the winner out (pairs are unique)
                s_y[bidx] = -CUDART_INF_F;
                s_flat[bidx] = 0x7fffffff;
            }
            if (tid == 0) {
                const int m = gidx * rounds + k;
                l_y[m] = found ? win.y : -CUDART_INF_F;
                l_flat[m] = win.flat;
                l_rank[m] = keep_all ? -1 : k;
            }
            __syncthreads();
        }
    }
    if (keep_all && tid == 0) {
        // the beams kept for the next step: the `beam` best of the layer's nodes (they are the best of all pairs)
        for (int k = 0; k < beam; ++k) {
            int bm = -1;
            for (int m = 0; m < per_layer; ++m)
                if (l_rank[m] < 0 && l_flat[m] != 0x7fffffff &&
                    (bm < 0 || before(Cand{l_y[m], l_flat[m]}, Cand{l_y[bm], l_flat[bm]})))
                    bm = m;
            if (bm >= 0) l_rank[bm] = k;
        }
    }
    __syncthreads();
    // every node of the layer, one thread each: the caller's tree, and for a kept node the beam state of the next step
    for (int m = tid; m < per_layer; m += 256) {
        const bool valid = l_flat[m] != 0x7fffffff;        // a vocabulary of at least per_layer tokens always fills the layer
        const int j = valid ? l_flat[m] / V : 0, v = valid ? l_flat[m] % V : 0;
        const int n = step * per_layer + m;
        const int row = step == 0 ? P - 1 : j;
        const float lq = s_lq[j] + logits[(size_t)(bi * R + row) * V + v] - s_lse[j];
        out.tok[bi * N + n] = v;
        out.parent[bi * N + n] = s_tree[j];
        out.depth[bi * N + n] = step + 1;
        out.node_logq[bi * N + n] = lq;
        const int k = l_rank[m];
        if (n < MTAD_DRAFT_NODES) ds.tree2slot[seq * MTAD_DRAFT_NODES + n] = k >= 0 ? step * beam + k : -1;
        if (k >= 0) {
            const int slot = step * beam + k, parent = s_slot[j];
            ds.node_tok[seq * MTAD_DRAFT_NODES + slot] = v;
            ds.node_parent[seq * MTAD_DRAFT_NODES + slot] = parent;
            ds.node_logq[seq * MTAD_DRAFT_NODES + slot] = lq;
            ds.tree_id[seq * MTAD_DRAFT_NODES + slot] = n;
            uint32_t* mk = ds.node_mask + ((size_t)seq * MTAD_DRAFT_NODES + slot) * MTAD_MASK_WORDS;
            for (int i = 0; i < MTAD_MASK_WORDS; ++i) {
                uint32_t w;
                if (parent >= 0) w = ds.node_mask[((size_t)seq * MTAD_DRAFT_NODES + parent) * MTAD_MASK_WORDS + i];
                else {                                        // child of the root: sees all pending rows
                    const int lo = i * 32;
                    w = P >= lo + 32 ? 0xffffffffu : (P > lo ? (1u << (P - lo)) - 1u : 0u);
                }
                if (((P + slot) >> 5) == i) w |= 1u << ((P + slot) & 31);
                mk[i] = w;
            }
        }
    }
    __syncthreads();
    if (tid == 0) ds.nb[seq * MTAD_MAX_DEPTH + step] = beam;      // every beam slot of the layer is taken
    if (step == gamma - 1 && tid == 0) {
        // x**: the final beam with the highest draft likelihood (lowest tree id on ties), and its prefix likelihoods
        __threadfence_block();
        int best = (gamma - 1) * beam;
        for (int k = 1; k < beam; ++k) {
            const int sl = (gamma - 1) * beam + k;
            const float a = ds.node_logq[seq * MTAD_DRAFT_NODES + sl], b0 = ds.node_logq[seq * MTAD_DRAFT_NODES + best];
            if (a > b0 || (a == b0 && ds.tree_id[seq * MTAD_DRAFT_NODES + sl] < ds.tree_id[seq * MTAD_DRAFT_NODES + best]))
                best = sl;
        }
        int cur = best;
        for (int i = gamma - 1; i >= 0 && cur >= 0; --i) {
            out.best_path[bi * gamma + i] = ds.tree_id[seq * MTAD_DRAFT_NODES + cur];
            out.logq_ref[bi * gamma + i] = ds.node_logq[seq * MTAD_DRAFT_NODES + cur];
            ds.best_path[seq * MTAD_MAX_DEPTH + i] = cur;
            cur = ds.node_parent[seq * MTAD_DRAFT_NODES + cur];
        }
        ds.gamma[seq] = gamma;
        ds.beam[seq] = beam;
        if (out.n_nodes) out.n_nodes[bi] = N;
    }
}

// ---------------------------------------------------------------------------------------------------------------
// selection on warped rows (App. F): every beam row has been cut to its kept tokens (warp_scan / warp_merge: at most
// MTAD_MAX_TOPK tokens with renormalised log-probabilities), so the candidates of a step are the at most
// beam * MTAD_MAX_TOPK (beam, kept token) pairs and one block per sequence ranks them all.  A step may find fewer
// pairs than beams: it keeps what there is, the layer holds fewer nodes, node ids stay consecutive.
// ---------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) draft_pick_warped_kernel(const WarpRow* __restrict__ rows, int V, int R, int step,
                                                                int gamma, int beam, int keep_all,
                                                                const float* __restrict__ uni, DraftState ds,
                                                                SeqList seqs, DraftOut out) {
    const int bi = blockIdx.x, seq = seqs.v[bi];
    const int tid = threadIdx.x;
    const int P = min(max(ds.npend[seq], 1), step == 0 ? R : MTAD_MAX_DEPTH + 1);
    const int n_beams = step == 0 ? 1 : min(max(ds.nb[seq * MTAD_MAX_DEPTH + step - 1], 0), beam);
    const int kpb = (keep_all && step == 0) ? beam * beam : beam;       // nodes a beam may contribute with all kept
    const int N = gamma * (keep_all ? beam * beam : beam);              // capacity of the caller's arrays
    constexpr int NC = MTAD_MAX_BEAM * MTAD_MAX_TOPK;
    __shared__ float s_lq[MTAD_MAX_BEAM];
    __shared__ int s_slot[MTAD_MAX_BEAM], s_tree[MTAD_MAX_BEAM];
    __shared__ float s_y[NC], s_lp[NC];
    __shared__ int s_flat[NC];
    __shared__ Cand s_w[8];
    __shared__ float l_y[MTAD_MAX_CAND], l_lp[MTAD_MAX_CAND];
    __shared__ int l_flat[MTAD_MAX_CAND], l_rank[MTAD_MAX_CAND], l_id[MTAD_MAX_CAND];
    __shared__ int s_count[2];                       // nodes of the layer, beams kept
    if (tid < n_beams) {
        const int slot = step == 0 ? -1 : (step - 1) * beam + tid;
        s_slot[tid] = slot;
        s_tree[tid] = slot < 0 ? -1 : ds.tree_id[seq * MTAD_DRAFT_NODES + slot];
        s_lq[tid] = slot < 0 ? 0.f : ds.node_logq[seq * MTAD_DRAFT_NODES + slot];
    }
    __syncthreads();
    if (tid < NC) {
        const int j = tid / MTAD_MAX_TOPK, i = tid % MTAD_MAX_TOPK;
        bool ok = j < n_beams;
        float y = -CUDART_INF_F, lp = 0.f;
        int flat = 0x7fffffff;
        if (ok) {
            const WarpRow& row = rows[bi * R + (step == 0 ? P - 1 : j)];
            ok = i < min(row.n, MTAD_MAX_TOPK);
            if (ok) {
                const int v = row.idx[i];
                ok = v >= 0 && v < V;
                if (ok) {
                    lp = row.lp[i];
                    y = (s_lq[j] + lp) - logf(-logf(uni[(((size_t)bi * gamma + step) * beam + j) * V + v]));
                    flat = j * V + v;
                }
            }
        }
        s_y[tid] = y; s_lp[tid] = lp; s_flat[tid] = flat;
    }
    __syncthreads();
    // the layer's nodes: the `beam` best pairs of all, or with every candidate kept each beam's kpb best, best first
    const int n_groups = keep_all ? n_beams : 1, rounds = keep_all ? min(kpb, MTAD_MAX_TOPK) : beam;
    for (int gidx = 0; gidx < n_groups; ++gidx) {
        const int lo = keep_all ? gidx * MTAD_MAX_TOPK : 0, hi = keep_all ? lo + MTAD_MAX_TOPK : NC;
        for (int k = 0; k < rounds; ++k) {
            Cand best{-CUDART_INF_F, 0x7fffffff};
            const int i = lo + tid;
            if (i < hi && s_flat[i] != 0x7fffffff) best = Cand{s_y[i], s_flat[i]};
            const Cand win = block_best(best, s_w, tid);
            const bool found = win.flat != 0x7fffffff;
            if (tid == 0) {
                const int m = gidx * rounds + k;
                if (m < MTAD_MAX_CAND) { l_y[m] = found ? win.y : -CUDART_INF_F; l_flat[m] = win.flat; l_rank[m] = -1; }
            }
            if (found && best.flat == win.flat) {                     // the owner (pairs are unique) strikes the winner out
                const int m = gidx * rounds + k;
                if (m < MTAD_MAX_CAND) l_lp[m] = s_lp[i];
                s_flat[i] = 0x7fffffff;
            }
            __syncthreads();
        }
    }
    const int per_layer = min(n_groups * rounds, MTAD_MAX_CAND);
    if (tid == 0) {
        // consecutive node ids for the pairs that exist; the beams kept: the `beam` best of them
        const int base_id = step == 0 ? 0 : max(ds.n_tree[seq], 0);
        int cnt = 0;
        for (int m = 0; m < per_layer; ++m) l_id[m] = l_flat[m] != 0x7fffffff ? base_id + cnt++ : -1;
        int kept = 0;
        for (int k = 0; k < beam; ++k) {
            int bm = -1;
            for (int m = 0; m < per_layer; ++m)
                if (l_rank[m] < 0 && l_flat[m] != 0x7fffffff &&
                    (bm < 0 || before(Cand{l_y[m], l_flat[m]}, Cand{l_y[bm], l_flat[bm]})))
                    bm = m;
            if (bm < 0) break;
            l_rank[bm] = k;
            ++kept;
        }
        s_count[0] = cnt;
        s_count[1] = kept;
        ds.nb[seq * MTAD_MAX_DEPTH + step] = kept;
        ds.n_tree[seq] = base_id + cnt;
    }
    __syncthreads();
    for (int m = tid; m < per_layer; m += 256) {
        const int n = l_id[m];
        if (n < 0 || n >= N || n >= MTAD_DRAFT_NODES) continue;
        const int j = l_flat[m] / V, v = l_flat[m] % V;
        const float lq = s_lq[j] + l_lp[m];
        out.tok[bi * N + n] = v;
        out.parent[bi * N + n] = s_tree[j];
        out.depth[bi * N + n] = step + 1;
        out.node_logq[bi * N + n] = lq;
        const int k = l_rank[m];
        ds.tree2slot[seq * MTAD_DRAFT_NODES + n] = k >= 0 ? step * beam + k : -1;
        if (k >= 0) {
            const int slot = step * beam + k, parent = s_slot[j];
            ds.node_tok[seq * MTAD_DRAFT_NODES + slot] = v;
            ds.node_parent[seq * MTAD_DRAFT_NODES + slot] = parent;
            ds.node_logq[seq * MTAD_DRAFT_NODES + slot] = lq;
            ds.tree_id[seq * MTAD_DRAFT_NODES + slot] = n;
            uint32_t* mk = ds.node_mask + ((size_t)seq * MTAD_DRAFT_NODES + slot) * MTAD_MASK_WORDS;
            for (int i = 0; i < MTAD_MASK_WORDS; ++i) {
                uint32_t w;
                if (parent >= 0) w = ds.node_mask[((size_t)seq * MTAD_DRAFT_NODES + parent) * MTAD_MASK_WORDS + i];
                else {                                        // child of the root: sees all pending rows
                    const int lo = i * 32;
                    w = P >= lo + 32 ? 0xffffffffu : (P > lo ? (1u << (P - lo)) - 1u : 0u);
                }
                if (((P + slot) >> 5) == i) w |= 1u << ((P + slot) & 31);
                mk[i] = w;
            }
        }
    }
    __syncthreads();
    if (step == gamma - 1 && tid == 0) {
        // x**: the final beam with the highest draft likelihood (lowest node id on ties), and its prefix likelihoods
        __threadfence_block();
        const int kept = s_count[1];
        int best = -1;
        for (int k = 0; k < kept; ++k) {
            const int sl = (gamma - 1) * beam + k;
            if (best < 0) { best = sl; continue; }
            const float a = ds.node_logq[seq * MTAD_DRAFT_NODES + sl], b0 = ds.node_logq[seq * MTAD_DRAFT_NODES + best];
            if (a > b0 || (a == b0 && ds.tree_id[seq * MTAD_DRAFT_NODES + sl] < ds.tree_id[seq * MTAD_DRAFT_NODES + best]))
                best = sl;
        }
        int cur = best;
        for (int i = gamma - 1; i >= 0 && cur >= 0; --i) {
            out.best_path[bi * gamma + i] = ds.tree_id[seq * MTAD_DRAFT_NODES + cur];
            out.logq_ref[bi * gamma + i] = ds.node_logq[seq * MTAD_DRAFT_NODES + cur];
            ds.best_path[seq * MTAD_MAX_DEPTH + i] = cur;
            cur = ds.node_parent[seq * MTAD_DRAFT_NODES + cur];
        }
        ds.gamma[seq] = gamma;
        ds.beam[seq] = beam;
        if (out.n_nodes) out.n_nodes[bi] = ds.n_tree[seq];
    }
}

cudaError_t launch_draft_select_warped(const ModelView& m, const DraftState& ds, const Scratch& sc, const SeqList& seqs,
                                       int B, int R, int step, int gamma, int beam, int keep_all, const float* uniforms,
                                       const DraftOut& out, cudaStream_t st) {
    draft_pick_warped_kernel<<<B, 256, 0, st>>>(sc.warp_row, m.d.vocab, R, step, gamma, beam, keep_all, uniforms, ds, seqs,
                                                out);
    return cudaGetLastError();
}

cudaError_t launch_draft_select(const ModelView& m, const DraftState& ds, const Scratch& sc, const SeqList& seqs, int B,
                                int R, int step, int gamma, int beam, int keep_all, const float* uniforms,
                                const DraftOut& out, bool pdl, cudaStream_t st) {
    const int V = m.d.vocab;
    int nch = (V + 1023) / 1024;
    nch = nch < 1 ? 1 : (nch > MTAD_DRAFT_CHUNKS ? MTAD_DRAFT_CHUNKS : nch);
    const int n_beams = step == 0 ? 1 : beam;
    const int kpb = (keep_all && step == 0) ? beam * beam : beam;
    cudaError_t e = launch_pdl(draft_scan_kernel, dim3(nch, n_beams, B), dim3(256), 0, st, pdl, (const float*)sc.logits,
                               V, R, step, gamma, beam, kpb, uniforms, ds, seqs, sc.draft_part, nch);
    if (e != cudaSuccess) return e;
    return launch_pdl(draft_pick_kernel, dim3(B), dim3(256), 0, st, pdl, (const float*)sc.logits, V, R, step, gamma,
                      beam, keep_all, kpb, ds, seqs, (const DraftPart*)sc.draft_part, nch, out);
}

// ---------------------------------------------------------------------------------------------------------------
// auxiliary cache roll-forward after a verification
// ---------------------------------------------------------------------------------------------------------------

// Beam slot of accepted node r of a verified draft.  mode 0: the verified chain was the draft's output sequence (chain
// node i = beam slot best_path[i]); mode 1: the verified tree was the draft's tree (node ids of that tree; a node that
// was recorded as a candidate only has no slot).  -1: no slot, -2: the path entry itself is out of range.
__device__ __forceinline__ int aux_slot_of(const DraftState& ds, const mtad_result& res, int bi, int seq, int D, int mode,
                                           int r) {
    const int pn = res.path[bi * D + r];
    if (pn < 0 || pn >= (mode == 0 ? MTAD_MAX_DEPTH : MTAD_DRAFT_NODES)) return -2;
    const int slot = mode == 0 ? ds.best_path[seq * MTAD_MAX_DEPTH + pn] : ds.tree2slot[seq * MTAD_DRAFT_NODES + pn];
    return slot >= MTAD_DRAFT_NODES ? -2 : (slot < 0 ? -1 : slot);
}

// Accepted nodes whose keys and values the draft left in the auxiliary cache: the leading ones that were beams of a
// layer before the last (the last layer, and candidates that were not kept, never ran).  At most one accepted token
// can follow them (such a node is a leaf of the tree).  Returns -1 when the path, the state or a cache row that the
// roll-forward would touch is out of range: accepted node r (r < kept) is read from slot base + beam slot and written
// to slot base + r, all inside [0, cap).
__device__ __forceinline__ int aux_kept_rows(const DraftState& ds, const mtad_result& res, int bi, int seq, int D, int mode,
                                             int eta, int base, long long cap) {
    const int gamma = ds.gamma[seq], beam = ds.beam[seq];
    if (gamma < 1 || gamma > MTAD_MAX_DEPTH || beam < 1 || beam > MTAD_MAX_BEAM || eta > D || base < 0) return -1;
    int kept = 0;
    for (; kept < eta; ++kept) {
        const int slot = aux_slot_of(ds, res, bi, seq, D, mode, kept);
        if (slot == -2) return -1;
        if (slot < 0 || slot >= (gamma - 1) * beam) break;
        if ((long long)base + slot >= cap) return -1;
    }
    if (eta - kept > 1 || kept > MTAD_MAX_DEPTH || (long long)base + kept > cap) return -1;
    return kept;
}

// Accepted node i (depth i + 1, slot base + beam slot) moves to position base + i when the draft ran it.
__global__ void aux_commit_kernel(__nv_bfloat16* __restrict__ cache, const int32_t* __restrict__ call_seq,
                                  DraftState ds, mtad_result res, int D, int mode, int max_batch, int Hkv, int hd,
                                  long long cap) {
    const int bi = blockIdx.y;
    if (res.status[bi] != 0) return;
    const int seq = call_seq[bi];
    if ((unsigned)seq >= (unsigned)max_batch) return;
    const int eta = res.eta[bi];
    if (eta <= 0) return;
    const int base = ds.base_len[seq] + ds.npend[seq];
    // every row read or written lies inside the cache, or nothing moves (aux_advance_kernel flags the sequence)
    const int kept = aux_kept_rows(ds, res, bi, seq, D, mode, eta, base, cap);
    if (kept <= 0) return;
    const int head = blockIdx.x % Hkv;
    const int kv = (blockIdx.x / Hkv) & 1;
    const int layer = blockIdx.x / (2 * Hkv);
    __nv_bfloat16* b = cache + idx_cache(layer, max_batch, seq, kv, Hkv, head, cap, 0, hd);
    extern __shared__ __nv_bfloat16 buf[];
    for (int i = threadIdx.x; i < kept * hd; i += blockDim.x) {
        const int r = i / hd, j = i % hd;
        const int node = aux_slot_of(ds, res, bi, seq, D, mode, r);
        buf[i] = b[(size_t)(base + node) * hd + j];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kept * hd; i += blockDim.x) {
        const int r = i / hd, j = i % hd;
        b[(size_t)(base + r) * hd + j] = buf[i];
    }
}

// New auxiliary state.  mode 0 / 1: after a draft (see above); mode 2: no draft produced the verified rows, the
// accepted tokens and the new root simply join the pending list (to be replayed by the next draft).
__global__ void aux_advance_kernel(SeqState s, DraftState ds, const int32_t* __restrict__ call_seq, mtad_result res,
                                   int D, int mode, int B, int max_batch, long long cap) {
    const int bi = blockIdx.x * blockDim.x + threadIdx.x;
    if (bi >= B || res.status[bi] != 0) return;
    const int seq = call_seq[bi];
    const int eta = res.eta[bi];
    if ((unsigned)seq >= (unsigned)max_batch || eta < 0 || eta > D) { atomicOr(&res.status[bi], MTAD_ST_RANGE); return; }
    int32_t* pend = s.aux_pend + seq * (MTAD_MAX_DEPTH + 1);
    const int bonus = res.out_tok[bi * (D + 1) + eta];
    if (mode == 2) {
        int np = s.aux_npend[seq];
        if (np + eta + 1 > MTAD_MAX_DEPTH + 1) { atomicOr(&res.status[bi], MTAD_ST_AUX_PENDING); return; }
        for (int i = 0; i <= eta; ++i) pend[np + i] = res.out_tok[bi * (D + 1) + i];
        s.aux_npend[seq] = np + eta + 1;
        return;
    }
    const int base = ds.base_len[seq] + ds.npend[seq];
    const int kept = aux_kept_rows(ds, res, bi, seq, D, mode, eta, base, cap);
    if (kept < 0) { atomicOr(&res.status[bi], MTAD_ST_RANGE); return; }
    s.aux_len[seq] = base + kept;
    int np = 0;
    if (eta > kept) pend[np++] = res.out_tok[bi * (D + 1) + eta - 1];   // accepted, but never run by the auxiliary model
    pend[np++] = bonus;
    s.aux_npend[seq] = np;
}

cudaError_t launch_aux_commit(const ModelView& aux, const SeqState& s, const DraftState& ds, int B,
                              const int32_t* call_seq_dev, const mtad_result& res, int max_depth, int mode,
                              cudaStream_t st) {
    if (mode != 2) {
        dim3 grid(aux.d.layers * 2 * aux.d.n_kv_heads, B);
        const size_t smem = (size_t)(max_depth > 0 ? max_depth : 1) * aux.d.head_dim * sizeof(__nv_bfloat16);
        aux_commit_kernel<<<grid, 128, smem, st>>>(static_cast<__nv_bfloat16*>(aux.d.kv_cache), call_seq_dev, ds, res,
                                                   max_depth, mode, aux.max_batch, aux.d.n_kv_heads, aux.d.head_dim,
                                                   (long long)aux.d.kv_capacity);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    aux_advance_kernel<<<1, 64, 0, st>>>(s, ds, call_seq_dev, res, max_depth, mode, B, aux.max_batch,
                                         (long long)aux.d.kv_capacity);
    return cudaGetLastError();
}

}  // namespace mtad
