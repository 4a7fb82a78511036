// mtad_verify_chain_static: the chain verification step for callers that cannot allocate device memory.
// All scratch of the step lives in one file-scope device array of fixed size instead of a caller workspace.
#include <mutex>

#include "common.cuh"

// Scratch for the no-allocation entry point.  Every GPU that loads this library holds these bytes until the
// process exits.  All calls share the array and it keeps whatever the previous call left in it.
static __device__ __align__(256) unsigned char g_static_scratch[MTAD_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;

struct PerDevice {
    void* scratch = nullptr;        // device address of g_static_scratch on this device
    mtad_ctx* ctx = nullptr;        // context carved out of the array for the last descriptor seen
    mtad_model_desc desc{};         // that descriptor (pointers included)
    std::vector<const void*> lw;    // and its layer pointer table
    int max_nodes = -1;
};

PerDevice g_dev[kMaxDevices];
std::mutex g_mu;

bool same_model(const PerDevice& p, const mtad_model_desc* m, int gamma) {
    if (!p.ctx || p.max_nodes != gamma) return false;
    const mtad_model_desc& a = p.desc;
    if (a.layers != m->layers || a.d_model != m->d_model || a.n_q_heads != m->n_q_heads ||
        a.n_kv_heads != m->n_kv_heads || a.head_dim != m->head_dim || a.d_ffn != m->d_ffn || a.vocab != m->vocab ||
        a.rope_base != m->rope_base || a.rms_eps != m->rms_eps || a.embed != m->embed || a.lm_head != m->lm_head ||
        a.final_norm != m->final_norm || a.kv_cache != m->kv_cache || a.kv_capacity != m->kv_capacity)
        return false;
    for (size_t i = 0; i < p.lw.size(); ++i)
        if (p.lw[i] != m->layer_weights[i]) return false;
    return true;
}

}  // namespace

extern "C" int mtad_verify_chain_static(const mtad_model_desc* target, int32_t kv_len, int32_t root_token, int gamma,
                                        const int32_t* draft_tok, const float* draft_logq, float log_tau,
                                        const float* bonus_uniform, const mtad_result* out, void* stream) {
    if (!target || !target->layer_weights || gamma < 0) return MTAD_E_INVALID;
    size_t need = 0;
    int rc = mtad_workspace_bytes(target, nullptr, 1, gamma, &need);
    if (rc != MTAD_OK) return rc;
    if (need > (size_t)MTAD_STATIC_SCRATCH_BYTES) return MTAD_E_WORKSPACE;   // model or chain too large for the array

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MTAD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    PerDevice& p = g_dev[dev];
    if (!p.scratch) {
        // Host code cannot use &g_static_scratch as a device pointer: ask the runtime for the array's address on
        // the current device, once.
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MTAD_E_CUDA;
        p.scratch = ptr;
    }
    if (!same_model(p, target, gamma)) {
        // The array is about to be laid out afresh and zeroed: work of earlier calls that still runs on the caller's
        // stream (a non-blocking stream does not wait for the zeroing on the default stream) must be over first.
        if (cudaDeviceSynchronize() != cudaSuccess) return MTAD_E_CUDA;
        if (p.ctx) { mtad_destroy(p.ctx); p.ctx = nullptr; }
        // mtad_create lays the step's scratch out inside the array and zeroes it (the array still holds the
        // previous caller's data); it allocates no device memory itself.
        rc = mtad_create(target, nullptr, 1, gamma, p.scratch, MTAD_STATIC_SCRATCH_BYTES, &p.ctx);
        if (rc != MTAD_OK) { p.ctx = nullptr; return rc; }
        p.desc = *target;
        p.lw.assign(target->layer_weights, target->layer_weights + (size_t)target->layers * MTAD_LAYER_TENSORS);
        p.max_nodes = gamma;
    }
    rc = mtad_seq_set(p.ctx, 0, kv_len, root_token, kv_len, nullptr, stream);
    if (rc != MTAD_OK) return rc;
    const int32_t seq0 = 0;
    return mtad_verify_chain(p.ctx, 1, &seq0, gamma, draft_tok, draft_logq, log_tau, bonus_uniform, out, stream);
}
