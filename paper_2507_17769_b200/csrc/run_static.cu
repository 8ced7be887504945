// ps_attn_run_static: the per-iteration attention call for callers that must
// not allocate device memory.  The scratch that ps_attn_run takes from its
// caller (the uploaded work list plus the split-KV partial results that the
// decode / prefill kernels write and the merge kernel reads) lives here in one
// fixed array inside the library's device image.
#include <mutex>

#include "common.cuh"

namespace ps {
size_t plan_workspace_bytes(const ps_plan* pl);
}

namespace {

constexpr size_t kStaticScratchBytes = size_t(PS_STATIC_WORKSPACE_BYTES);
constexpr int kMaxDevices = 64;

// One copy per GPU that loads the library, resident until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not an
// address a kernel can use; the device address is looked up once per device.
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

}  // namespace

extern "C" ps_status ps_attn_run_static(ps_plan* plan, const ps_kv* kv, const void* q_dev, const int32_t* block_table_dev,
                                        void* out_dev, float* lse_out_dev, void* stream) {
    using namespace ps;
    if (!plan || !kv || !q_dev || !block_table_dev || !out_dev) return fail(PS_ERR_INVALID, "null argument");
    const size_t need = plan_workspace_bytes(plan);
    if (need > kStaticScratchBytes)
        return fail(PS_ERR_WORKSPACE,
                    "this plan needs %zu bytes of scratch but the built-in scratch holds %zu; use ps_attn_run with a "
                    "caller-provided workspace, or plan smaller batches",
                    need, kStaticScratchBytes);
    int dev = -1;
    PS_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(PS_ERR_UNSUPPORTED, "device ordinal %d is outside [0, %d)", dev, kMaxDevices);
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            PS_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    // The work-list upload at the head of the run rewrites the header (status word and
    // work counters start at zero); the partial rows are fully written before they are read.
    return ps_attn_run(plan, kv, q_dev, block_table_dev, out_dev, lse_out_dev, scratch, kStaticScratchBytes, stream);
}
