// Combine split-KV partial results.  For one query, attention over a union of
// disjoint key sets is the mix of the per-set results weighted by each set's
// exponential mass: with M = max_s lse_s,
//     out = sum_s e^{lse_s - M} o_s / sum_s e^{lse_s - M},  lse = M + log sum_s e^{lse_s - M}.
// Segments are combined in a fixed order, so the result is deterministic.
#include "common.cuh"

namespace ps {

namespace {

template <int D>
__global__ void __launch_bounds__(128) merge_kernel(const MergeEntry* __restrict__ entries, const float* __restrict__ part_lse,
                                                    const float* __restrict__ part_o, __nv_bfloat16* __restrict__ out,
                                                    float* __restrict__ lse, int Hq, int G) {
    constexpr int V = D / 32;  // floats per lane
    const MergeEntry e = entries[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = e.n_tok * G;
    for (int rw = warp + 4 * blockIdx.y; rw < rows; rw += 4 * gridDim.y) {
        const int i = rw / G, hh = rw % G;
        const int64_t slot0 = (int64_t)e.base + (int64_t)i * G + hh;
        float M = -INFINITY;
        for (int s = lane; s < e.n_seg; s += 32) M = fmaxf(M, part_lse[slot0 + (int64_t)s * e.seg_stride]);
#pragma unroll
        for (int k = 16; k >= 1; k >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, k));
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        float denom = 0.f;
        for (int s = 0; s < e.n_seg; ++s) {
            const int64_t slot = slot0 + (int64_t)s * e.seg_stride;
            const float ls = part_lse[slot];
            if (ls == -INFINITY) continue;  // segment saw no visible key for this row
            const float w = __expf(ls - M);
            denom += w;
            const float* po = part_o + slot * D + lane * V;
#pragma unroll
            for (int v = 0; v < V; ++v) acc[v] += w * po[v];
        }
        const float inv = 1.f / denom;
        const int64_t orow = (int64_t)(e.q_tok + i) * Hq + e.kv_head * G + hh;
        __nv_bfloat16* op = out + orow * D + lane * V;
#pragma unroll
        for (int v = 0; v < V; v += 2)
            *reinterpret_cast<__nv_bfloat162*>(op + v) = __floats2bfloat162_rn(acc[v] * inv, acc[v + 1] * inv);
        if (lse && lane == 0) lse[orow] = M + __logf(denom);
    }
}

}  // namespace

ps_status launch_merge(const RunArgs& a) {
    if (a.w.n_merge == 0) return PS_OK;
    const int Hq = a.shape.n_q_heads, G = Hq / a.shape.n_kv_heads;
    // blockIdx.x = merge entry; blockIdx.y spreads an entry's rows (up to 256 for a prefill item) over blocks
    const dim3 grid(a.w.n_merge, a.w.n_prefill > 0 ? 16 : 1);
    if (a.shape.head_dim == 128)
        merge_kernel<128><<<grid, 128, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    else
        merge_kernel<64><<<grid, 128, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

}  // namespace ps
