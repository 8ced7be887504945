// Combine split-KV partial results.  For one query, attention over a union of
// disjoint key sets is the mix of the per-set results weighted by each set's
// exponential mass: with M = max_s lse_s,
//     out = sum_s e^{lse_s - M} o_s / sum_s e^{lse_s - M},  lse = M + log sum_s e^{lse_s - M}.
// Segments are combined in a fixed order, so the result is deterministic.
// Used for prefill q tile pairs cut into segments: a separate launch spreads the rows over all SMs (letting
// the last-arriving prefill CTA combine them instead was measured slower: one SM pulls the partial rows
// too slowly).  Decode rows are combined inside the decode kernel.
// One warp per output row: the lanes first fetch the row's log-sum-exps in
// parallel (max and sum by shuffles), then stream the partial rows with several
// loads in flight.
#include "common.cuh"

namespace ps {

namespace {

constexpr int kMergeWarps = 4;

template <int D>
__global__ void __launch_bounds__(kMergeWarps * 32) merge_kernel(const MergeEntry* __restrict__ entries,
                                                                  const float* __restrict__ part_lse,
                                                                  const float* __restrict__ part_o,
                                                                  __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                                                  int Hq, int G) {
    constexpr int V = D / 32;  // floats per lane
    const MergeEntry e = entries[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = e.n_tok * G;
    for (int rw = warp + kMergeWarps * blockIdx.y; rw < rows; rw += kMergeWarps * gridDim.y) {
        const int i = rw / G, hh = rw % G;
        const int64_t slot0 = (int64_t)e.base + (int64_t)i * G + hh;
        // a segment that saw no visible key for this row carries lse = -inf and weight 0
        float M = -INFINITY;
        for (int s = lane; s < e.n_seg; s += 32) M = fmaxf(M, part_lse[slot0 + (int64_t)s * e.seg_stride]);
#pragma unroll
        for (int k = 16; k >= 1; k >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, k));
        float denom = 0.f;
        for (int s = lane; s < e.n_seg; s += 32) denom += __expf(part_lse[slot0 + (int64_t)s * e.seg_stride] - M);
#pragma unroll
        for (int k = 16; k >= 1; k >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, k);
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
#pragma unroll 4
        for (int s = 0; s < e.n_seg; ++s) {
            const int64_t slot = slot0 + (int64_t)s * e.seg_stride;
            const float w = __expf(part_lse[slot] - M);  // exp(-inf) = 0
            const float* po = part_o + slot * D + lane * V;
            if constexpr (V == 4) {
                const float4 x = *reinterpret_cast<const float4*>(po);
                acc[0] += w * x.x; acc[1] += w * x.y; acc[2] += w * x.z; acc[3] += w * x.w;
            } else {
                const float2 x = *reinterpret_cast<const float2*>(po);
                acc[0] += w * x.x; acc[1] += w * x.y;
            }
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
    // blockIdx.x = merge entry (a prefill item cut into segments, up to 256 rows); blockIdx.y spreads its rows
    const dim3 grid(a.w.n_merge, kPrefillRowsPerItem / kMergeWarps / 2);
    if (a.shape.head_dim == 128)
        merge_kernel<128><<<grid, kMergeWarps * 32, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    else
        merge_kernel<64><<<grid, kMergeWarps * 32, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

}  // namespace ps
