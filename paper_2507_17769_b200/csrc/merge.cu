// Combine split-KV partial results.  For one query, attention over a union of
// disjoint key sets is the mix of the per-set results weighted by each set's
// exponential mass: with M = max_s lse_s,
//     out = sum_s e^{lse_s - M} o_s / sum_s e^{lse_s - M},  lse = M + log sum_s e^{lse_s - M}.
// Segments are combined in a fixed order, so the result is deterministic.
// Used for prefill q tile pairs cut into segments: a separate launch spreads the rows over all SMs (letting
// the last-arriving prefill CTA combine them instead was measured slower: one SM pulls the partial rows
// too slowly).  Decode rows are combined inside the decode kernel.
// One warp per output row.  The first partial rows are requested before the
// row's log-sum-exps have arrived (their addresses do not depend on them), the
// log-sum-exps are fetched one per lane, and the weights travel by shuffle, so a
// row costs about one round trip to L2 after its entry record.
#include <type_traits>

#include "common.cuh"

namespace ps {

namespace {

constexpr int kMergeWarps = 8;
constexpr int kMergeAhead = 4;  // partial rows in flight per warp

template <int D>
__global__ void __launch_bounds__(kMergeWarps * 32) merge_kernel(const MergeEntry* __restrict__ entries,
                                                                  const float* __restrict__ part_lse,
                                                                  const float* __restrict__ part_o,
                                                                  __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                                                                  int Hq, int G) {
    constexpr int V = D / 32;  // floats per lane
    using Vec = typename std::conditional<V == 4, float4, float2>::type;
    const MergeEntry e = entries[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = e.n_tok * G;
    const int rw = warp + kMergeWarps * blockIdx.y;
    if (rw >= rows) return;
    const int i = rw / G, hh = rw % G;
    const int64_t slot0 = (int64_t)e.base + (int64_t)i * G + hh;
    const int n_seg = e.n_seg;
    auto row_ptr = [&](int s) { return reinterpret_cast<const Vec*>(part_o + (slot0 + (int64_t)s * e.seg_stride) * D) + lane; };

    Vec x[kMergeAhead];
#pragma unroll
    for (int k = 0; k < kMergeAhead; ++k)
        if (k < n_seg) x[k] = *row_ptr(k);
    // a segment that saw no visible key for this row carries lse = -inf and weight 0
    const float lse_mine = lane < n_seg ? part_lse[slot0 + (int64_t)lane * e.seg_stride] : -INFINITY;  // segments 0..31
    float M = lse_mine;
    for (int s = lane + 32; s < n_seg; s += 32) M = fmaxf(M, part_lse[slot0 + (int64_t)s * e.seg_stride]);
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, k));
    const float w_mine = __expf(lse_mine - M);  // exp(-inf) = 0
    float denom = w_mine;
    for (int s = lane + 32; s < n_seg; s += 32) denom += __expf(part_lse[slot0 + (int64_t)s * e.seg_stride] - M);
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, k);

    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.f;
    // segments in a fixed order, kMergeAhead rows at a time
    for (int s0 = 0; s0 < n_seg; s0 += kMergeAhead) {
        if (s0 > 0) {
#pragma unroll
            for (int k = 0; k < kMergeAhead; ++k)
                if (s0 + k < n_seg) x[k] = *row_ptr(s0 + k);
        }
#pragma unroll
        for (int k = 0; k < kMergeAhead; ++k) {
            const int s = s0 + k;
            if (s < n_seg) {  // warp-uniform
                const float w = s < 32 ? __shfl_sync(0xffffffffu, w_mine, s)
                                       : __expf(part_lse[slot0 + (int64_t)s * e.seg_stride] - M);
                if constexpr (V == 4) {
                    acc[0] += w * x[k].x; acc[1] += w * x[k].y; acc[2] += w * x[k].z; acc[3] += w * x[k].w;
                } else {
                    acc[0] += w * x[k].x; acc[1] += w * x[k].y;
                }
            }
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

}  // namespace

ps_status launch_merge(const RunArgs& a) {
    if (a.w.n_merge == 0) return PS_OK;
    const int Hq = a.shape.n_q_heads, G = Hq / a.shape.n_kv_heads;
    // blockIdx.x = merge entry (a prefill item cut into segments, up to 256 rows); blockIdx.y = its rows, one per warp
    const dim3 grid(a.w.n_merge, kPrefillRowsPerItem / kMergeWarps);
    if (a.shape.head_dim == 128)
        merge_kernel<128><<<grid, kMergeWarps * 32, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    else
        merge_kernel<64><<<grid, kMergeWarps * 32, 0, a.stream>>>(a.w.merge, a.w.part_lse, a.w.part_o, a.out, a.lse, Hq, G);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

}  // namespace ps
