// Decode attention over the paged KV cache (rows with one new token).
//
// Decode attention streams every cached K and V of a request once and cannot
// share those loads across requests (paper section 2.2), so it is bound by HBM
// bandwidth.  Design for that bound:
//   * each warp is an independent streaming engine with its own ring of
//     shared-memory stages; one lane issues one bulk async copy per
//     (page, kv head) block (K and V of 16 tokens, contiguous in the pool) and
//     the warp waits on that stage's mbarrier -- no CTA-wide barrier anywhere;
//   * the q heads that share a kv head ride in the N = 8 columns of
//     mma.m16n8k16: S^T[16 tokens x heads] = K[16 x d] Q^T, then
//     O^T[d x heads] += V^T[d x 16 tokens] P^T, so K and V are read from shared
//     memory exactly once per group and no tensor-core row is padding at G = 8;
//   * the softmax is over the token (row) axis of the accumulator fragment:
//     two in-thread values plus three shuffles per head column;
//   * P^T goes from accumulator layout to B-operand layout with movmatrix;
//   * work arrives as equal-sized units of consecutive pages (possibly
//     spanning several (request, kv head) pieces) fetched from one atomic
//     counter; the producer side of the warp runs STAGES pages ahead of the
//     consumer side, across piece and unit boundaries.
#include <type_traits>

#include "common.cuh"

namespace ps {

namespace {

// streaming warps per CTA (one CTA per SM) and ring depth per warp: 12 x 2 x 8 KB = 192 KB in flight per SM;
// measured on B200: 12 x 2 and 10 x 2 beat 8 x 3, 6 x 4 and 4 x 6 by 2-6 %
constexpr int kWarps = 12;
constexpr int kStagesPerWarp = 2;
constexpr int kRing = 8;  // unit ids in flight between the producer and consumer cursors of a warp
constexpr int kDeferred = 8;  // merges a warp can postpone until its KV stream has drained

// FP8 = the E4M3 cache variant: a (page, kv head) block is K codes, V codes (one byte per element, rows of D bytes
// with the same 16-byte-unit swizzle), then the 16 tokens' K scales and V scales (fp32).
template <int D, bool FP8>
struct DecodeCfg {
    static constexpr int kBlockBytes = FP8 ? kPage * D : kPage * D * 2;                  // K (or V) of one page, one kv head
    static constexpr int kStageBytes = FP8 ? (int)fp8_page_head_bytes(D) : 2 * kBlockBytes;  // K then V (then the scales)
    // 8 KB (4 KB at D = 64) stages per warp; the FP8 blocks are half as large, so twice as many are kept in flight
    static constexpr int kStages = (FP8 ? 2 : 1) * ((D == 128) ? kStagesPerWarp : 2 * kStagesPerWarp);
    static constexpr int kSmemBytes =
        kWarps * kStages * kStageBytes + kWarps * kStages * 8 + kWarps * kRing * 4 + kWarps * kDeferred * 12 + 1024;
};

// The FP8 variant feeds the warp MMA with f16 operands: an E4M3 code converts to f16 exactly in one instruction
// (every E4M3 value, subnormals included, is a normal f16 or zero), where a conversion to bf16 would cost the ALU
// pipe four -- and with them the kernel its memory-bound rate.  Q (bf16) is converted once per row, clamped to the
// f16 range; a softmax weight times its key's V scale is carried as f16 after a multiplication by 2^8 (taken back
// out with the row sum), which keeps weights down to 2^-22 / scale out of f16's subnormals.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes) {
    uint32_t h;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h) : "h"((unsigned short)two_codes));
    return h;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t h;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h) : "f"(fminf(fmaxf(hi, -65504.f), 65504.f)), "f"(fminf(fmaxf(lo, -65504.f), 65504.f)));
    return h;
}
// D(16x8, fp32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_16816_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
constexpr float kWeightScale = 256.f;  // 2^8, see above

struct DecodeParams {
    const char* pool;
    int64_t num_pages;
    const __nv_bfloat16* q;
    const int32_t* block_table;
    int32_t max_pages;
    __nv_bfloat16* out;
    float* lse;
    WsHeader* hdr;
    const DecodePiece* pieces;
    const DecodeUnit* units;
    int32_t n_units;
    const DecodeMerge* dmerge;
    int32_t* dmerge_cnt;
    float* part_lse;
    float* part_o;
    int32_t Hq, Hkv, G;
    float scale_log2;  // log2(e) / sqrt(d)
    int32_t n_req, total_q, n_dmerge;  // extents the work records are checked against
    int64_t n_part_slots;
    int64_t wait_limit_ns;
};

// A work record that points outside the batch (it can only come from a damaged work list) is replaced by one that
// stays inside it, and the run is flagged: both cursors of a warp apply the same rule to the same record, so they
// keep agreeing on how many pages it stands for.
__device__ __forceinline__ bool piece_pages_ok(const int4& a, const DecodeParams& p) {
    return (uint32_t)a.x < (uint32_t)p.n_req && (uint32_t)a.y < (uint32_t)p.Hkv && a.z >= 0 && a.z < a.w && a.w <= p.max_pages;
}

template <int D, bool FP8>
__global__ void __launch_bounds__(kWarps * 32, 1) decode_kernel(const DecodeParams p) {
    using Cfg = DecodeCfg<D, FP8>;
    constexpr int STAGES = Cfg::kStages;
    constexpr int KS = D / 16;  // k-steps of QK^T == m-tiles of PV

    extern __shared__ char smem_raw[];
    char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    char* my_stages = smem + (size_t)warp * STAGES * Cfg::kStageBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kWarps * STAGES * Cfg::kStageBytes) + warp * STAGES;
    int32_t* ring = reinterpret_cast<int32_t*>(smem + (size_t)kWarps * STAGES * Cfg::kStageBytes + kWarps * STAGES * 8) +
                    warp * kRing;
    int32_t* deferred = reinterpret_cast<int32_t*>(smem + (size_t)kWarps * STAGES * Cfg::kStageBytes + kWarps * STAGES * 8 +
                                                   kWarps * kRing * 4) + warp * kDeferred * 3;
    const uint32_t stage0 = smem_u32(my_stages);
    const uint32_t bar0 = smem_u32(bars);

    if (lane == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
        mbar_fence_init();
    }
    __syncwarp();

    // K/V pages are read once: marked first to go in L2, they leave the partial rows, Q and the work list resident
    // (measured: 100.9 -> 96.9 us on the 64-sequence decode batch, 465.6 -> 452.7 us on 512 sequences)
    const uint64_t kv_policy = l2_policy_evict_first();
    // ---- producer cursor (warp-uniform) ----
    bool P_done = false;
    int P_piece = 0, P_piece_end = 0, P_page = 0, P_page_end = 0, P_g = 0, P_bt0 = 0, P_bt = 0;
    const int32_t* P_row = p.block_table;
    uint32_t n_prod = 0, pseq = 0;

    auto produce = [&]() {
        while (!P_done && P_page >= P_page_end) {
            if (++P_piece >= P_piece_end) {
                // a warp's first unit is its own index (no round trip); later ones come from the shared counter
                int u = blockIdx.x * kWarps + warp;
                if (pseq > 0) {
                    if (lane == 0) u = atomicAdd(&p.hdr->decode_next, 1) + gridDim.x * kWarps;
                    u = __shfl_sync(0xffffffffu, u, 0);
                }
                if (lane == 0) ring[pseq % kRing] = u;
                ++pseq;
                if (u >= p.n_units) { P_done = true; break; }
                const DecodeUnit du = p.units[u];
                P_piece = du.piece_begin;
                P_piece_end = du.piece_end;
            }
            int4 a = __ldg(reinterpret_cast<const int4*>(&p.pieces[P_piece]));
            if (!piece_pages_ok(a, p)) a = make_int4(0, 0, 0, 1);  // flagged by the consumer side
            P_page = a.z;
            P_page_end = a.w;
            P_g = a.y;
            P_row = p.block_table + (int64_t)a.x * p.max_pages;
            P_bt0 = P_page;
            P_bt = (P_bt0 + lane < P_page_end) ? __ldg(P_row + P_bt0 + lane) : 0;
        }
        if (P_done) return;
        if (P_page >= P_bt0 + 32) {
            P_bt0 += 32;
            P_bt = (P_bt0 + lane < P_page_end) ? __ldg(P_row + P_bt0 + lane) : 0;
        }
        const int page = __shfl_sync(0xffffffffu, P_bt, P_page - P_bt0);
        const uint32_t stage = n_prod % STAGES;
        if (lane == 0) {
            const uint32_t bar = bar0 + 8 * stage;
            if ((uint32_t)page < (uint64_t)p.num_pages) {
                mbar_expect_tx(bar, Cfg::kStageBytes);
                bulk_g2s_hint(stage0 + stage * Cfg::kStageBytes,
                              p.pool + ((int64_t)page * p.Hkv + P_g) * (int64_t)Cfg::kStageBytes, Cfg::kStageBytes, bar, kv_policy);
            } else {
                atomicOr(&p.hdr->status, kStatusBounds);
                mbar_arrive(bar);  // complete the phase without data; the run is flagged invalid
            }
        }
        ++P_page;
        ++n_prod;
    };

    for (int s = 0; s < STAGES; ++s) produce();

    // ---- consumer cursor ----
    int C_piece = 0, C_piece_end = 0, C_page = 0, C_page_end = 0;
    int C_qtok = 0, C_slot = -1, C_kvlen = 0, C_g = 0, C_midx = 0;
    bool have_piece = false, timed_out = false;
    uint32_t n_cons = 0, cseq = 0;

    uint32_t qb[KS][2];
    float o[KS][4];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    const int col = 2 * (lane & 3);  // this thread's head columns: col, col + 1
    const int row = lane >> 2;       // token rows row, row + 8 of S^T; d rows of O^T
    const int mi = lane >> 3, l7 = lane & 7;
    // ldmatrix row addresses (byte offsets inside a block, before the per-step unit term)
    const uint32_t k_tok_off = (uint32_t)(((mi & 1) * 8 + l7) * 128);
    const uint32_t v_tok_off = (uint32_t)(((mi >> 1) * 8 + l7) * 128);

    // Combine the partials of merge record midx (output token qtok, kv head g), in segment order.
    int n_deferred = 0;
    auto combine = [&](int midx, int qtok, int g) {
        __syncwarp();  // lane 0's acquiring increment is ordered before every lane's partial loads
        const DecodeMerge dm = p.dmerge[midx];
        // The n_seg * G log-sum-exps are contiguous (segment-major, head-minor).  Lane i reads entries
        // i, i + 32, ...; since G divides 32 they all belong to head i % G, so the per-head max and
        // sum are reductions over the lanes that are congruent mod G.
        const int n = dm.n_seg * p.G;
        const float* lse_in = p.part_lse + dm.base;
        float mx = -INFINITY;
        for (int i = lane; i < n; i += 32) mx = fmaxf(mx, __ldcg(lse_in + i));
        for (int off = p.G; off < 32; off <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float den = 0.f;
        for (int i = lane; i < n; i += 32) den += __expf(__ldcg(lse_in + i) - mx);
        for (int off = p.G; off < 32; off <<= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
        // All heads at once: lane -> (head hh, slice of d); a lane owns D * G / 32 consecutive floats
        // of its head's row, so every segment costs it a few independent 16-byte loads.
        const int lanes_per_head = 32 / p.G;
        const int hh = lane / lanes_per_head, part = lane % lanes_per_head;
        const float M = __shfl_sync(0xffffffffu, mx, hh);
        const float inv = 1.f / __shfl_sync(0xffffffffu, den, hh);
        const int64_t orow = (int64_t)qtok * p.Hq + g * p.G + hh;
        auto run = [&](auto nvec_tag) {
            constexpr int NV = decltype(nvec_tag)::value;  // float4 per lane
            float4 acc[NV];
#pragma unroll
            for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
            // fixed segment order; kAhead segments' rows are requested before the first is used, so that a long
            // list of segments costs about one trip to L2 per kAhead of them
            constexpr int kAhead = NV <= 2 ? 8 : NV <= 4 ? 4 : 2;  // at most 16 float4 in flight per lane
            for (int s0 = 0; s0 < dm.n_seg; s0 += kAhead) {
                float4 x[kAhead][NV];
                float lw[kAhead];
#pragma unroll
                for (int k = 0; k < kAhead; ++k) {
                    const int sk = min(s0 + k, dm.n_seg - 1);  // past the end: a repeat that is not accumulated
                    const int64_t slot = (int64_t)dm.base + sk * p.G + hh;
                    lw[k] = __ldcg(p.part_lse + slot);
                    const float4* po = reinterpret_cast<const float4*>(p.part_o + slot * D) + part * NV;
#pragma unroll
                    for (int v = 0; v < NV; ++v) x[k][v] = __ldcg(po + v);
                }
#pragma unroll
                for (int k = 0; k < kAhead; ++k) {
                    if (s0 + k < dm.n_seg) {  // warp-uniform
                        const float w = __expf(lw[k] - M);
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            acc[v].x += w * x[k][v].x; acc[v].y += w * x[k][v].y; acc[v].z += w * x[k][v].z; acc[v].w += w * x[k][v].w;
                        }
                    }
                }
            }
            uint2* op = reinterpret_cast<uint2*>(p.out + orow * D) + part * NV;
#pragma unroll
            for (int v = 0; v < NV; ++v)
                op[v] = make_uint2(pack_bf16(acc[v].x * inv, acc[v].y * inv), pack_bf16(acc[v].z * inv, acc[v].w * inv));
        };
        // NV = D * G / 128: one float4 at (D, G) = (64, 2) or (128, 1) up to eight at (128, 8)
        switch (D * p.G / 128) {
            case 8: run(std::integral_constant<int, 8>{}); break;
            case 4: run(std::integral_constant<int, 4>{}); break;
            case 2: run(std::integral_constant<int, 2>{}); break;
            case 1: run(std::integral_constant<int, 1>{}); break;
            default: {  // D = 64, G = 1: half a float4 per lane -- let the first 16 lanes take one each
                if (lane < 16) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int s = 0; s < dm.n_seg; ++s) {
                        const int64_t slot = (int64_t)dm.base + s;
                        const float w = __expf(__ldcg(p.part_lse + slot) - __shfl_sync(0xffffu, mx, 0));
                        const float4 x = __ldcg(reinterpret_cast<const float4*>(p.part_o + slot * D) + lane);
                        acc.x += w * x.x; acc.y += w * x.y; acc.z += w * x.z; acc.w += w * x.w;
                    }
                    const float inv1 = 1.f / __shfl_sync(0xffffu, den, 0);
                    reinterpret_cast<uint2*>(p.out + ((int64_t)qtok * p.Hq + g) * D)[lane] =
                        make_uint2(pack_bf16(acc.x * inv1, acc.y * inv1), pack_bf16(acc.z * inv1, acc.w * inv1));
                }
            }
        }
        if (p.lse && part == 0 && hh < p.G) p.lse[orow] = M + __logf(1.f / inv);
    };

    auto finalize = [&]() {
        // column sums over the 8 row-groups of the fragment
        l0 += __shfl_xor_sync(0xffffffffu, l0, 4);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 4);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 8);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 8);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 16);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 16);
        // (FP8: the accumulators hold the outputs times kWeightScale)
        const float inv0 = (FP8 ? 1.f / kWeightScale : 1.f) / l0, inv1 = (FP8 ? 1.f / kWeightScale : 1.f) / l1;
        const float lse0 = (m0 + log2f(l0)) * 0.6931471805599453f;
        const float lse1 = (m1 + log2f(l1)) * 0.6931471805599453f;
        const int h_base = C_g * p.G;
        // accumulator rows `row` and `row + 8` of m-tile mt hold d = 16 mt + row and + 8 -- in the FP8 variant, whose
        // transposed V fragments pair neighbouring bytes, d = 16 mt + 2 row and the next one
        constexpr int kRowStep = FP8 ? 2 : 1, kPairStep = FP8 ? 1 : 8;
        if (C_slot < 0) {
            __nv_bfloat16* o0 = p.out + ((int64_t)C_qtok * p.Hq + h_base + col) * D;
            __nv_bfloat16* o1 = o0 + D;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                const int dd = mt * 16 + kRowStep * row;
                if (col < p.G) {
                    o0[dd] = __float2bfloat16_rn(o[mt][0] * inv0);
                    o0[dd + kPairStep] = __float2bfloat16_rn(o[mt][2] * inv0);
                }
                if (col + 1 < p.G) {
                    o1[dd] = __float2bfloat16_rn(o[mt][1] * inv1);
                    o1[dd + kPairStep] = __float2bfloat16_rn(o[mt][3] * inv1);
                }
            }
            if (p.lse && row == 0) {
                if (col < p.G) p.lse[(int64_t)C_qtok * p.Hq + h_base + col] = lse0;
                if (col + 1 < p.G) p.lse[(int64_t)C_qtok * p.Hq + h_base + col + 1] = lse1;
            }
        } else {
            float* o0 = p.part_o + ((int64_t)C_slot + col) * D;
            float* o1 = o0 + D;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                const int dd = mt * 16 + kRowStep * row;
                if (col < p.G) {
                    o0[dd] = o[mt][0] * inv0;
                    o0[dd + kPairStep] = o[mt][2] * inv0;
                }
                if (col + 1 < p.G) {
                    o1[dd] = o[mt][1] * inv1;
                    o1[dd + kPairStep] = o[mt][3] * inv1;
                }
            }
            if (row == 0) {
                if (col < p.G) p.part_lse[C_slot + col] = lse0;
                if (col + 1 < p.G) p.part_lse[C_slot + col + 1] = lse1;
            }
            // The warp that delivers the last piece of a (request, kv head) combines all of its
            // partials, always in segment order, so the result does not depend on which warp that is.
            // Release: the warp barrier orders every lane's partial stores before lane 0's
            // acq_rel increment, which the combining warp's increment (acquire) observes.
            __syncwarp();
            int arrived = 0;
            const DecodeMerge dm = p.dmerge[C_midx];
            if (lane == 0)
                asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;"
                             : "=r"(arrived) : "l"(p.dmerge_cnt + C_midx) : "memory");
            arrived = __shfl_sync(0xffffffffu, arrived, 0);
            if (arrived == dm.n_seg - 1) {
                // Combining now would stall this warp's KV stream on dependent L2 reads; queue it
                // for after the stream has drained (done at once only if the queue is full).
                if (n_deferred < kDeferred) {
                    if (lane == 0) {
                        deferred[3 * n_deferred + 0] = C_midx;
                        deferred[3 * n_deferred + 1] = C_qtok;
                        deferred[3 * n_deferred + 2] = C_g;
                    }
                    ++n_deferred;
                } else {
                    combine(C_midx, C_qtok, C_g);
                }
            }
        }
    };

    while (true) {
        if (C_page >= C_page_end) {
            if (have_piece) finalize();
            have_piece = false;
            if (++C_piece >= C_piece_end) {
                __syncwarp();
                const int u = ring[cseq % kRing];
                ++cseq;
                if (u >= p.n_units) break;
                const DecodeUnit du = p.units[u];
                C_piece = du.piece_begin;
                C_piece_end = du.piece_end;
            }
            int4 a = __ldg(reinterpret_cast<const int4*>(&p.pieces[C_piece]));
            int4 b = __ldg(reinterpret_cast<const int4*>(&p.pieces[C_piece]) + 1);
            {
                bool bad = false;
                if (!piece_pages_ok(a, p)) {
                    a = make_int4(0, 0, 0, 1);
                    bad = true;
                }
                if ((uint32_t)b.x >= (uint32_t)p.total_q) {
                    b.x = 0;
                    bad = true;
                }
                if (b.y >= 0 && ((int64_t)b.y + p.G > p.n_part_slots || (uint32_t)b.w >= (uint32_t)p.n_dmerge)) {
                    b.y = -1;
                    bad = true;
                }
                if (b.z <= (a.w - 1) * kPage) {  // the row's keys end inside the piece's last page or behind it
                    b.z = a.w * kPage;
                    bad = true;
                }
                if (bad && lane == 0) atomicOr(&p.hdr->status, kStatusBounds);
            }
            C_g = a.y;
            C_page = a.z;
            C_page_end = a.w;
            C_qtok = b.x;
            C_slot = b.y;
            C_kvlen = b.z;
            C_midx = b.w;
            have_piece = true;
            // Q^T as B fragments: thread holds head (lane / 4), d = 16 ks + 2 (lane % 4) + {0, 1} (+ 8)
            const int hh = lane >> 2;
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + ((int64_t)C_qtok * p.Hq + C_g * p.G + hh) * D);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                if constexpr (FP8) {  // k-step ks covers d = 16 ks + 4 (lane % 4) + {0, 1 | 2, 3}: the order of the K bytes a thread gets
                    const uint32_t w0 = hh < p.G ? __ldg(qrow + ks * 8 + 2 * (lane & 3)) : 0u;
                    const uint32_t w1 = hh < p.G ? __ldg(qrow + ks * 8 + 2 * (lane & 3) + 1) : 0u;
                    qb[ks][0] = pack_f16(bf16_lo(w0), bf16_hi(w0));
                    qb[ks][1] = pack_f16(bf16_lo(w1), bf16_hi(w1));
                } else {
                    qb[ks][0] = hh < p.G ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
                    qb[ks][1] = hh < p.G ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
                }
            }
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
            m0 = m1 = -INFINITY;
            l0 = l1 = 0.f;
        }

        const uint32_t stage = n_cons % STAGES;
        if (!mbar_wait(bar0 + 8 * stage, (n_cons / STAGES) & 1, p.wait_limit_ns)) {
            if (lane == 0) atomicOr(&p.hdr->status, kStatusTimeout);
            timed_out = true;
            break;
        }
        const uint32_t kbase = stage0 + stage * Cfg::kStageBytes;
        const uint32_t vbase = kbase + Cfg::kBlockBytes;
        const int nvalid = C_kvlen - C_page * kPage;  // >= 1

        if (nvalid < kPage) {
            // Slots past the sequence end hold whatever the pool holds (possibly NaN):
            // zero those V rows so that 0 * V stays 0; their scores are masked below.
            char* vb = my_stages + stage * Cfg::kStageBytes + Cfg::kBlockBytes;
            const int units = (kPage - nvalid) * 8;  // 16-byte units per region of 16 rows x 128 bytes
            for (int h = 0; h < Cfg::kBlockBytes / 2048; ++h)
                for (int u = lane; u < units; u += 32)
                    *reinterpret_cast<uint4*>(vb + h * 2048 + nvalid * 128 + u * 16) = make_uint4(0, 0, 0, 0);
            fence_proxy_async_smem();  // order these generic writes before the stage's next bulk copy
            __syncwarp();
        }

        // S^T = K Q^T : 16 tokens x 8 head columns
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        float x0, x1, x2, x3;
        float sv_lo = 1.f, sv_hi = 1.f;  // FP8: V scales of this thread's two token rows
        if constexpr (FP8) {
            // One ldmatrix brings 16 tokens x 32 bytes: the thread gets bytes d = 16 u + 4 (lane % 4) + {0..3} of rows
            // `row` and `row + 8` for two 16-byte chunks u, each of which is one k-step after conversion.
#pragma unroll
            for (int kp = 0; kp < KS / 2; ++kp) {
                const uint32_t unit = (uint32_t)(((kp * 2 + (mi >> 1)) & 7) ^ l7);
                uint32_t r0, r1, r2, r3;
                ldsm_x4(kbase + k_tok_off + (unit << 4), r0, r1, r2, r3);
                mma_16816_f16(sa, e4m3x2_to_f16x2(r0), e4m3x2_to_f16x2(r1), e4m3x2_to_f16x2(r0 >> 16), e4m3x2_to_f16x2(r1 >> 16),
                              qb[2 * kp][0], qb[2 * kp][1]);
                mma_16816_f16(sb, e4m3x2_to_f16x2(r2), e4m3x2_to_f16x2(r3), e4m3x2_to_f16x2(r2 >> 16), e4m3x2_to_f16x2(r3 >> 16),
                              qb[2 * kp + 1][0], qb[2 * kp + 1][1]);
            }
            const float* scales = reinterpret_cast<const float*>(my_stages + stage * Cfg::kStageBytes + 2 * Cfg::kBlockBytes);
            const float fk_lo = scales[row] * p.scale_log2, fk_hi = scales[row + 8] * p.scale_log2;
            x0 = (sa[0] + sb[0]) * fk_lo, x1 = (sa[1] + sb[1]) * fk_lo;
            x2 = (sa[2] + sb[2]) * fk_hi, x3 = (sa[3] + sb[3]) * fk_hi;
            // slots past the sequence end hold arbitrary scales: their weights are zero, keep 0 * scale = 0
            sv_lo = row < nvalid ? scales[kPage + row] * kWeightScale : 0.f;
            sv_hi = row + 8 < nvalid ? scales[kPage + row + 8] * kWeightScale : 0.f;
        } else {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const uint32_t unit = (uint32_t)(((ks * 2 + (mi >> 1)) & 7) ^ l7);
                uint32_t a0, a1, a2, a3;
                ldsm_x4(kbase + (ks >> 2) * 2048 + k_tok_off + (unit << 4), a0, a1, a2, a3);
                if (ks & 1) mma_16816(sb, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
                else mma_16816(sa, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
            }
            x0 = (sa[0] + sb[0]) * p.scale_log2, x1 = (sa[1] + sb[1]) * p.scale_log2;
            x2 = (sa[2] + sb[2]) * p.scale_log2, x3 = (sa[3] + sb[3]) * p.scale_log2;
        }
        if (row >= nvalid) x0 = x1 = -INFINITY;
        if (row + 8 >= nvalid) x2 = x3 = -INFINITY;

        float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 4));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 4));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 8));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 8));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 16));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 16));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // finite: token 0 of the page is valid
        const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
        m0 = mn0;
        m1 = mn1;
        const float p0 = fast_exp2(x0 - mn0), p1 = fast_exp2(x1 - mn1);
        const float p2 = fast_exp2(x2 - mn0), p3 = fast_exp2(x3 - mn1);
        // the row sum uses the bf16-rounded weights that PV multiplies, so that the
        // normalised output is an exact convex mix of V rows
        uint32_t pk0, pk1;
        if constexpr (FP8) {
            // each key's V scale rides on its weight into the MMA; the row sum is over the weights themselves
            pk0 = pack_f16(p0 * sv_lo, p1 * sv_lo), pk1 = pack_f16(p2 * sv_hi, p3 * sv_hi);
            l0 = l0 * al0 + p0 + p2;
            l1 = l1 * al1 + p1 + p3;
        } else {
            pk0 = pack_bf16(p0, p1), pk1 = pack_bf16(p2, p3);
            l0 = l0 * al0 + bf16_lo(pk0) + bf16_lo(pk1);
            l1 = l1 * al1 + bf16_hi(pk0) + bf16_hi(pk1);
        }
        const uint32_t pb0 = movmatrix_t(pk0);
        const uint32_t pb1 = movmatrix_t(pk1);

        // O^T += V^T P^T : d x 8 head columns
        if constexpr (FP8) {
            // A transposed ldmatrix over 16-bit units hands the thread, per 16-byte chunk u, the bytes
            // V[token 2c][d], V[token 2c][d + 1], V[token 2c + 1][d], V[token 2c + 1][d + 1] with d = 16 u + 2 row
            // (tokens 2c, 2c + 1 of the first eight in one register, of the second eight in the next); a byte
            // permute pairs the two tokens of one d, so accumulator row `row` is d and row `row + 8` is d + 1.
#pragma unroll
            for (int mp = 0; mp < KS / 2; ++mp) {
                o[2 * mp][0] *= al0, o[2 * mp][1] *= al1, o[2 * mp][2] *= al0, o[2 * mp][3] *= al1;
                o[2 * mp + 1][0] *= al0, o[2 * mp + 1][1] *= al1, o[2 * mp + 1][2] *= al0, o[2 * mp + 1][3] *= al1;
                const uint32_t unit = (uint32_t)(((mp * 2 + (mi >> 1)) & 7) ^ l7);
                uint32_t r0, r1, r2, r3;
                ldsm_x4_t(vbase + k_tok_off + (unit << 4), r0, r1, r2, r3);
                r0 = __byte_perm(r0, 0, 0x3120), r1 = __byte_perm(r1, 0, 0x3120);
                r2 = __byte_perm(r2, 0, 0x3120), r3 = __byte_perm(r3, 0, 0x3120);
                mma_16816_f16(o[2 * mp], e4m3x2_to_f16x2(r0), e4m3x2_to_f16x2(r0 >> 16), e4m3x2_to_f16x2(r1), e4m3x2_to_f16x2(r1 >> 16),
                              pb0, pb1);
                mma_16816_f16(o[2 * mp + 1], e4m3x2_to_f16x2(r2), e4m3x2_to_f16x2(r2 >> 16), e4m3x2_to_f16x2(r3), e4m3x2_to_f16x2(r3 >> 16),
                              pb0, pb1);
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                o[mt][0] *= al0;
                o[mt][1] *= al1;
                o[mt][2] *= al0;
                o[mt][3] *= al1;
                const uint32_t unit = (uint32_t)(((mt * 2 + (mi & 1)) & 7) ^ l7);
                uint32_t a0, a1, a2, a3;
                ldsm_x4_t(vbase + (mt >> 2) * 2048 + v_tok_off + (unit << 4), a0, a1, a2, a3);
                mma_16816(o[mt], a0, a1, a2, a3, pb0, pb1);
            }
        }

        __syncwarp();  // every lane has read this stage
        ++C_page;
        ++n_cons;
        produce();     // refill the stage just released
    }

    if (!timed_out) {
        __syncwarp();
        for (int k = 0; k < n_deferred; ++k) combine(deferred[3 * k], deferred[3 * k + 1], deferred[3 * k + 2]);
    }
    if (timed_out) {
        // let the copies still in flight (the one waited for included) land before the CTA's shared memory is released
        for (uint32_t n = n_cons; n < n_prod; ++n) mbar_wait(bar0 + 8 * (n % STAGES), (n / STAGES) & 1, kDrainLimitNs);
    }
}

}  // namespace

int decode_warps_per_sm() { return kWarps; }

template <int D, bool FP8>
static ps_status launch_decode_d(const RunArgs& a) {
    using Cfg = DecodeCfg<D, FP8>;
    static PerDeviceOnce configured;
    const ps_status cfg = once_per_device(configured, []() -> ps_status {
        PS_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<D, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
        return PS_OK;
    });
    if (cfg != PS_OK) return cfg;
    DecodeParams p;
    p.pool = a.pool;
    p.num_pages = a.num_pages;
    p.q = a.q;
    p.block_table = a.block_table;
    p.max_pages = a.max_pages;
    p.out = a.out;
    p.lse = a.lse;
    p.hdr = a.w.hdr;
    p.pieces = a.w.pieces;
    p.units = a.w.units;
    p.n_units = a.w.n_units;
    p.dmerge = a.w.dmerge;
    p.dmerge_cnt = a.w.dmerge_cnt;
    p.part_lse = a.w.part_lse;
    p.part_o = a.w.part_o;
    p.Hq = a.shape.n_q_heads;
    p.Hkv = a.shape.n_kv_heads;
    p.G = p.Hq / p.Hkv;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)D);
    p.n_req = a.n_req;
    p.total_q = a.total_q;
    p.n_dmerge = a.w.n_dmerge;
    p.n_part_slots = a.w.n_part_slots;
    p.wait_limit_ns = a.wait_limit_ns;
    int grid = (a.w.n_units + kWarps - 1) / kWarps;
    if (grid > a.dec_sms) grid = a.dec_sms;
    decode_kernel<D, FP8><<<grid, kWarps * 32, Cfg::kSmemBytes, a.stream>>>(p);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status launch_decode(const RunArgs& a) {
    if (a.w.n_units == 0) return PS_OK;
    if (a.shape.dtype == 1) return launch_decode_d<128, true>(a);  // the FP8 cache variant exists for head_dim 128
    return a.shape.head_dim == 128 ? launch_decode_d<128, false>(a) : launch_decode_d<64, false>(a);
}

}  // namespace ps
