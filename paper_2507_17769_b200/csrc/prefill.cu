// Prefill-chunk attention on the 5th-generation tensor cores.
//
// A chunk's rows attend the prior context plus the chunk's own earlier tokens
// (paper sections 2.4 and 4.7); this part is a dense contraction and compute
// bound (section 3.4), so QK^T and PV run as tcgen05.mma with fp32
// accumulators in tensor memory.
//
// One CTA works on one item = up to two consecutive q tiles (A, B) of 128
// (token, head) rows each -- the G heads that share a kv head x 128 / G
// consecutive tokens -- over one key range.  Both tiles consume the same K and V
// tiles from shared memory, and while one tile's softmax runs on the CUDA cores
// the tensor core works for the other tile (ping-pong).
//
//   warps 0-3  softmax of tile A: thread t owns row t (= TMEM lane t); one
//              tcgen05.ld pass over S, causal mask by prior + i, running max
//              with lazy rescaling of O, P (bf16) stored back into the TMEM
//              columns S occupied, O / l and the log-sum-exp at the end
//   warps 4-7  the same for tile B
//   warp 8     producer: one 2 KB bulk async copy per (page, K|V, d half) into
//              2-stage K and V rings; the pool's page layout already is the
//              128-byte-swizzled operand layout, so blocks are consumed in place
//   warp 9     MMA issue: S_X = Q_X K^T (SS form, M128 N128 K16) and
//              O_X += P_X V (A operand from TMEM, V as MN-major B operand,
//              M128 N=d K16); completion signalled with tcgen05.commit
//
// TMEM columns: S_A 0..127, S_B 128..255, O_A 256.., O_B 384.. (512 allocated).
// Every wait is bounded; on expiry the CTA sets the timeout status and drains.
#include "common.cuh"

namespace ps {

namespace {

constexpr int kSoftmaxThreads = 256;
// Three warpgroups: two of softmax warps and one holding the producer and MMA warps (its
// other two warps only take part in the CTA-wide barriers).  Registers are re-split after
// start-up: 384 threads x 168 at launch = 2 x 128 x 200 + 128 x 104.
constexpr int kThreads = kSoftmaxThreads + 128;
constexpr int kRegsSoftmax = 200, kRegsOther = 104;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kTileKeys = 128;
constexpr int kRows = 128;
constexpr float kRescaleThreshold = 8.f;  // log2 units
// ---- tcgen05 wrappers -------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// One leader lane of a converged warp (always the same one for the full mask).  Issuing the MMAs under this
// predicate, rather than under a test of the lane index, keeps the descriptor arithmetic warp-uniform.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.b32 %0, 1, 0, P;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// 3-input max and packed fp32 pairs (two lanes per 64-bit register)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row atoms of 1024 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version for this architecture
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kRows >> 4) << 24);
}

template <int D>
struct PrefillCfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kHalfBytes = kTileKeys * 128;          // [128 rows][128 B]
    static constexpr int kQBytes = kHalves * kHalfBytes;         // one Q tile
    static constexpr int kKBytes = kHalves * kHalfBytes;         // one K stage
    static constexpr int kVBytes = kHalves * kHalfBytes;         // one V stage
    static constexpr int kStages = 2;
    static constexpr int kOffQ = 0;                              // Q_A, Q_B
    static constexpr int kOffK = kOffQ + 2 * kQBytes;
    static constexpr int kOffV = kOffK + kStages * kKBytes;
    static constexpr int kOffBar = kOffV + kStages * kVBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;      // + alignment slack
    static constexpr int kTmemCols = 512;
    static constexpr uint32_t kColS = 0, kColO = 256, kColTile = 128;  // tile X at + X * 128
};

struct PrefillParams {
    const char* pool;
    int64_t num_pages;
    const __nv_bfloat16* q;
    const int32_t* block_table;
    int32_t max_pages;
    __nv_bfloat16* out;
    float* lse;
    WsHeader* hdr;
    const PrefillItem* items;
    int32_t n_items;
    const int32_t* cta_start;  // static partition: this CTA runs items [cta_start[b], cta_start[b + 1]); null = dynamic queue
    float* part_lse;
    float* part_o;
    int32_t Hq, Hkv, G;
    float scale_log2;
};

struct Bars {  // byte offsets from the barrier block; [2] = one per stage or per tile
    static constexpr int k_full = 0, k_empty = 16, v_full = 32, v_empty = 48, s_full = 64, p_ready = 80, o_done = 96;
    static constexpr int tmem_slot = 112, item_slot = 116, abort_slot = 120;
};

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < 40000000u; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// warp-uniform result, so that the warp-collective instructions that follow stay converged
__device__ __forceinline__ bool wait_all(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, wait_or_abort(bar, parity, abort_flag));
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1) prefill_kernel(const PrefillParams p) {
    using Cfg = PrefillCfg<D>;
    extern __shared__ char smem_raw[];
    char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + Cfg::kOffBar;
    volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::tmem_slot);
    volatile int* s_item = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::item_slot);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::abort_slot);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(bars + Bars::k_full + 8 * s, 1);
            mbar_init(bars + Bars::k_empty + 8 * s, 1);
            mbar_init(bars + Bars::v_full + 8 * s, 1);
            mbar_init(bars + Bars::v_empty + 8 * s, 1);
            mbar_init(bars + Bars::s_full + 8 * s, 1);
            mbar_init(bars + Bars::p_ready + 8 * s, kRows / 32);
            mbar_init(bars + Bars::o_done + 8 * s, 1);
        }
        mbar_fence_init();
        *s_abort = 0;
    }
    if (warp == 0) {
        tmem_alloc(bars + Bars::tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)*s_tmem;

    // Phase counters; every role advances them identically.  Tile B's barriers only move in
    // items that have a second q tile, so they are counted separately.
    uint32_t tile_ctr = 0, tile_ctr_b = 0;  // key tiles processed so far (all items / items with a tile B)
    uint32_t item_ctr = 0, item_ctr_b = 0;  // items processed (phase of the per-item o_done barriers)
    constexpr uint32_t kIdescQK = instr_desc(kTileKeys, false);
    constexpr uint32_t kIdescPV = instr_desc(D, true);
    static_assert(kPrefillRowsPerItem == 2 * kRows, "the planner pairs two q tiles per item");
    const int tile_tok = kRows / p.G;

    // Every role runs this at the top of each item; two CTA-wide barriers per item (after the
    // item fetch, after the Q tiles are in shared memory) are executed by all 12 warps.
    PrefillItem it;
    int n_tiles = 0;
    bool has_b = false;
    int static_cur = p.cta_start ? p.cta_start[blockIdx.x] : 0;
    const int static_end = p.cta_start ? p.cta_start[blockIdx.x + 1] : 0;
    auto next_item = [&]() -> bool {
        if (threadIdx.x == 0)
            *s_item = p.cta_start ? (static_cur < static_end ? static_cur : p.n_items) : atomicAdd(&p.hdr->prefill_next, 1);
        ++static_cur;
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        const int item_idx = *s_item;
        if (item_idx >= p.n_items || *s_abort) return false;
        it = p.items[item_idx];
        n_tiles = (it.key_end - it.key_begin + kTileKeys - 1) / kTileKeys;
        has_b = it.n_tok > tile_tok;
        return true;
    };
    auto advance = [&]() {
        tile_ctr += n_tiles;
        ++item_ctr;
        if (has_b) {
            tile_ctr_b += n_tiles;
            ++item_ctr_b;
        }
    };

    if (warp < 8) {
        // ====================================================================
        // softmax warpgroups: tile x = warp / 4, row t = thread within the group
        // ====================================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        const int x = warp >> 2, t = threadIdx.x & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr + Cfg::kColS + x * Cfg::kColTile;
        const uint32_t o_addr = tmem + lane_addr + Cfg::kColO + x * Cfg::kColTile;
        const int hh = t % p.G;
        while (next_item()) {
            // ---- Q tile x -> shared memory (row t = token x * tile_tok + t / G, head t % G) ----
            const int i = x * tile_tok + t / p.G;
            const bool valid = i < it.n_tok;
            {
                const uint4* src = reinterpret_cast<const uint4*>(
                    p.q + ((int64_t)(it.q_tok + (valid ? i : 0)) * p.Hq + it.kv_head * p.G + hh) * D);
                char* qdst = smem + Cfg::kOffQ + x * Cfg::kQBytes + t * 128;
#pragma unroll
                for (int U = 0; U < D / 8; ++U) {
                    const uint4 v = valid ? __ldg(src + U) : make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(qdst + (U >> 3) * Cfg::kHalfBytes + (((U & 7) ^ (t & 7)) << 4)) = v;
                }
                fence_proxy_async_smem();
            }
            __syncthreads();

            if (x == 0 || has_b) {
                const int limit = it.first_pos + i;  // last visible key of this row
                const int tile_first_pos = it.first_pos + x * tile_tok;
                float m = -INFINITY, l = 0.f;
                bool ok = true;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const uint32_t tc = tile_ctr + j;                          // K/V stage phase
                    const uint32_t tcx = (x ? tile_ctr_b : tile_ctr) + j;     // phase of this tile's own barriers
                    ok = wait_all(bars + Bars::s_full + 8 * x, tcx & 1, s_abort);
                    if (!ok) break;
                    tc_fence_after();
                    const int tile_base = it.key_begin + j * kTileKeys;
                    const bool need_mask = (tile_base + kTileKeys - 1 > tile_first_pos) || (tile_base + kTileKeys > it.key_end);
                    const int vis = min(limit + 1, it.key_end) - tile_base;  // columns [0, vis) are visible to this row

                    uint32_t sv[4][32];
                    tmem_ld32(s_addr + 0, sv[0]);
                    tmem_ld32(s_addr + 32, sv[1]);
                    tmem_ld32(s_addr + 64, sv[2]);
                    tmem_ld32(s_addr + 96, sv[3]);
                    tmem_wait_ld();

                    // row max of the raw scores, four independent chains
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
                    if (need_mask) {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                const int col = q * 32 + c;
                                mx0 = (col < vis) ? fmaxf(mx0, __uint_as_float(sv[q][c])) : mx0;
                                mx1 = (col + 1 < vis) ? fmaxf(mx1, __uint_as_float(sv[q][c + 1])) : mx1;
                                mx2 = (col + 2 < vis) ? fmaxf(mx2, __uint_as_float(sv[q][c + 2])) : mx2;
                                mx3 = (col + 3 < vis) ? fmaxf(mx3, __uint_as_float(sv[q][c + 3])) : mx3;
                            }
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                mx0 = max3(mx0, __uint_as_float(sv[q][c]), __uint_as_float(sv[q][c + 1]));
                                mx1 = max3(mx1, __uint_as_float(sv[q][c + 2]), __uint_as_float(sv[q][c + 3]));
                                mx2 = max3(mx2, __uint_as_float(sv[q][c + 4]), __uint_as_float(sv[q][c + 5]));
                                mx3 = max3(mx3, __uint_as_float(sv[q][c + 6]), __uint_as_float(sv[q][c + 7]));
                            }
                    }
                    const float mx_s = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                    float m_new = m;
                    if (mx_s > m + kRescaleThreshold) m_new = mx_s;  // also the first finite max (m = -inf)
                    const float alpha = (m_new == m) ? 1.f : fast_exp2(m - m_new);

                    // O_x holds tiles 0..j-1 (the commit that raised s_full came after PV_x(j-1))
                    if (j > 0 && __any_sync(0xffffffffu, m_new != m)) {
#pragma unroll 1
                        for (int c0 = 0; c0 < D; c0 += 32) {
                            uint32_t v[32];
                            tmem_ld32(o_addr + c0, v);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) v[c] = __float_as_uint(__uint_as_float(v[c]) * alpha);
                            tmem_st32(o_addr + c0, v);
                        }
                        tmem_wait_st();
                    }
                    l *= alpha;
                    m = m_new;
                    const float m_sub = (m == -INFINITY) ? 0.f : m;

                    // P = exp2(scale * s - m) as bf16 pairs, written over S's first 64 columns
                    float l0 = 0.f, l1 = 0.f;
                    if (need_mask) {
                        // Diagonal and ragged tiles (the only tiles of rows with few visible keys): mask by
                        // select, and sum the bf16-rounded weights that PV multiplies, so that the output
                        // of a row with a handful of keys stays an exact convex mix of V rows.
#pragma unroll
                        for (int hhalf = 0; hhalf < 2; ++hhalf) {
                            uint32_t packed[32];
#pragma unroll
                            for (int qq = 0; qq < 2; ++qq) {
                                const int q = hhalf * 2 + qq;
#pragma unroll
                                for (int c = 0; c < 32; c += 2) {
                                    float p0 = fast_exp2(fmaf(__uint_as_float(sv[q][c]), p.scale_log2, -m_sub));
                                    float p1 = fast_exp2(fmaf(__uint_as_float(sv[q][c + 1]), p.scale_log2, -m_sub));
                                    p0 = (q * 32 + c < vis) ? p0 : 0.f;
                                    p1 = (q * 32 + c + 1 < vis) ? p1 : 0.f;
                                    const uint32_t pk = pack_bf16(p0, p1);
                                    l0 += bf16_lo(pk);
                                    l1 += bf16_hi(pk);
                                    packed[qq * 16 + (c >> 1)] = pk;
                                }
                            }
                            tmem_st32(s_addr + hhalf * 32, packed);
                        }
                    } else {
                        // Interior tiles: two scores per instruction (packed fp32 FMA and add); four sum chains.
                        const uint64_t sc2 = pack2(p.scale_log2, p.scale_log2), nm2 = pack2(-m_sub, -m_sub);
                        uint64_t ls0 = 0ull, ls1 = 0ull;
#pragma unroll
                        for (int hhalf = 0; hhalf < 2; ++hhalf) {
                            uint32_t packed[32];
#pragma unroll
                            for (int qq = 0; qq < 2; ++qq) {
                                const int q = hhalf * 2 + qq;
#pragma unroll
                                for (int c = 0; c < 32; c += 4) {
                                    const uint64_t x01 = fma2(pack2(__uint_as_float(sv[q][c]), __uint_as_float(sv[q][c + 1])), sc2, nm2);
                                    const uint64_t x23 = fma2(pack2(__uint_as_float(sv[q][c + 2]), __uint_as_float(sv[q][c + 3])), sc2, nm2);
                                    float x0, x1, x2, x3;
                                    unpack2(x01, x0, x1);
                                    unpack2(x23, x2, x3);
                                    // (a cubic on the FMA pipe for part of these was measured slower in every mix)
                                    const float e0 = fast_exp2(x0), e1 = fast_exp2(x1), e2 = fast_exp2(x2), e3 = fast_exp2(x3);
                                    ls0 = add2(ls0, pack2(e0, e1));
                                    ls1 = add2(ls1, pack2(e2, e3));
                                    packed[qq * 16 + (c >> 1)] = pack_bf16(e0, e1);
                                    packed[qq * 16 + (c >> 1) + 1] = pack_bf16(e2, e3);
                                }
                            }
                            tmem_st32(s_addr + hhalf * 32, packed);
                        }
                        float a0, a1, a2, a3;
                        unpack2(ls0, a0, a1);
                        unpack2(ls1, a2, a3);
                        l0 = a0 + a2;
                        l1 = a1 + a3;
                    }
                    l += l0 + l1;
                    tmem_wait_st();

                    // keys at or past key_end: their V rows may be stale or poisoned; zero them so 0 * V = 0
                    const int n_keys = it.key_end - tile_base;
                    if (x == 0 && n_keys < kTileKeys) {
                        const uint32_t s = tc & 1;
                        ok = wait_all(bars + Bars::v_full + 8 * s, (tc >> 1) & 1, s_abort);
                        if (!ok) break;
                        if (t >= n_keys) {
                            char* vrow = smem + Cfg::kOffV + s * Cfg::kVBytes + t * 128;
#pragma unroll
                            for (int h = 0; h < Cfg::kHalves; ++h)
#pragma unroll
                                for (int u = 0; u < 8; ++u)
                                    *reinterpret_cast<uint4*>(vrow + h * Cfg::kHalfBytes + u * 16) = make_uint4(0, 0, 0, 0);
                        }
                        fence_proxy_async_smem();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bars + Bars::p_ready + 8 * x);  // one arrival per softmax warp
                }
                // ---- epilogue: O / l ----
                if (ok) ok = wait_all(bars + Bars::o_done + 8 * x, (x ? item_ctr_b : item_ctr) & 1, s_abort);
                if (ok) {
                    tc_fence_after();
                    const float inv = l > 0.f ? 1.f / l : 0.f;
                    const float lse_v = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
                    const int64_t orow = (int64_t)(it.q_tok + i) * p.Hq + it.kv_head * p.G + hh;
                    const int64_t prow = (int64_t)it.part_slot + (int64_t)i * p.G + hh;
#pragma unroll 1
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(o_addr + c0, v);
                        tmem_wait_ld();
                        if (!valid) continue;
                        if (it.part_slot < 0) {
                            uint4* dst = reinterpret_cast<uint4*>(p.out + orow * D + c0);
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                uint4 w;
                                w.x = pack_bf16(__uint_as_float(v[8 * u + 0]) * inv, __uint_as_float(v[8 * u + 1]) * inv);
                                w.y = pack_bf16(__uint_as_float(v[8 * u + 2]) * inv, __uint_as_float(v[8 * u + 3]) * inv);
                                w.z = pack_bf16(__uint_as_float(v[8 * u + 4]) * inv, __uint_as_float(v[8 * u + 5]) * inv);
                                w.w = pack_bf16(__uint_as_float(v[8 * u + 6]) * inv, __uint_as_float(v[8 * u + 7]) * inv);
                                dst[u] = w;
                            }
                        } else {
                            float4* dst = reinterpret_cast<float4*>(p.part_o + prow * D + c0);
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                dst[u] = make_float4(__uint_as_float(v[4 * u]) * inv, __uint_as_float(v[4 * u + 1]) * inv,
                                                     __uint_as_float(v[4 * u + 2]) * inv, __uint_as_float(v[4 * u + 3]) * inv);
                        }
                    }
                    if (valid) {
                        if (it.part_slot < 0) {
                            if (p.lse) p.lse[orow] = lse_v;
                        } else {
                            p.part_lse[prow] = lse_v;
                        }
                    }
                }
            }
            advance();
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        if (warp == kProducerWarp) {
            // ================================================================
            // producer
            // ================================================================
            const int pg = lane >> 2, which = lane & 3;  // page in tile; 0/1 = K half 0/1, 2/3 = V half 0/1
            constexpr uint32_t kPieceBytes = kPage * 128;  // 16 tokens x 64 elements
            while (next_item()) {
                // K and V do not depend on the Q tiles: the first tile's copies are issued before this
                // warp joins the item's second CTA-wide barrier (Q tiles in shared memory)
                bool joined = false;
                const int32_t* bt = p.block_table + (int64_t)it.req * p.max_pages + it.key_begin / kPage;
                bool ok = true;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const uint32_t tc = tile_ctr + j;
                    const uint32_t s = tc & 1, par = (tc >> 1) & 1;
                    const int n_keys = min(kTileKeys, it.key_end - (it.key_begin + j * kTileKeys));
                    const int n_pages = (n_keys + kPage - 1) / kPage;
                    const int page = (lane < n_pages) ? __ldg(bt + j * 8 + lane) : 0;
                    const bool in_range = (uint32_t)page < (uint64_t)p.num_pages;
                    const uint32_t good = __ballot_sync(0xffffffffu, lane < n_pages && in_range);
                    if (__popc(good) != n_pages && lane == 0) atomicOr(&p.hdr->status, kStatusBounds);
                    const int my_page = __shfl_sync(0xffffffffu, page, pg);
                    const bool mine = (good >> pg) & 1u;
                    const uint32_t tile_bytes = (uint32_t)__popc(good) * Cfg::kHalves * kPieceBytes;
                    const char* src = p.pool + ((int64_t)my_page * p.Hkv + it.kv_head) * (int64_t)(2 * Cfg::kHalves * kPieceBytes);

                    ok = wait_all(bars + Bars::k_empty + 8 * s, par ^ 1, s_abort);
                    if (!ok) break;
                    if (lane == 0) mbar_expect_tx(bars + Bars::k_full + 8 * s, tile_bytes);
                    __syncwarp();
                    if (mine && which < Cfg::kHalves)
                        bulk_g2s(sbase + Cfg::kOffK + s * Cfg::kKBytes + which * Cfg::kHalfBytes + pg * kPieceBytes,
                                 src + which * kPieceBytes, kPieceBytes, bars + Bars::k_full + 8 * s);

                    ok = wait_all(bars + Bars::v_empty + 8 * s, par ^ 1, s_abort);
                    if (!ok) break;
                    if (lane == 0) mbar_expect_tx(bars + Bars::v_full + 8 * s, tile_bytes);
                    __syncwarp();
                    if (mine && which >= 2 && which - 2 < Cfg::kHalves)
                        bulk_g2s(sbase + Cfg::kOffV + s * Cfg::kVBytes + (which - 2) * Cfg::kHalfBytes + pg * kPieceBytes,
                                 src + (Cfg::kHalves + which - 2) * kPieceBytes, kPieceBytes, bars + Bars::v_full + 8 * s);
                    if (!joined) {
                        __syncthreads();
                        joined = true;
                    }
                }
                if (!joined) __syncthreads();
                advance();
            }
        } else if (warp == kMmaWarp) {
            // ================================================================
            // MMA issue
            // ================================================================
            // descriptors without their start address; a k-step adds its byte offset / 16 to the low word
            const uint64_t desc_kmajor = smem_desc(0, 16, 1024);
            const uint64_t desc_v = smem_desc(0, Cfg::kHalfBytes, 1024);
            while (next_item()) {
                __syncthreads();
                bool ok = true;
                const int n_x = has_b ? 2 : 1;
                // S_x(j) = Q_x K(j)^T; the last tile to read K stage s releases it
                auto issue_qk = [&](int j, int x) {
                    const uint32_t tc = tile_ctr + j;
                    const uint32_t s = tc & 1;
                    if (x == 0) {
                        ok = wait_all(bars + Bars::k_full + 8 * s, (tc >> 1) & 1, s_abort);
                        if (!ok) return;
                        tc_fence_after();
                    }
                    if (elect_one()) {
                        const uint32_t d_addr = tmem + Cfg::kColS + x * Cfg::kColTile;
                        const uint64_t qd = desc_kmajor + ((sbase + Cfg::kOffQ + x * Cfg::kQBytes) >> 4);
                        const uint64_t kd = desc_kmajor + ((sbase + Cfg::kOffK + s * Cfg::kKBytes) >> 4);
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk >> 2) * Cfg::kHalfBytes + (kk & 3) * 32) >> 4;
                            tc_mma_ss(d_addr, qd + off, kd + off, kIdescQK, kk > 0);
                        }
                        tc_commit(bars + Bars::s_full + 8 * x);
                        if (x == n_x - 1) tc_commit(bars + Bars::k_empty + 8 * s);
                    }
                    __syncwarp();
                };
                for (int x = 0; x < n_x && ok; ++x) issue_qk(0, x);
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const uint32_t tc = tile_ctr + j;
                    const uint32_t s = tc & 1;
                    for (int x = 0; x < n_x && ok; ++x) {
                        ok = wait_all(bars + Bars::p_ready + 8 * x, ((x ? tile_ctr_b : tile_ctr) + j) & 1, s_abort);
                        if (!ok) break;
                        if (x == 0) {
                            ok = wait_all(bars + Bars::v_full + 8 * s, (tc >> 1) & 1, s_abort);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        if (elect_one()) {
                            // O_x += P_x V(j): P_x sits in S_x's first 64 columns, two bf16 per column
                            const uint32_t a_addr = tmem + Cfg::kColS + x * Cfg::kColTile;
                            const uint32_t d_addr = tmem + Cfg::kColO + x * Cfg::kColTile;
                            const uint64_t vd = desc_v + ((sbase + Cfg::kOffV + s * Cfg::kVBytes) >> 4);
#pragma unroll
                            for (int kk = 0; kk < kTileKeys / 16; ++kk)
                                tc_mma_ts(d_addr, a_addr + kk * 8, vd + kk * (2048 >> 4), kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                            if (j == n_tiles - 1) tc_commit(bars + Bars::o_done + 8 * x);
                            if (x == n_x - 1) tc_commit(bars + Bars::v_empty + 8 * s);
                        }
                        __syncwarp();
                        // the tensor pipe runs this thread's MMAs in issue order, so S_x may be
                        // overwritten by the next QK^T right behind the PV that reads P_x
                        if (j + 1 < n_tiles) issue_qk(j + 1, x);
                    }
                }
                advance();
            }
        } else {
            // the warpgroup's two spare warps only keep the CTA-wide barriers complete
            while (next_item()) {
                __syncthreads();
                advance();
            }
        }
    }

    // after an abort: flag the run and give copies in flight a bounded time to land
    if (*s_abort) {
        if (threadIdx.x == 0) atomicOr(&p.hdr->status, kStatusTimeout);
        for (int s = 0; s < 2; ++s) {
            mbar_wait(bars + Bars::k_full + 8 * s, 0, 200000u);
            mbar_wait(bars + Bars::v_full + 8 * s, 0, 200000u);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace

template <int D>
static ps_status launch_prefill_d(const RunArgs& a) {
    using Cfg = PrefillCfg<D>;
    static bool configured = false;
    if (!configured) {
        PS_CUDA_TRY(cudaFuncSetAttribute(prefill_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
        configured = true;
    }
    PrefillParams p;
    p.pool = a.pool;
    p.num_pages = a.num_pages;
    p.q = a.q;
    p.block_table = a.block_table;
    p.max_pages = a.max_pages;
    p.out = a.out;
    p.lse = a.lse;
    p.hdr = a.w.hdr;
    p.items = a.w.prefill;
    p.n_items = a.w.n_prefill;
    p.cta_start = a.w.n_prefill_ctas > 0 ? a.w.prefill_cta_start : nullptr;
    p.part_lse = a.w.part_lse;
    p.part_o = a.w.part_o;
    p.Hq = a.shape.n_q_heads;
    p.Hkv = a.shape.n_kv_heads;
    p.G = p.Hq / p.Hkv;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)D);
    const int grid = a.w.n_prefill_ctas > 0 ? a.w.n_prefill_ctas : (a.w.n_prefill < a.pf_sms ? a.w.n_prefill : a.pf_sms);
    prefill_kernel<D><<<grid, kThreads, Cfg::kSmemBytes, a.stream>>>(p);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status launch_prefill(const RunArgs& a) {
    if (a.w.n_prefill == 0) return PS_OK;
    return a.shape.head_dim == 128 ? launch_prefill_d<128>(a) : launch_prefill_d<64>(a);
}

}  // namespace ps
