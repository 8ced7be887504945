// Prefill-chunk attention on the 5th-generation tensor cores.
//
// A chunk's rows attend the prior context plus the chunk's own earlier tokens
// (paper sections 2.4 and 4.7); this part is a dense contraction and compute
// bound (section 3.4), so QK^T and PV run as tcgen05.mma with fp32
// accumulators in tensor memory.
//
// One CTA works through a list of items; an item = up to two consecutive q tiles
// (A, B) of 128 (token, head) rows each -- the G heads that share a kv head x
// 128 / G consecutive tokens -- over one key range.  Both tiles consume the same
// K and V tiles from shared memory, and while one tile's softmax runs on the
// CUDA cores the tensor core works for the other tile (ping-pong).
//
//   warps 0-3  softmax of tile A: thread t owns row t (= TMEM lane t); one
//              tcgen05.ld pass over S, causal mask by prior + i, running max
//              with lazy rescaling of O, P (bf16) stored back into the TMEM
//              columns S occupied; at the end of the item O / l and the
//              log-sum-exp, transposed through shared memory so that global
//              stores cover whole rows
//   warps 4-7  the same for tile B
//   warp 8     producer: fetches the CTA's next item and publishes its record in
//              a shared-memory ring; Q tiles by tensor-map loads (128-byte
//              swizzle); one 2 KB bulk async copy per (page, K|V, d half) into
//              2-stage K and V rings -- the pool's page layout already is the
//              128-byte-swizzled operand layout, so blocks are consumed in place
//   warp 9     MMA issue: S_X = Q_X K^T (SS form, M128 N128 K16) and
//              O_X += P_X V (A operand from TMEM, V as MN-major B operand,
//              M128 N=d K16); completion signalled with tcgen05.commit
//
// The roles synchronise through mbarriers only, so consecutive items overlap:
// the next item's Q, first K/V tiles and first QK^T are under way while the
// current item's last softmax, PV and output are still running.
//
// TMEM columns: S_A 0..127, S_B 128..255, O_A 256.., O_B 384.. (512 allocated).
// Every wait is bounded; on expiry the CTA sets the timeout status and drains.
#include <cuda.h>

#include "common.cuh"

namespace ps {

namespace {

constexpr int kSoftmaxThreads = 256;
// Three warpgroups: two of softmax warps and one holding the producer and MMA warps (its
// other two warps have no work).  Registers are re-split after
// start-up: 384 threads x 168 at launch = 2 x 128 x 192 + 128 x 120.
constexpr int kThreads = kSoftmaxThreads + 128;
constexpr int kRegsSoftmax = 192, kRegsOther = 120;
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
// One box of a 3-d tensor map into shared memory; completion is counted in bytes on `bar`.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
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

constexpr int kBarBlockBytes = 512;  // mbarriers, flags and the item record ring

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
    static constexpr int kStageWarpBytes = 32 * 128;             // output staging: 32 rows x 128 bytes per softmax warp
    static constexpr int kOffStage = kOffV + kStages * kVBytes;
    static constexpr int kOffBar = kOffStage + 8 * kStageWarpBytes;
    static constexpr int kSmemBytes = kOffBar + kBarBlockBytes + 1024;  // + alignment slack
    static constexpr int kTmemCols = 512;
    static constexpr uint32_t kColS = 0, kColO = 256, kColTile = 128;  // tile X at + X * 128
};

// Kept within 128 bytes: a larger parameter block makes the compiler copy it (and the tensor map) to the stack.
struct PrefillParams {
    const char* pool;
    const int32_t* block_table;
    __nv_bfloat16* out;
    float* lse;
    WsHeader* hdr;
    const PrefillItem* items;
    const int32_t* cta_start;  // static partition: this CTA runs items [cta_start[b], cta_start[b + 1]); null = dynamic queue
    float* part_lse;
    float* part_o;
    int64_t num_pages;
    uint32_t wait_limit_ns;
    int32_t max_pages;
    int32_t n_items;
    int32_t Hq, Hkv, G;
    int32_t n_req, total_q, n_part_slots;  // extents the item records are checked against
};
static_assert(sizeof(PrefillParams) <= 128, "parameter block");

constexpr int kItemRing = 4;        // item records in flight between the producer and the other roles
constexpr int kConsumerWarps = 9;   // eight softmax warps and the MMA warp read every record

struct Bars {  // byte offsets from the barrier block; [2] = one per stage or per q tile
    static constexpr int k_full = 0, k_empty = 16, v_full = 32, v_empty = 48, s_full = 64, p_ready = 80, o_done = 96;
    static constexpr int q_full = 112, q_empty = 128, item_full = 144, item_empty = item_full + 8 * kItemRing;
    static constexpr int tmem_slot = item_empty + 8 * kItemRing, abort_slot = tmem_slot + 4;
    static constexpr int limit_slot = abort_slot + 4;   // wait limit in ns, directly behind the abort flag
    static constexpr int mma_drained = limit_slot + 8;  // after an abort: the MMAs issued so far have retired
    static constexpr int armed = mma_drained + 8;       // 6 ints: parity of the last phase armed with copies (K, V stages, Q tiles)
    static constexpr int ring = 256;  // kItemRing PrefillItem records
    static constexpr int bytes = ring + kItemRing * (int)sizeof(PrefillItem);
};
static_assert(Bars::mma_drained % 8 == 0 && Bars::armed + 24 <= Bars::ring && sizeof(PrefillItem) == 32 &&
                  Bars::bytes <= kBarBlockBytes,
              "barrier block layout");

// Wait for a phase for at most about the CTA's wait limit (nanoseconds, in the word behind the abort flag; the low
// half of the nanosecond clock serves, so limits reach 4 s); gives up early when another role of the CTA has already
// given up.  The role whose wait runs out raises the CTA's abort flag.  One non-blocking probe first; a limit of
// zero gives up right after it.  The clock is read only every kWaitPollsPerClockRead failed polls.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_test_wait(bar, parity)) return true;
    const uint32_t limit_ns = (uint32_t)abort_flag[1];  // the wait limit sits behind the abort flag
    if (limit_ns > 0) {
        uint32_t t0 = 0;
        for (uint32_t i = 1;; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((i & (kWaitPollsPerClockRead - 1)) == 0) {
                if (*abort_flag) return false;
                const uint32_t now = global_timer_lo() | 1u;
                if (t0 == 0) t0 = now;
                else if (now - t0 > limit_ns) break;
            }
        }
    }
    *abort_flag = 1;
    return false;
}
template <int D>
__global__ void __launch_bounds__(kThreads, 1) prefill_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap q_map) {
    using Cfg = PrefillCfg<D>;
    extern __shared__ char smem_raw[];
    char* smem = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + Cfg::kOffBar;
    volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::tmem_slot);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::abort_slot);
    uint4* ring = reinterpret_cast<uint4*>(smem + Cfg::kOffBar + Bars::ring);  // two uint4 per record
    // written by the producer's lane 0: parity of the last phase of each K / V stage and Q buffer that it armed with
    // copies (-1: none yet); read only after an abort
    volatile int* const s_armed = reinterpret_cast<volatile int*>(smem + Cfg::kOffBar + Bars::armed);
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
            mbar_init(bars + Bars::q_full + 8 * s, 1);
            mbar_init(bars + Bars::q_empty + 8 * s, 1);
        }
        for (int s = 0; s < kItemRing; ++s) {
            mbar_init(bars + Bars::item_full + 8 * s, 1);
            mbar_init(bars + Bars::item_empty + 8 * s, kConsumerWarps);
        }
        mbar_init(bars + Bars::mma_drained, 1);
        mbar_fence_init();
        *s_abort = 0;
        s_abort[1] = (int)p.wait_limit_ns;
        for (int k = 0; k < 6; ++k) s_armed[k] = -1;
    }
    if (warp == 0) {
        tmem_alloc(bars + Bars::tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)*s_tmem;
    // warp-uniform result, so that the warp-collective instructions that follow stay converged
    auto wait_all = [](uint32_t bar, uint32_t parity, volatile int* abort_flag) {
        return __all_sync(0xffffffffu, wait_or_abort(bar, parity, abort_flag));
    };

    // The roles never meet at a CTA-wide barrier after this point: items flow through the record ring
    // and the mbarriers, so the next item's Q, K and first QK^T overlap the current item's last
    // softmax, PV and output.  Every role counts items and key tiles identically to derive barrier
    // phases; tile B's barriers only move in items that have a second q tile.
    constexpr uint32_t kIdescQK = instr_desc(kTileKeys, false);
    constexpr uint32_t kIdescPV = instr_desc(D, true);
    static_assert(kPrefillRowsPerItem == 2 * kRows, "the planner pairs two q tiles per item");
    const int tile_tok = kRows / p.G;
    const int g_shift = 31 - __clz(p.G);  // G is a power of two
    constexpr float kScaleLog2 = D == 128 ? 0.12751743f : 0.18033688f;  // log2(e) / sqrt(D)

    // consumer side of the record ring: record number n into `it`; false at the end-of-work record or on abort
    auto take_item = [&](uint32_t n, PrefillItem& it) -> bool {
        const uint32_t slot = n % kItemRing;
        if (!wait_all(bars + Bars::item_full + 8 * slot, (n / kItemRing) & 1, s_abort)) return false;
        const uint4 a = ring[2 * slot], b = ring[2 * slot + 1];
        it.req = (int32_t)a.x, it.kv_head = (int32_t)a.y, it.key_begin = (int32_t)a.z, it.key_end = (int32_t)a.w;
        it.q_tok = (int32_t)b.x, it.n_tok = (int32_t)b.y, it.part_slot = (int32_t)b.z, it.first_pos = (int32_t)b.w;
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + Bars::item_empty + 8 * slot);
        return it.n_tok > 0;
    };
    auto tiles_of = [](const PrefillItem& it) { return (it.key_end - it.key_begin + kTileKeys - 1) / kTileKeys; };
    // the MMA warp needs only an item's key-tile count and how many q tiles it has (0 q tiles: end of work)
    auto take_shape = [&](uint32_t n, int& n_tiles, int& n_x) -> bool {
        const uint32_t slot = n % kItemRing;
        if (!wait_all(bars + Bars::item_full + 8 * slot, (n / kItemRing) & 1, s_abort)) return false;
        const uint4 a = ring[2 * slot], b = ring[2 * slot + 1];
        n_tiles = ((int32_t)a.w - (int32_t)a.z + kTileKeys - 1) / kTileKeys;
        n_x = (int32_t)b.y > tile_tok ? 2 : 1;
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + Bars::item_empty + 8 * slot);
        return (int32_t)b.y > 0;
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
        const int hh = t & (p.G - 1);
        char* const stg = smem + Cfg::kOffStage + warp * Cfg::kStageWarpBytes;
        uint32_t n_item = 0, tile_ctr = 0, tiles_x = 0, items_x = 0;
        PrefillItem it;
        bool ok = true;
        while (ok && take_item(n_item, it)) {
            ++n_item;
            const int n_tiles = tiles_of(it);
            const bool has_b = it.n_tok > tile_tok;
            if (x == 0 || has_b) {
                const int i = x * tile_tok + (t >> g_shift);  // token of this row within the item
                const bool valid = i < it.n_tok;               // rows past the chunk's end compute on whatever the Q load brought
                const int limit = it.first_pos + i;            // last visible key of this row
                const int tile_first_pos = it.first_pos + x * tile_tok;
                float m = -INFINITY, l = 0.f;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const uint32_t tc = tile_ctr + j;  // K/V stage phase
                    ok = wait_all(bars + Bars::s_full + 8 * x, (tiles_x + j) & 1, s_abort);
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
                    const float mx_s = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * kScaleLog2;
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
                                    float p0 = fast_exp2(fmaf(__uint_as_float(sv[q][c]), kScaleLog2, -m_sub));
                                    float p1 = fast_exp2(fmaf(__uint_as_float(sv[q][c + 1]), kScaleLog2, -m_sub));
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
                        const uint64_t sc2 = pack2(kScaleLog2, kScaleLog2), nm2 = pack2(-m_sub, -m_sub);
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
                // ---- output: O / l through this warp's staging slice, so that global stores cover whole rows ----
                if (ok) ok = wait_all(bars + Bars::o_done + 8 * x, items_x & 1, s_abort);
                if (ok) {
                    tc_fence_after();
                    const float inv = l > 0.f ? 1.f / l : 0.f;
                    const float lse_v = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
                    const int row0 = (warp & 3) * 32;          // first tile row of this warp
                    const int sub = lane >> 3, unit = lane & 7;  // write-out: 4 rows per instruction, 8 lanes x 16 bytes per row
                    char* const my_row = stg + lane * 128;
                    if (it.part_slot < 0) {
                        // final output: bf16, 64 columns (128 bytes of each row) per pass
#pragma unroll 1
                        for (int c0 = 0; c0 < D; c0 += 64) {
                            uint32_t v[2][32];
                            tmem_ld32(o_addr + c0, v[0]);
                            tmem_ld32(o_addr + c0 + 32, v[1]);
                            tmem_wait_ld();
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const uint32_t* s = &v[u >> 2][(u & 3) * 8];
                                uint4 w;
                                w.x = pack_bf16(__uint_as_float(s[0]) * inv, __uint_as_float(s[1]) * inv);
                                w.y = pack_bf16(__uint_as_float(s[2]) * inv, __uint_as_float(s[3]) * inv);
                                w.z = pack_bf16(__uint_as_float(s[4]) * inv, __uint_as_float(s[5]) * inv);
                                w.w = pack_bf16(__uint_as_float(s[6]) * inv, __uint_as_float(s[7]) * inv);
                                *reinterpret_cast<uint4*>(my_row + ((u ^ (lane & 7)) << 4)) = w;
                            }
                            __syncwarp();
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const int r = k * 4 + sub, tt = row0 + r;
                                const int i_r = x * tile_tok + (tt >> g_shift);
                                if (i_r < it.n_tok) {
                                    const uint4 w = *reinterpret_cast<const uint4*>(stg + r * 128 + ((unit ^ (r & 7)) << 4));
                                    const int64_t orow_r = (int64_t)(it.q_tok + i_r) * p.Hq + it.kv_head * p.G + (tt & (p.G - 1));
                                    *reinterpret_cast<uint4*>(p.out + orow_r * D + c0 + unit * 8) = w;
                                }
                            }
                            __syncwarp();
                        }
                        if (valid && p.lse) p.lse[(int64_t)(it.q_tok + i) * p.Hq + it.kv_head * p.G + hh] = lse_v;
                    } else {
                        // partial result of a cut item: fp32 rows at consecutive slots, 32 columns per pass
                        const int64_t prow0 = (int64_t)it.part_slot + x * kRows + row0;
#pragma unroll 1
                        for (int c0 = 0; c0 < D; c0 += 32) {
                            uint32_t v[32];
                            tmem_ld32(o_addr + c0, v);
                            tmem_wait_ld();
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                *reinterpret_cast<float4*>(my_row + ((u ^ (lane & 7)) << 4)) =
                                    make_float4(__uint_as_float(v[4 * u]) * inv, __uint_as_float(v[4 * u + 1]) * inv,
                                                __uint_as_float(v[4 * u + 2]) * inv, __uint_as_float(v[4 * u + 3]) * inv);
                            __syncwarp();
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const int r = k * 4 + sub, tt = row0 + r;
                                if (x * tile_tok + (tt >> g_shift) < it.n_tok)
                                    *reinterpret_cast<float4*>(p.part_o + (prow0 + r) * D + c0 + unit * 4) =
                                        *reinterpret_cast<const float4*>(stg + r * 128 + ((unit ^ (r & 7)) << 4));
                            }
                            __syncwarp();
                        }
                        if (valid) p.part_lse[prow0 + lane] = lse_v;
                    }
                }
                tiles_x += n_tiles;
                ++items_x;
            }
            tile_ctr += n_tiles;
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        if (warp == kProducerWarp) {
            // K/V tiles of a chunk's sequence are read again by every q tile of that sequence (and of its other chunks' items
            // on other CTAs): they are marked last to leave L2, the decode kernel's streamed pages first.  Measured beside decode
            // rows: a 2048-token chunk on 8 K with 32 decode rows 275 -> 266 us, 512 on 2 K with 128 rows 171 -> 169 us; alone
            // within 1 %.
            const uint64_t kv_policy = l2_policy_evict_last();
            // ================================================================
            // producer: item records, Q tiles (tensor-map loads), K and V tiles (bulk copies of pool blocks)
            // ================================================================
            const int pg = lane >> 2, which = lane & 3;  // page in tile; 0/1 = K half 0/1, 2/3 = V half 0/1
            constexpr uint32_t kPieceBytes = kPage * 128;  // 16 tokens x 64 elements
            uint32_t n_item = 0, tile_ctr = 0, items_x[2] = {0, 0};
            int static_cur = p.cta_start ? p.cta_start[blockIdx.x] : 0;
            const int static_end = p.cta_start ? p.cta_start[blockIdx.x + 1] : 0;
            bool ok = true;
            while (ok) {
                // next item of this CTA's static share, or of the queue all CTAs of the run drain
                int idx = 0;
                if (lane == 0)
                    idx = p.cta_start ? (static_cur < static_end ? static_cur : p.n_items) : atomicAdd(&p.hdr->prefill_next, 1);
                ++static_cur;
                idx = __shfl_sync(0xffffffffu, idx, 0);
                uint4 rec0 = make_uint4(0, 0, 0, 0), rec1 = make_uint4(0, 0, 0, 0);  // n_tok = 0: end of work
                if (idx < p.n_items) {
                    const uint4* src = reinterpret_cast<const uint4*>(p.items + idx);
                    rec0 = __ldg(src);
                    rec1 = __ldg(src + 1);
                    // A record that points outside the batch (only a damaged work list has one) ends this CTA's
                    // work and flags the run; nothing is read or written through it.
                    const int32_t r_req = (int32_t)rec0.x, r_g = (int32_t)rec0.y, r_kb = (int32_t)rec0.z, r_ke = (int32_t)rec0.w;
                    const int32_t r_q = (int32_t)rec1.x, r_n = (int32_t)rec1.y, r_slot = (int32_t)rec1.z, r_pos = (int32_t)rec1.w;
                    const bool rec_ok = (uint32_t)r_req < (uint32_t)p.n_req && (uint32_t)r_g < (uint32_t)p.Hkv && r_kb >= 0 &&
                                        r_kb % kTileKeys == 0 && r_kb < r_ke && r_ke <= p.max_pages * kPage && r_n >= 1 &&
                                        r_n <= 2 * tile_tok && r_q >= 0 && (int64_t)r_q + r_n <= p.total_q && r_pos >= 0 &&
                                        (int64_t)r_pos + r_n >= r_ke &&
                                        (r_slot < 0 || (int64_t)r_slot + (int64_t)r_n * p.G <= p.n_part_slots);
                    if (!rec_ok) {
                        if (lane == 0) atomicOr(&p.hdr->status, kStatusBounds);
                        rec0 = rec1 = make_uint4(0, 0, 0, 0);
                    }
                }
                const uint32_t slot = n_item % kItemRing;
                ok = wait_all(bars + Bars::item_empty + 8 * slot, ((n_item / kItemRing) & 1) ^ 1, s_abort);
                if (!ok) break;
                if (lane == 0) {
                    ring[2 * slot] = rec0;
                    ring[2 * slot + 1] = rec1;
                    mbar_arrive(bars + Bars::item_full + 8 * slot);
                }
                ++n_item;
                struct { int32_t req, kv_head, key_begin, key_end, q_tok, n_tok; } it;
                it.req = (int32_t)rec0.x, it.kv_head = (int32_t)rec0.y, it.key_begin = (int32_t)rec0.z, it.key_end = (int32_t)rec0.w;
                it.q_tok = (int32_t)rec1.x, it.n_tok = (int32_t)rec1.y;
                if (it.n_tok <= 0) break;
                const int n_tiles = (it.key_end - it.key_begin + kTileKeys - 1) / kTileKeys;
                const int n_x = it.n_tok > tile_tok ? 2 : 1;
                const int32_t* bt = p.block_table + (int64_t)it.req * p.max_pages + it.key_begin / kPage;
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
                    if (lane == 0) {
                        mbar_expect_tx(bars + Bars::k_full + 8 * s, tile_bytes);
                        s_armed[s] = (int)par;
                    }
                    __syncwarp();
                    if (mine && which < Cfg::kHalves)
                        bulk_g2s_hint(sbase + Cfg::kOffK + s * Cfg::kKBytes + which * Cfg::kHalfBytes + pg * kPieceBytes,
                                      src + which * kPieceBytes, kPieceBytes, bars + Bars::k_full + 8 * s, kv_policy);

                    if (j == 0) {
                        // Q tile x: rows (token, head of the group) in token-major order, one box of
                        // [128 / G tokens][G heads][64 elements] per 64-element half, written with the
                        // 128-byte swizzle the MMA descriptors expect.  The buffer is free once the
                        // previous item's last QK^T of that tile has run.
                        for (int x = 0; x < n_x && ok; ++x) {
                            ok = wait_all(bars + Bars::q_empty + 8 * x, (items_x[x] & 1) ^ 1, s_abort);
                            if (!ok) break;
                            if (lane == 0) {
                                mbar_expect_tx(bars + Bars::q_full + 8 * x, Cfg::kQBytes);
                                s_armed[4 + x] = (int)(items_x[x] & 1);
#pragma unroll
                                for (int h = 0; h < Cfg::kHalves; ++h)
                                    tma_load_3d(sbase + Cfg::kOffQ + x * Cfg::kQBytes + h * Cfg::kHalfBytes, &q_map, h * 64,
                                                it.kv_head * p.G, it.q_tok + x * tile_tok, bars + Bars::q_full + 8 * x);
                            }
                            __syncwarp();
                        }
                        if (!ok) break;
                    }

                    ok = wait_all(bars + Bars::v_empty + 8 * s, par ^ 1, s_abort);
                    if (!ok) break;
                    if (lane == 0) {
                        mbar_expect_tx(bars + Bars::v_full + 8 * s, tile_bytes);
                        s_armed[2 + s] = (int)par;
                    }
                    __syncwarp();
                    if (mine && which >= 2 && which - 2 < Cfg::kHalves)
                        bulk_g2s_hint(sbase + Cfg::kOffV + s * Cfg::kVBytes + (which - 2) * Cfg::kHalfBytes + pg * kPieceBytes,
                                      src + (Cfg::kHalves + which - 2) * kPieceBytes, kPieceBytes, bars + Bars::v_full + 8 * s, kv_policy);
                }
                tile_ctr += n_tiles;
                ++items_x[0];
                if (n_x == 2) ++items_x[1];
            }
        } else if (warp == kMmaWarp) {
            // ================================================================
            // MMA issue
            // ================================================================
            // descriptors without their start address; a k-step adds its byte offset / 16 to the low word
            const uint64_t desc_kmajor = smem_desc(0, 16, 1024);
            const uint64_t desc_v = smem_desc(0, Cfg::kHalfBytes, 1024);
            uint32_t n_item = 0, tile_ctr = 0, tiles_x[2] = {0, 0}, items_x[2] = {0, 0};
            bool ok = true;
            // S_x = Q_x K^T for key tile number tc (counted over all items) of an item with n_x q tiles.
            // `first`: the item's first key tile (wait for its Q tile, phase q_par); `last`: its last one
            // (release the Q buffer).  The last q tile to read K stage s releases it.
            auto issue_qk = [&](uint32_t tc, int x, int n_x, bool first, bool last, uint32_t q_par) {
                const uint32_t s = tc & 1;
                if (x == 0) {
                    ok = wait_all(bars + Bars::k_full + 8 * s, (tc >> 1) & 1, s_abort);
                    if (!ok) return;
                }
                if (first) {
                    ok = wait_all(bars + Bars::q_full + 8 * x, q_par & 1, s_abort);
                    if (!ok) return;
                }
                tc_fence_after();
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
                    if (last) tc_commit(bars + Bars::q_empty + 8 * x);
                }
                __syncwarp();
            };
            int n_tiles = 0, n_x = 0, nx_tiles = 0, nx_n_x = 0;
            bool have = take_shape(n_item, n_tiles, n_x);
            ++n_item;
            bool pre[2] = {false, false};  // S_x of the item's first key tile was issued at the end of the previous item
            while (have && ok) {
                bool have_next = false;
                for (int x = 0; x < n_x && ok; ++x)
                    if (!pre[x]) issue_qk(tile_ctr, x, n_x, true, n_tiles == 1, items_x[x]);
                pre[0] = pre[1] = false;
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const uint32_t tc = tile_ctr + j;
                    const uint32_t s = tc & 1;
                    if (j == n_tiles - 1) {
                        have_next = take_shape(n_item, nx_tiles, nx_n_x);
                        ++n_item;
                    }
                    for (int x = 0; x < n_x && ok; ++x) {
                        ok = wait_all(bars + Bars::p_ready + 8 * x, (tiles_x[x] + j) & 1, s_abort);
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
                        // The tensor pipe runs this thread's MMAs in issue order, so S_x may be overwritten by
                        // the next QK^T right behind the PV that reads P_x -- the next key tile's, or after the
                        // item's last tile the next item's first (its O_x is not touched before that item's
                        // first P_x is ready, which the softmax warps signal only after writing this item's
                        // output).
                        if (j + 1 < n_tiles) {
                            issue_qk(tc + 1, x, n_x, false, j + 2 == n_tiles, 0);
                        } else if (have_next && x < nx_n_x) {
                            issue_qk(tile_ctr + n_tiles, x, nx_n_x, true, nx_tiles == 1, items_x[x] + 1);
                            pre[x] = true;
                        }
                    }
                }
                tile_ctr += n_tiles;
                for (int x = 0; x < n_x; ++x) {
                    tiles_x[x] += n_tiles;
                    ++items_x[x];
                }
                n_tiles = nx_tiles;
                n_x = nx_n_x;
                have = have_next;
            }
        }
        // (the warpgroup's two other warps have no work; they wait at the final barrier)
    }

    tc_fence_before();
    __syncthreads();  // every role has left its loop
    if (*s_abort) {
        // A bounded wait ran out somewhere in this CTA: the output is invalid and the run is flagged.  Before the CTA
        // gives back its shared and tensor memory, the copies the producer has requested get a bounded time to land
        // and the MMAs issued so far (they read shared memory and write tensor memory) to retire.
        if (threadIdx.x == 0) atomicOr(&p.hdr->status, kStatusTimeout);
        if (warp == kProducerWarp) {
            for (int k = 0; k < 2; ++k) {
                const int ak = s_armed[k], av = s_armed[2 + k], aq = s_armed[4 + k];
                if (ak >= 0) mbar_wait(bars + Bars::k_full + 8 * k, (uint32_t)ak, kDrainLimitNs);
                if (av >= 0) mbar_wait(bars + Bars::v_full + 8 * k, (uint32_t)av, kDrainLimitNs);
                if (aq >= 0) mbar_wait(bars + Bars::q_full + 8 * k, (uint32_t)aq, kDrainLimitNs);
            }
        }
        if (warp == kMmaWarp) {
            if (elect_one()) tc_commit(bars + Bars::mma_drained);
            __syncwarp();
            mbar_wait(bars + Bars::mma_drained, 0, kDrainLimitNs);
        }
        tc_fence_before();
        __syncthreads();
    }
    if (warp == 0) tmem_dealloc(tmem, Cfg::kTmemCols);
}

}  // namespace

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so that the library does not link libcuda.
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return (EncodeTiledFn)f;
    }();
    return fn;
}

}  // namespace

template <int D>
static ps_status launch_prefill_d(const RunArgs& a) {
    using Cfg = PrefillCfg<D>;
    static PerDeviceOnce configured;
    const ps_status cfg = once_per_device(configured, []() -> ps_status {
        PS_CUDA_TRY(cudaFuncSetAttribute(prefill_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
        return PS_OK;
    });
    if (cfg != PS_OK) return cfg;
    PrefillParams p;
    p.pool = a.pool;
    p.num_pages = a.num_pages;
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
    p.n_req = a.n_req;
    p.total_q = a.total_q;
    p.n_part_slots = (int32_t)a.w.n_part_slots;
    p.wait_limit_ns = (uint32_t)a.wait_limit_ns;

    // Q as a [T tokens][Hq heads][D] tensor; a box is one 64-element half of a q tile's 128 rows
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return fail(PS_ERR_CUDA, "the driver does not provide cuTensorMapEncodeTiled");
    CUtensorMap q_map;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)p.Hq, (cuuint64_t)a.total_q};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)p.Hq * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)p.G, (cuuint32_t)(kRows / p.G)};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    const CUresult r = encode(&q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(a.q), dims, strides, box,
                              elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(PS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);

    const int grid = a.w.n_prefill_ctas > 0 ? a.w.n_prefill_ctas : (a.w.n_prefill < a.pf_sms ? a.w.n_prefill : a.pf_sms);
    prefill_kernel<D><<<grid, kThreads, Cfg::kSmemBytes, a.stream>>>(p, q_map);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status launch_prefill(const RunArgs& a) {
    if (a.w.n_prefill == 0) return PS_OK;
    return a.shape.head_dim == 128 ? launch_prefill_d<128>(a) : launch_prefill_d<64>(a);
}

}  // namespace ps
