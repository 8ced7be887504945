// Internal declarations shared by the library's translation units: error
// plumbing, the KV pool layout, the device work-list records and thin wrappers
// over the PTX the kernels use (mbarrier, bulk async copy, ldmatrix, mma).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <mutex>

#include "../../include/polyserve_attn.h"

namespace ps {

// ---------------------------------------------------------------------------
// errors
// ---------------------------------------------------------------------------
ps_status fail(ps_status code, const char* fmt, ...);
void clear_error();

#define PS_CUDA_TRY(expr)                                                                     \
    do {                                                                                      \
        cudaError_t e__ = (expr);                                                             \
        if (e__ != cudaSuccess) {                                                             \
            (void)cudaGetLastError(); /* reported here: do not leave it for an unrelated later call */ \
            return ps::fail(PS_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), \
                            __FILE__, __LINE__);                                              \
        }                                                                                     \
    } while (0)

ps_status check_shape(const ps_shape* s);

// Kernel attributes (the opt-in to large dynamic shared memory) belong to a device: run `configure` once
// per device the calling process launches on.  `state` is a function-local static of the caller.
struct PerDeviceOnce {
    std::mutex mu;
    uint64_t done[4] = {0, 0, 0, 0};  // one bit per device ordinal (up to 256)
};
template <typename F>
ps_status once_per_device(PerDeviceOnce& state, F configure) {
    int dev = 0;
    PS_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(state.mu);
    uint64_t& word = state.done[(dev >> 6) & 3];
    const uint64_t bit = 1ull << (dev & 63);
    if (word & bit) return PS_OK;
    const ps_status st = configure();
    if (st == PS_OK) word |= bit;
    return st;
}

// ---------------------------------------------------------------------------
// KV pool layout
//
// A page holds kPage = 16 tokens.  For one (page, kv head) the pool stores a
// K block followed by a V block, each 16 * d bf16:
//     pool + ((page * Hkv + g) * 2 + kv) * (16 * d * 2 bytes)
// A block is d / 64 "halves" of [16 tokens][64 elements = 128 bytes]; inside a
// half the eight 16-byte units of token row t are stored at unit index
// u ^ (t & 7).  This is the 128-byte-swizzle pattern that both ldmatrix
// (conflict-free 8x8 fetches) and the tcgen05 shared-memory descriptors
// (SWIZZLE_128B, 8-row atoms of 1024 bytes) expect, so a block moves from HBM to
// shared memory as one plain bulk copy and is consumed in place.
// ---------------------------------------------------------------------------
constexpr int kPage = 16;

__host__ __device__ inline size_t block_bytes(int d) { return (size_t)kPage * d * 2; }
__host__ __device__ inline size_t page_head_bytes(int d) { return 2 * block_bytes(d); }
// FP8 (E4M3) cache variant: K codes, V codes (16 tokens x d bytes each, rows swizzled by 16-byte unit like a bf16
// half), then the 16 tokens' K scales and their V scales (fp32)
__host__ __device__ constexpr size_t fp8_page_head_bytes(int d) { return 2 * (size_t)kPage * d + 2 * kPage * sizeof(float); }

// byte offset of the 16-byte unit holding elements [8u', 8u'+8) of token t,
// where e = element index in [0, d), inside a K or V block
__host__ __device__ inline uint32_t unit_offset(int t, int e) {
    int half = e >> 6;
    int u = (e & 63) >> 3;
    return (uint32_t)(half * 2048 + t * 128 + ((u ^ (t & 7)) << 4));
}

struct KvPool {
    ps_shape shape;
    int64_t num_pages;
    char* base;
    bool owned;
    int32_t* meta_dev;   // q_start[n+1], prior[n] for ps_kv_write
    int32_t meta_cap;    // ints
    int32_t* flag_dev;   // bounds flag
};

const KvPool& pool_of(const ps_kv* kv);

// ---------------------------------------------------------------------------
// device work list
// ---------------------------------------------------------------------------
// (token, head) rows one prefill item covers: two q tiles of 128 rows that share their K/V stream
constexpr int kPrefillRowsPerItem = 256;

constexpr int kStatusOk = 0, kStatusBounds = 1, kStatusTimeout = 2;

// Device-side waits (on an mbarrier: a bulk copy landing, another warp's hand-over, an MMA group retiring) give up
// after this long and flag the run instead of holding the GPU; ps_plan_set_wait_limit changes it per plan.
constexpr int64_t kDefaultWaitLimitNs = 2000000000ll;
constexpr int64_t kMaxWaitLimitNs = 4000000000ll;  // the kernels time their waits on the low 32 bits of the nanosecond clock
// After a wait has run out, the copies a warp still has in flight get this long to land before its shared
// memory is released (independent of the plan's limit, which a test may set to zero).
constexpr int64_t kDrainLimitNs = 1000000000ll;

struct WsHeader {         // 64 bytes at the start of the workspace
    int32_t status;       // sticky OR of kStatus* seen by any kernel of the run
    int32_t decode_next;  // dynamic work counters
    int32_t prefill_next;
    int32_t pad[13];
};

// One contiguous page range of one (request, kv head) for the decode kernel.
struct DecodePiece {
    int32_t req;
    int32_t kv_head;
    int32_t page_begin;   // logical page indices within the request
    int32_t page_end;
    int32_t q_tok;        // packed q token index
    int32_t part_slot;    // first partial slot (head 0 of the group), or -1: write final output
    int32_t kv_len;       // keys visible to the row
    int32_t merge_idx;    // index into the decode merge records when part_slot >= 0
};

// A (request, kv head) whose keys were cut into n_seg pieces: partial (s, hh) is slot base + s * G + hh.
// The decode warp that delivers the last piece combines them (arrival counted in a zeroed int per record).
struct DecodeMerge {
    int32_t base;
    int32_t n_seg;
};

// A decode work unit: pieces [piece_begin, piece_end) processed by one warp.
struct DecodeUnit {
    int32_t piece_begin;
    int32_t piece_end;
};

// One q tile x key range of a prefill chunk for the prefill kernel.
struct PrefillItem {
    int32_t req;
    int32_t kv_head;
    int32_t key_begin;    // multiple of 128
    int32_t key_end;      // exclusive; <= first_pos + n_tok
    int32_t q_tok;        // packed index of the tile's first q token
    int32_t n_tok;        // q tokens in the item (<= 256 / G)
    int32_t part_slot;    // partial slot of (segment, token 0, head 0), or -1: write final output
    int32_t first_pos;    // absolute position of the tile's first q token (prior + index in chunk)
};

// Outputs combined from several segments: tokens [q_tok, q_tok + n_tok) x heads of
// kv head g; partial (i, s, hh) is slot base + s * seg_stride + i * G + hh.
struct MergeEntry {
    int32_t q_tok;
    int32_t n_tok;
    int32_t kv_head;
    int32_t base;
    int32_t n_seg;
    int32_t seg_stride;
    int32_t pad[2];
};

struct DeviceWork {       // pointers into the workspace for one run
    WsHeader* hdr;
    const DecodePiece* pieces;
    const DecodeUnit* units;
    const PrefillItem* prefill;
    const MergeEntry* merge;           // prefill q tile pairs cut into segments, combined by the merge kernel
    const DecodeMerge* dmerge;
    int32_t* dmerge_cnt;
    float* part_lse;
    float* part_o;
    int32_t n_units, n_prefill, n_merge, n_dmerge;
    int64_t n_part_slots;              // rows of part_lse / part_o
    const int32_t* prefill_cta_start;  // static prefill partition (n_prefill_ctas + 1 entries), unused when 0
    int32_t n_prefill_ctas;
};

struct RunArgs {
    ps_shape shape;
    const char* pool;
    int64_t num_pages;
    const __nv_bfloat16* q;
    const int32_t* block_table;
    int32_t max_pages;
    __nv_bfloat16* out;
    float* lse;           // may be null
    DeviceWork w;
    cudaStream_t stream;
    int num_sms;
    int dec_sms, pf_sms;  // SMs (= CTAs) for the decode and the prefill kernel
    int32_t total_q;      // q tokens of the batch (rows of q and out)
    int32_t n_req;        // requests of the batch (rows of the block table)
    int64_t wait_limit_ns;
};

ps_status launch_decode(const RunArgs& a);
ps_status launch_prefill(const RunArgs& a);
ps_status launch_merge(const RunArgs& a);
int decode_warps_per_sm();

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint32_t global_timer_lo() {
    uint32_t t;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t));
    return t;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait bounded in time: false if the phase did not complete within about limit_ns nanoseconds.  One
// non-blocking probe first; a limit of zero gives up right after it (the phase must already be complete).
// Otherwise the suspending form polls, and the clock is read only every kWaitPollsPerClockRead failed polls
// (it starts at the first such read), so a wait that ends normally never reads it.
constexpr uint32_t kWaitPollsPerClockRead = 64;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int64_t limit_ns) {
    if (mbar_test_wait(bar, parity)) return true;
    if (limit_ns <= 0) return false;
    uint64_t t0 = 0;
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i % kWaitPollsPerClockRead == 0) {
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > (uint64_t)limit_ns) return false;
        }
    }
}

// global -> shared bulk copy; bytes multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

// the same copy with an L2 eviction-priority hint (policy from l2_policy_evict_first)
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// the two bf16 halves of a packed pair, widened exactly
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

#endif  // __CUDACC__

}  // namespace ps
