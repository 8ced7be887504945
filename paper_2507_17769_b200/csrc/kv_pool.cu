// Paged KV pool: allocation, scatter of new tokens into pages, and the
// bit-exact gather used to read a sequence back.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

namespace ps {

static thread_local char g_err[512] = "";

ps_status fail(ps_status code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}
void clear_error() { g_err[0] = 0; }

ps_status check_shape(const ps_shape* s) {
    if (!s) return fail(PS_ERR_INVALID, "shape is null");
    if (s->n_q_heads < 1 || s->n_kv_heads < 1 || s->n_q_heads % s->n_kv_heads != 0)
        return fail(PS_ERR_INVALID, "n_q_heads=%d must be a positive multiple of n_kv_heads=%d", s->n_q_heads,
                    s->n_kv_heads);
    if (s->head_dim != 64 && s->head_dim != 128)
        return fail(PS_ERR_UNSUPPORTED, "head_dim=%d: only 64 and 128 are supported", s->head_dim);
    if (s->page_size != kPage) return fail(PS_ERR_UNSUPPORTED, "page_size=%d: only 16 is supported", s->page_size);
    if (s->dtype != 0 && s->dtype != 1) return fail(PS_ERR_UNSUPPORTED, "dtype=%d: 0 (bf16 cache) and 1 (FP8 E4M3 cache) are supported", s->dtype);
    if (s->dtype == 1 && s->head_dim != 128) return fail(PS_ERR_UNSUPPORTED, "the FP8 cache is supported for head_dim 128 only");
    int G = s->n_q_heads / s->n_kv_heads;
    if (G > 8 || (G & (G - 1)) != 0)
        return fail(PS_ERR_UNSUPPORTED, "q heads per kv head = %d: supported group sizes are 1, 2, 4, 8", G);
    return PS_OK;
}

// One thread moves one 16-byte unit of K and of V.
// grid.x covers T * Hkv * (d / 8) units.
__global__ void kv_write_kernel(char* pool, int64_t num_pages, const uint4* __restrict__ k_new,
                                const uint4* __restrict__ v_new, const int32_t* __restrict__ block_table,
                                int max_pages, const int32_t* __restrict__ q_start, const int32_t* __restrict__ prior,
                                int n, int Hkv, int d, int* flag) {
    const int units_per_tok = Hkv * (d >> 3);
    const int64_t total = (int64_t)q_start[n] * units_per_tok;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(idx / units_per_tok);
        const int rem = (int)(idx % units_per_tok);
        const int g = rem / (d >> 3);
        const int u = rem % (d >> 3);
        // request of packed token t: last r with q_start[r] <= t
        int lo = 0, hi = n - 1;
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (q_start[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int r = lo;
        const int pos = prior[r] + (t - q_start[r]);
        const int64_t page = block_table[(int64_t)r * max_pages + pos / kPage];
        if (page < 0 || page >= num_pages) { atomicOr(flag, kStatusBounds); continue; }
        const int slot = pos % kPage;
        char* blk = pool + ((page * Hkv + g) * 2) * block_bytes(d);
        const uint32_t off = unit_offset(slot, u * 8);
        *reinterpret_cast<uint4*>(blk + off) = k_new[idx];
        *reinterpret_cast<uint4*>(blk + block_bytes(d) + off) = v_new[idx];
    }
}

__global__ void kv_gather_kernel(const char* pool, int64_t num_pages, const int32_t* __restrict__ bt_row, int len,
                                 int Hkv, int d, uint4* k_out, uint4* v_out, int* flag) {
    const int units_per_tok = Hkv * (d >> 3);
    const int64_t total = (int64_t)len * units_per_tok;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int pos = (int)(idx / units_per_tok);
        const int rem = (int)(idx % units_per_tok);
        const int g = rem / (d >> 3);
        const int u = rem % (d >> 3);
        const int64_t page = bt_row[pos / kPage];
        if (page < 0 || page >= num_pages) { atomicOr(flag, kStatusBounds); continue; }
        const char* blk = pool + ((page * Hkv + g) * 2) * block_bytes(d);
        const uint32_t off = unit_offset(pos % kPage, u * 8);
        if (k_out) k_out[idx] = *reinterpret_cast<const uint4*>(blk + off);
        if (v_out) v_out[idx] = *reinterpret_cast<const uint4*>(blk + block_bytes(d) + off);
    }
}

// ---------------------------------------------------------------------------
// FP8 (E4M3) cache variant.  Each (token, kv head) vector of K and of V is stored as head_dim E4M3 codes with one
// fp32 scale: scale = amax / 448 rounded up to 8 significant bits (1 if the vector is zero), code =
// round-to-nearest-even(x / scale) saturating at +-448, both divisions IEEE fp32.  A token's codes never change
// when later tokens are appended.  (With 8 significant bits a softmax weight of exactly 1 times the scale is still
// exact in the 16-bit operand of the decode kernel's MMA.)
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t quantise4(float x0, float x1, float x2, float x3, float scale) {
    uint16_t lo, hi;  // cvt packs its first operand into the upper byte
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(x1, scale)), "f"(__fdiv_rn(x0, scale)));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(x3, scale)), "f"(__fdiv_rn(x2, scale)));
    return (uint32_t)lo | ((uint32_t)hi << 16);
}

// One warp quantises K and V of one (new token, kv head): lane l holds elements 4 l .. 4 l + 3 (head_dim = 128).
__global__ void kv_write_fp8_kernel(char* pool, int64_t num_pages, const uint2* __restrict__ k_new,
                                    const uint2* __restrict__ v_new, const int32_t* __restrict__ block_table, int max_pages,
                                    const int32_t* __restrict__ q_start, const int32_t* __restrict__ prior, int n, int Hkv,
                                    int* flag) {
    constexpr int d = 128;
    const int lane = threadIdx.x & 31;
    const int64_t total = (int64_t)q_start[n] * Hkv;
    for (int64_t vec = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); vec < total;
         vec += (int64_t)gridDim.x * (blockDim.x >> 5)) {
        const int t = (int)(vec / Hkv), g = (int)(vec % Hkv);
        int lo = 0, hi = n - 1;
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (q_start[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int r = lo;
        const int pos = prior[r] + (t - q_start[r]);
        const int64_t page = block_table[(int64_t)r * max_pages + pos / kPage];
        if (page < 0 || page >= num_pages) {
            if (lane == 0) atomicOr(flag, kStatusBounds);
            continue;
        }
        const int slot = pos % kPage;
        char* blk = pool + (page * Hkv + g) * fp8_page_head_bytes(d);
        const uint32_t off = (uint32_t)(slot * d + (((lane >> 2) ^ (slot & 7)) << 4) + 4 * (lane & 3));
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            const uint2 w = (kv == 0 ? k_new : v_new)[vec * (d / 4) + lane];
            const float x0 = bf16_lo(w.x), x1 = bf16_hi(w.x), x2 = bf16_lo(w.y), x3 = bf16_hi(w.y);
            float amax = fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3)));
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            float scale = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
            uint32_t sbits = __float_as_uint(scale);  // rounded up to 8 significant bits
            if (sbits & 0xffffu) sbits = (sbits | 0xffffu) + 1u;
            scale = __uint_as_float(sbits);
            *reinterpret_cast<uint32_t*>(blk + kv * (kPage * d) + off) = quantise4(x0, x1, x2, x3, scale);
            if (lane == 0) reinterpret_cast<float*>(blk + 2 * kPage * d)[kv * kPage + slot] = scale;
        }
    }
}

// Codes of logical tokens [0, len) of one sequence, one byte per element, and their scales.
__global__ void kv_gather_fp8_kernel(const char* pool, int64_t num_pages, const int32_t* __restrict__ bt_row, int len, int Hkv,
                                     uint32_t* k_out, uint32_t* v_out, float* k_scale_out, float* v_scale_out, int* flag) {
    constexpr int d = 128;
    const int64_t total = (int64_t)len * Hkv * (d / 4);
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int pos = (int)(idx / (Hkv * (d / 4)));
        const int rem = (int)(idx % (Hkv * (d / 4)));
        const int g = rem / (d / 4), w = rem % (d / 4);  // 4-byte word of the vector
        const int64_t page = bt_row[pos / kPage];
        if (page < 0 || page >= num_pages) { atomicOr(flag, kStatusBounds); continue; }
        const int slot = pos % kPage;
        const char* blk = pool + (page * Hkv + g) * fp8_page_head_bytes(d);
        const uint32_t off = (uint32_t)(slot * d + (((w >> 2) ^ (slot & 7)) << 4) + 4 * (w & 3));
        if (k_out) k_out[idx] = *reinterpret_cast<const uint32_t*>(blk + off);
        if (v_out) v_out[idx] = *reinterpret_cast<const uint32_t*>(blk + kPage * d + off);
        if (w == 0) {
            const float* sc = reinterpret_cast<const float*>(blk + 2 * kPage * d);
            if (k_scale_out) k_scale_out[(int64_t)pos * Hkv + g] = sc[slot];
            if (v_scale_out) v_scale_out[(int64_t)pos * Hkv + g] = sc[kPage + slot];
        }
    }
}

}  // namespace ps

using namespace ps;

struct ps_kv {
    KvPool p;
};

extern "C" {

const char* ps_last_error(void) { return g_err; }
const char* ps_version(void) { return "polyserve-attn 0.1 (sm_100a)"; }

ps_status ps_kv_bytes(const ps_shape* shape, int64_t num_pages, size_t* bytes_out) {
    ps_status st = check_shape(shape);
    if (st != PS_OK) return st;
    if (num_pages < 1 || !bytes_out) return fail(PS_ERR_INVALID, "num_pages=%lld or bytes_out invalid", (long long)num_pages);
    *bytes_out = (size_t)num_pages * shape->n_kv_heads *
                 (shape->dtype == 1 ? fp8_page_head_bytes(shape->head_dim) : page_head_bytes(shape->head_dim));
    return PS_OK;
}

ps_status ps_kv_alloc(const ps_shape* shape, int64_t num_pages, void* dev_mem, size_t dev_bytes, ps_kv** out) {
    size_t need = 0;
    ps_status st = ps_kv_bytes(shape, num_pages, &need);
    if (st != PS_OK) return st;
    if (!out) return fail(PS_ERR_INVALID, "out is null");
    if (num_pages > 0x7fffffffLL) return fail(PS_ERR_INVALID, "num_pages exceeds int32 page ids");
    if (dev_mem) {
        if (dev_bytes < need) return fail(PS_ERR_INVALID, "dev_bytes=%zu < required %zu", dev_bytes, need);
        if ((uintptr_t)dev_mem % 1024 != 0) return fail(PS_ERR_INVALID, "dev_mem must be 1024-byte aligned");
    }
    ps_kv* kv = new (std::nothrow) ps_kv();
    if (!kv) return fail(PS_ERR_OOM, "host allocation failed");
    kv->p.shape = *shape;
    kv->p.num_pages = num_pages;
    kv->p.owned = dev_mem == nullptr;
    kv->p.base = (char*)dev_mem;
    kv->p.meta_dev = nullptr;
    kv->p.flag_dev = nullptr;
    kv->p.meta_cap = 1 << 16;
    if (kv->p.owned) {
        cudaError_t e = cudaMalloc((void**)&kv->p.base, need);
        if (e != cudaSuccess) {
            delete kv;
            return fail(e == cudaErrorMemoryAllocation ? PS_ERR_OOM : PS_ERR_CUDA, "cudaMalloc(%zu) failed: %s", need,
                        cudaGetErrorString(e));
        }
    }
    cudaError_t e = cudaMalloc((void**)&kv->p.meta_dev, sizeof(int32_t) * (size_t)kv->p.meta_cap + 256);
    if (e == cudaSuccess) {
        kv->p.flag_dev = kv->p.meta_dev + kv->p.meta_cap;
        e = cudaMemset(kv->p.flag_dev, 0, 256);
    }
    if (e != cudaSuccess) {
        if (kv->p.owned) cudaFree(kv->p.base);
        if (kv->p.meta_dev) cudaFree(kv->p.meta_dev);
        delete kv;
        return fail(PS_ERR_CUDA, "pool metadata allocation failed: %s", cudaGetErrorString(e));
    }
    *out = kv;
    return PS_OK;
}

ps_status ps_kv_free(ps_kv* kv) {
    if (!kv) return PS_OK;
    if (kv->p.owned && kv->p.base) cudaFree(kv->p.base);
    if (kv->p.meta_dev) cudaFree(kv->p.meta_dev);
    delete kv;
    return PS_OK;
}

ps_status ps_kv_write(ps_kv* kv, const void* k_new_dev, const void* v_new_dev, const int32_t* block_table_dev,
                      int32_t max_pages, const int32_t* prior_host, const int32_t* q_len_host, int32_t n,
                      void* stream) {
    if (!kv || !k_new_dev || !v_new_dev || !block_table_dev || !prior_host || !q_len_host)
        return fail(PS_ERR_INVALID, "null argument");
    if (n < 1 || max_pages < 1) return fail(PS_ERR_INVALID, "n=%d, max_pages=%d must be positive", n, max_pages);
    if (2 * (int64_t)n + 1 > kv->p.meta_cap) return fail(PS_ERR_INVALID, "n=%d exceeds %d requests per call", n, (kv->p.meta_cap - 1) / 2);
    std::vector<int32_t> meta(2 * (size_t)n + 1);
    int64_t T = 0;
    for (int r = 0; r < n; ++r) {
        if (q_len_host[r] < 1 || prior_host[r] < 0)
            return fail(PS_ERR_INVALID, "request %d: q_len=%d prior=%d", r, q_len_host[r], prior_host[r]);
        if ((int64_t)prior_host[r] + q_len_host[r] > (int64_t)max_pages * kPage)
            return fail(PS_ERR_INVALID, "request %d: kv_len exceeds max_pages * page_size", r);
        meta[r] = (int32_t)T;
        T += q_len_host[r];
        if (T > 0x7fffffffLL / 64) return fail(PS_ERR_INVALID, "too many new tokens");
        meta[n + 1 + r] = prior_host[r];
    }
    meta[n] = (int32_t)T;
    cudaStream_t s = (cudaStream_t)stream;
    // pageable source: the runtime has staged the bytes when the call returns; calls on one
    // pool must be stream-ordered because they share meta_dev
    PS_CUDA_TRY(cudaMemcpyAsync(kv->p.meta_dev, meta.data(), meta.size() * sizeof(int32_t), cudaMemcpyHostToDevice, s));
    const int Hkv = kv->p.shape.n_kv_heads, d = kv->p.shape.head_dim;
    if (kv->p.shape.dtype == 1) {
        const int64_t warps = T * Hkv;
        const int blocks = (int)((warps + 7) / 8 < 148 * 16 ? (warps + 7) / 8 : 148 * 16);
        kv_write_fp8_kernel<<<blocks, 256, 0, s>>>(kv->p.base, kv->p.num_pages, (const uint2*)k_new_dev, (const uint2*)v_new_dev,
                                                   block_table_dev, max_pages, kv->p.meta_dev, kv->p.meta_dev + n + 1, n, Hkv,
                                                   kv->p.flag_dev);
        PS_CUDA_TRY(cudaGetLastError());
        return PS_OK;
    }
    const int64_t total = T * Hkv * (d / 8);
    const int threads = 256;
    const int blocks = (int)((total + threads - 1) / threads < 148 * 32 ? (total + threads - 1) / threads : 148 * 32);
    kv_write_kernel<<<blocks, threads, 0, s>>>(kv->p.base, kv->p.num_pages, (const uint4*)k_new_dev,
                                               (const uint4*)v_new_dev, block_table_dev, max_pages, kv->p.meta_dev,
                                               kv->p.meta_dev + n + 1, n, Hkv, d, kv->p.flag_dev);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status ps_kv_gather(const ps_kv* kv, const int32_t* block_table_row_dev, int32_t len, void* k_out_dev,
                       void* v_out_dev, void* stream) {
    if (!kv || !block_table_row_dev) return fail(PS_ERR_INVALID, "null argument");
    if (len < 0) return fail(PS_ERR_INVALID, "len=%d", len);
    if (len == 0 || (!k_out_dev && !v_out_dev)) return PS_OK;
    if (kv->p.shape.dtype == 1) return ps_kv_gather_fp8(kv, block_table_row_dev, len, k_out_dev, v_out_dev, nullptr, nullptr, stream);
    const int Hkv = kv->p.shape.n_kv_heads, d = kv->p.shape.head_dim;
    const int64_t total = (int64_t)len * Hkv * (d / 8);
    const int threads = 256;
    const int blocks = (int)((total + threads - 1) / threads < 148 * 32 ? (total + threads - 1) / threads : 148 * 32);
    kv_gather_kernel<<<blocks, threads, 0, (cudaStream_t)stream>>>(kv->p.base, kv->p.num_pages, block_table_row_dev,
                                                                   len, Hkv, d, (uint4*)k_out_dev, (uint4*)v_out_dev,
                                                                   kv->p.flag_dev);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status ps_kv_gather_fp8(const ps_kv* kv, const int32_t* block_table_row_dev, int32_t len, void* k_codes_out_dev,
                           void* v_codes_out_dev, float* k_scale_out_dev, float* v_scale_out_dev, void* stream) {
    if (!kv || !block_table_row_dev) return fail(PS_ERR_INVALID, "null argument");
    if (kv->p.shape.dtype != 1) return fail(PS_ERR_INVALID, "the pool does not hold an FP8 cache");
    if (len < 0) return fail(PS_ERR_INVALID, "len=%d", len);
    if (len == 0 || (!k_codes_out_dev && !v_codes_out_dev && !k_scale_out_dev && !v_scale_out_dev)) return PS_OK;
    const int Hkv = kv->p.shape.n_kv_heads;
    const int64_t total = (int64_t)len * Hkv * 32;
    const int threads = 256;
    const int blocks = (int)((total + threads - 1) / threads < 148 * 32 ? (total + threads - 1) / threads : 148 * 32);
    kv_gather_fp8_kernel<<<blocks, threads, 0, (cudaStream_t)stream>>>(kv->p.base, kv->p.num_pages, block_table_row_dev, len, Hkv,
                                                                       (uint32_t*)k_codes_out_dev, (uint32_t*)v_codes_out_dev,
                                                                       k_scale_out_dev, v_scale_out_dev, kv->p.flag_dev);
    PS_CUDA_TRY(cudaGetLastError());
    return PS_OK;
}

ps_status ps_kv_status(ps_kv* kv, void* stream) {
    if (!kv) return fail(PS_ERR_INVALID, "null argument");
    int flag = 0;
    PS_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    PS_CUDA_TRY(cudaMemcpy(&flag, kv->p.flag_dev, sizeof flag, cudaMemcpyDeviceToHost));
    if (flag) {
        PS_CUDA_TRY(cudaMemset(kv->p.flag_dev, 0, sizeof flag));
        return fail(PS_ERR_BOUNDS, "a block-table entry pointed outside the pool; that token was skipped");
    }
    return PS_OK;
}

}  // extern "C"

namespace ps {
const KvPool& pool_of(const ps_kv* kv) { return kv->p; }
}
