// Latency-table sweep: times one iteration's attention over a grid of
// (prefill chunk size, decode count, mean context length) cells.  The serving
// scheduler predicts iteration time from such a profiled table keyed by token
// batch size and KV-cache size (paper section 4.5).
#include <algorithm>
#include <chrono>
#include <cstdio>
#include <numeric>
#include <vector>

#include "common.cuh"

namespace ps {

namespace {

// SplitMix64 (Steele, Lea, Flood 2014): draw k of the stream keyed s is the
// finaliser applied to s + (k + 1) * gamma.  Stream ids and the multiply-shift
// range reduction match the published recipe of the sweep's length law, so a
// caller can regenerate every draw's lengths from its seed.
constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
inline uint64_t finalise(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
inline uint64_t mix64(uint64_t x) { return finalise(x + kGamma); }
inline uint64_t stream_key(uint64_t seed, uint64_t stream, uint64_t seq) {
    uint64_t k = mix64(seed) ^ stream;
    k = mix64(k) ^ seq;
    return mix64(k);
}
inline uint64_t draw(uint64_t key, uint64_t idx) { return finalise(key + (idx + 1) * kGamma); }
inline int64_t uniform_int(uint64_t key, uint64_t idx, int64_t lo, int64_t hi) {
    const uint64_t r = draw(key, idx) >> 32;
    return lo + (int64_t)((r * (uint64_t)(hi - lo + 1)) >> 32);
}
constexpr uint64_t kStreamLen = 11, kStreamPerm = 12, kStreamPrior = 13;

struct Draw {
    std::vector<int32_t> prior, q_len;
    std::vector<int32_t> block_table;  // [n, max_pages]
    int32_t max_pages = 0;
    int64_t num_pages = 0, kv_tokens = 0;
    int32_t prefill_prior = 0;
};

void make_draw(int chunk, int n_decode, int mean_ctx, uint64_t seed, Draw* d) {
    const int64_t lo = mean_ctx / 2, hi = (3LL * mean_ctx) / 2;
    const uint64_t klen = stream_key(seed, kStreamLen, 0), kpr = stream_key(seed, kStreamPrior, 0);
    d->prior.clear();
    d->q_len.clear();
    for (int i = 0; i < n_decode; ++i) {
        d->prior.push_back((int32_t)(uniform_int(klen, i, lo, hi) - 1));
        d->q_len.push_back(1);
    }
    d->prefill_prior = 0;
    if (chunk > 0) {
        d->prefill_prior = (int32_t)uniform_int(kpr, 0, lo, hi);
        d->prior.push_back(d->prefill_prior);
        d->q_len.push_back(chunk);
    }
    const int n = (int)d->prior.size();
    std::vector<int64_t> need(n);
    int64_t total = 0;
    d->kv_tokens = 0;
    d->max_pages = 1;
    for (int r = 0; r < n; ++r) {
        const int64_t kv = (int64_t)d->prior[r] + d->q_len[r];
        d->kv_tokens += kv;
        need[r] = (kv + kPage - 1) / kPage;
        total += need[r];
        d->max_pages = std::max<int32_t>(d->max_pages, (int32_t)need[r]);
    }
    d->num_pages = std::max<int64_t>((total * 5 + 3) / 4, total + 8);
    // seeded permutation: stable order of the pages' keyed draws
    const uint64_t kperm = stream_key(seed, kStreamPerm, 0);
    std::vector<uint64_t> keys((size_t)d->num_pages);
    for (int64_t i = 0; i < d->num_pages; ++i) keys[(size_t)i] = draw(kperm, (uint64_t)i);
    std::vector<int32_t> perm((size_t)d->num_pages);
    std::iota(perm.begin(), perm.end(), 0);
    std::stable_sort(perm.begin(), perm.end(), [&](int32_t a, int32_t b) { return keys[a] < keys[b]; });
    d->block_table.assign((size_t)n * d->max_pages, -1);
    int64_t off = 0;
    for (int r = 0; r < n; ++r) {
        for (int64_t k = 0; k < need[r]; ++k) d->block_table[(size_t)r * d->max_pages + k] = perm[(size_t)(off + k)];
        off += need[r];
    }
}

// bounded pseudo-random bf16 (uniform on about [-1.73, 1.73], unit variance); timing data only
__global__ void fill_kernel(uint16_t* dst, int64_t n, uint64_t seed) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        uint64_t z = seed + (uint64_t)(i + 1) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z ^= z >> 31;
        const float u = (float)(uint32_t)(z >> 40) * (1.0f / 16777216.0f);  // [0, 1)
        dst[i] = __bfloat16_as_ushort(__float2bfloat16_rn((u - 0.5f) * 3.4641016f));
    }
}

struct DevBuf {
    void* p = nullptr;
    ~DevBuf() { if (p) cudaFree(p); }
    cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 256); }
};

constexpr int64_t kRotateBytes = 320ll << 20;  // rotate small batches over this much KV (> 2 x L2)
constexpr int kMaxRotate = 32;

}  // namespace

}  // namespace ps

using namespace ps;

extern "C" ps_status ps_profile_grid(const ps_shape* shape, const ps_grid_spec* spec, ps_grid_row* rows, int64_t max_rows,
                                     int64_t* n_rows_out, const char* csv_path, void* stream) {
    ps_status st = check_shape(shape);
    if (st != PS_OK) return st;
    if (!spec || !rows || !n_rows_out) return fail(PS_ERR_INVALID, "null argument");
    if (shape->dtype != 0) return fail(PS_ERR_UNSUPPORTED, "the sweep profiles the bf16 cache only");
    if (!spec->chunk_sizes || !spec->decode_counts || !spec->mean_ctxs || spec->n_chunk_sizes < 1 ||
        spec->n_decode_counts < 1 || spec->n_mean_ctxs < 1 || spec->seeds_per_cell < 1 || spec->warmup < 1 || spec->iters < 1)
        return fail(PS_ERR_INVALID, "empty grid axis, or seeds_per_cell / warmup / iters < 1");
    const int64_t n_cells = (int64_t)spec->n_chunk_sizes * spec->n_decode_counts * spec->n_mean_ctxs;
    const int64_t n_rows = n_cells * spec->seeds_per_cell;
    if (max_rows < n_rows) return fail(PS_ERR_INVALID, "max_rows=%lld < %lld rows", (long long)max_rows, (long long)n_rows);
    for (int i = 0; i < spec->n_chunk_sizes; ++i)
        if (spec->chunk_sizes[i] < 0) return fail(PS_ERR_INVALID, "negative chunk size");
    for (int i = 0; i < spec->n_decode_counts; ++i)
        if (spec->decode_counts[i] < 0) return fail(PS_ERR_INVALID, "negative decode count");
    for (int i = 0; i < spec->n_mean_ctxs; ++i)
        if (spec->mean_ctxs[i] < 2) return fail(PS_ERR_INVALID, "mean context must be >= 2");

    const int Hq = shape->n_q_heads, Hkv = shape->n_kv_heads, d = shape->head_dim;
    const size_t page_bytes = (size_t)Hkv * page_head_bytes(d);
    cudaStream_t s = (cudaStream_t)stream;

    // capacity pass: largest pool (with rotation), batch, block table and workspace
    int64_t cap_pages = 0, cap_q = 1, cap_bt = 1;
    {
        Draw dr;
        for (int a = 0; a < spec->n_chunk_sizes; ++a)
            for (int b = 0; b < spec->n_decode_counts; ++b)
                for (int c = 0; c < spec->n_mean_ctxs; ++c) {
                    const int chunk = spec->chunk_sizes[a], nd = spec->decode_counts[b], m = spec->mean_ctxs[c];
                    if (chunk == 0 && nd == 0) return fail(PS_ERR_INVALID, "cell with no rows");
                    // worst case of the length law: every context at 3m/2
                    const int64_t hi = (3LL * m) / 2;
                    int64_t pages = (int64_t)nd * ((hi + kPage - 1) / kPage) + (chunk ? (hi + chunk + kPage - 1) / kPage : 0);
                    pages = std::max<int64_t>((pages * 5 + 3) / 4, pages + 8);
                    const int64_t rot = std::min<int64_t>(kMaxRotate, std::max<int64_t>(1, (kRotateBytes + pages * page_bytes - 1) / (pages * page_bytes)));
                    cap_pages = std::max(cap_pages, pages * rot);
                    cap_q = std::max<int64_t>(cap_q, nd + chunk);
                    const int64_t mp = (hi + chunk + kPage - 1) / kPage;
                    cap_bt = std::max<int64_t>(cap_bt, rot * (nd + 1) * mp);
                }
        (void)dr;
    }
    DevBuf pool_mem, q_mem, out_mem, bt_mem, ws_mem, knew_mem, vnew_mem;
    size_t ws_cap = 0;
    if (pool_mem.alloc((size_t)cap_pages * page_bytes) != cudaSuccess)
        return fail(PS_ERR_OOM, "cannot allocate %zu bytes of KV pool for the sweep", (size_t)cap_pages * page_bytes);
    const size_t q_bytes = (size_t)cap_q * Hq * d * 2;
    if (q_mem.alloc(q_bytes) != cudaSuccess || out_mem.alloc(q_bytes) != cudaSuccess ||
        bt_mem.alloc((size_t)cap_bt * sizeof(int32_t)) != cudaSuccess)
        return fail(PS_ERR_OOM, "cannot allocate sweep buffers");
    const size_t new_bytes = (size_t)cap_q * Hkv * d * 2;  // K (or V) of one batch's new tokens
    if (spec->include_kv_write) {
        if (knew_mem.alloc(new_bytes) != cudaSuccess || vnew_mem.alloc(new_bytes) != cudaSuccess)
            return fail(PS_ERR_OOM, "cannot allocate sweep buffers");
        fill_kernel<<<148, 256, 0, s>>>((uint16_t*)knew_mem.p, (int64_t)(new_bytes / 2), 0x9abc);
        fill_kernel<<<148, 256, 0, s>>>((uint16_t*)vnew_mem.p, (int64_t)(new_bytes / 2), 0xdef0);
    }
    fill_kernel<<<148 * 8, 256, 0, s>>>((uint16_t*)pool_mem.p, (int64_t)((size_t)cap_pages * page_bytes / 2), 0x1234);
    fill_kernel<<<148, 256, 0, s>>>((uint16_t*)q_mem.p, (int64_t)(q_bytes / 2), 0x5678);
    PS_CUDA_TRY(cudaGetLastError());
    PS_CUDA_TRY(cudaStreamSynchronize(s));

    ps_kv* kv = nullptr;
    st = ps_kv_alloc(shape, cap_pages, pool_mem.p, (size_t)cap_pages * page_bytes, &kv);
    if (st != PS_OK) return st;
    ps_plan* plan = nullptr;
    const int n_ev = spec->warmup + spec->iters;
    std::vector<cudaEvent_t> ev0(n_ev), ev1(n_ev);
    for (int i = 0; i < n_ev; ++i) {
        cudaEventCreate(&ev0[i]);
        cudaEventCreate(&ev1[i]);
    }
    auto cleanup = [&]() {
        for (int i = 0; i < n_ev; ++i) {
            cudaEventDestroy(ev0[i]);
            cudaEventDestroy(ev1[i]);
        }
        ps_plan_free(plan);
        ps_kv_free(kv);
    };

    FILE* csv = nullptr;
    if (csv_path) {
        csv = fopen(csv_path, "w");
        if (!csv) {
            cleanup();
            return fail(PS_ERR_INVALID, "cannot open %s for writing", csv_path);
        }
        fprintf(csv, "component,chunk,n_decode,mean_ctx,seed_index,seed,token_batch,prefill_prior,kv_tokens,decode_bytes,"
                     "prefill_flops,latency_us,latency_min_us,latency_max_us,plan_us,decode_TBps,prefill_TFLOPs,roofline_frac\n");
    }

    Draw dr;
    std::vector<int32_t> bt_all;
    std::vector<float> times;
    int64_t row_idx = 0, cell = 0;
    ps_status result = PS_OK;
    for (int a = 0; a < spec->n_chunk_sizes && result == PS_OK; ++a)
        for (int b = 0; b < spec->n_decode_counts && result == PS_OK; ++b)
            for (int c = 0; c < spec->n_mean_ctxs && result == PS_OK; ++c, ++cell)
                for (int sd = 0; sd < spec->seeds_per_cell && result == PS_OK; ++sd) {
                    const int chunk = spec->chunk_sizes[a], nd = spec->decode_counts[b], m = spec->mean_ctxs[c];
                    const uint64_t seed = spec->seed_base + (uint64_t)spec->seeds_per_cell * (uint64_t)cell + (uint64_t)sd;
                    make_draw(chunk, nd, m, seed, &dr);
                    const int n = (int)dr.prior.size();
                    const int64_t rot = std::min<int64_t>(
                        std::min<int64_t>(kMaxRotate, std::max<int64_t>(1, cap_bt / (int64_t)dr.block_table.size())),
                        std::max<int64_t>(1, std::min<int64_t>(cap_pages / dr.num_pages,
                                                                             (kRotateBytes + dr.num_pages * page_bytes - 1) / (dr.num_pages * page_bytes))));
                    bt_all.resize((size_t)rot * dr.block_table.size());
                    for (int64_t k = 0; k < rot; ++k)
                        for (size_t i = 0; i < dr.block_table.size(); ++i)
                            bt_all[(size_t)k * dr.block_table.size() + i] =
                                dr.block_table[i] < 0 ? -1 : (int32_t)(dr.block_table[i] + k * dr.num_pages);
                    cudaError_t e = cudaMemcpyAsync(bt_mem.p, bt_all.data(), bt_all.size() * sizeof(int32_t), cudaMemcpyHostToDevice, s);
                    if (e != cudaSuccess) { result = fail(PS_ERR_CUDA, "block table upload failed: %s", cudaGetErrorString(e)); break; }

                    size_t ws_bytes = 0;
                    const auto t0 = std::chrono::steady_clock::now();
                    result = ps_attn_plan(shape, dr.prior.data(), dr.q_len.data(), n, dr.max_pages, nullptr, &plan, &ws_bytes);
                    const auto t1 = std::chrono::steady_clock::now();
                    if (result != PS_OK) break;
                    if (ws_bytes > ws_cap) {
                        cudaStreamSynchronize(s);
                        if (ws_mem.p) cudaFree(ws_mem.p);
                        ws_mem.p = nullptr;
                        ws_cap = ws_bytes * 2;
                        if (ws_mem.alloc(ws_cap) != cudaSuccess) { result = fail(PS_ERR_OOM, "cannot allocate workspace"); break; }
                    }
                    for (int it = 0; it < n_ev && result == PS_OK; ++it) {
                        const int32_t* bt_k = (const int32_t*)bt_mem.p + (size_t)(it % rot) * dr.block_table.size();
                        cudaEventRecord(ev0[it], s);
                        if (spec->include_kv_write) {
                            result = ps_kv_write(kv, knew_mem.p, vnew_mem.p, bt_k, dr.max_pages, dr.prior.data(), dr.q_len.data(), n, s);
                            if (result != PS_OK) break;
                        }
                        result = ps_attn_run(plan, kv, q_mem.p, bt_k, out_mem.p, nullptr, ws_mem.p, ws_cap, s);
                        cudaEventRecord(ev1[it], s);
                    }
                    if (result != PS_OK) break;
                    result = ps_plan_status(plan, s);
                    if (result != PS_OK) break;
                    times.clear();
                    for (int it = spec->warmup; it < n_ev; ++it) {
                        float ms = 0.f;
                        cudaEventElapsedTime(&ms, ev0[it], ev1[it]);
                        times.push_back(ms * 1000.f);
                    }
                    std::sort(times.begin(), times.end());
                    ps_grid_row& r = rows[row_idx++];
                    r.chunk = chunk;
                    r.n_decode = nd;
                    r.mean_ctx = m;
                    r.seed_index = sd;
                    r.seed = seed;
                    r.token_batch = chunk + nd;
                    r.prefill_prior = dr.prefill_prior;
                    r.kv_tokens = dr.kv_tokens;
                    double dec_tokens = 0;
                    for (int i = 0; i < nd; ++i) dec_tokens += (double)dr.prior[i] + 1.0;
                    r.decode_bytes = dec_tokens * 2.0 * Hkv * d * 2.0;
                    r.prefill_flops = chunk ? 4.0 * d * Hq * ((double)chunk * dr.prefill_prior + 0.5 * chunk * (chunk + 1.0)) : 0.0;
                    r.latency_us = times[times.size() / 2];
                    r.latency_min_us = times.front();
                    r.latency_max_us = times.back();
                    r.plan_us = (float)std::chrono::duration<double, std::micro>(t1 - t0).count();
                    {
                        const double sec = (double)r.latency_us * 1e-6;
                        const double hbm = (spec->hbm_peak_gbs > 0 ? spec->hbm_peak_gbs : 8000.0) * 1e9;
                        const double tensor = (spec->bf16_peak_tflops > 0 ? spec->bf16_peak_tflops : 2250.0) * 1e12;
                        r.decode_TBps = sec > 0 ? (float)(r.decode_bytes / sec / 1e12) : 0.f;
                        r.prefill_TFLOPs = sec > 0 ? (float)(r.prefill_flops / sec / 1e12) : 0.f;
                        r.roofline_frac = sec > 0 ? (float)(std::max(r.decode_bytes / hbm, r.prefill_flops / tensor) / sec) : 0.f;
                    }
                    if (csv)
                        fprintf(csv, "%s,%d,%d,%d,%d,%llu,%d,%d,%lld,%.0f,%.0f,%.3f,%.3f,%.3f,%.3f,%.4f,%.2f,%.4f\n",
                                spec->include_kv_write ? "attn+kv_write" : "attn", r.chunk, r.n_decode,
                                r.mean_ctx, r.seed_index, (unsigned long long)r.seed, r.token_batch, r.prefill_prior,
                                (long long)r.kv_tokens, r.decode_bytes, r.prefill_flops, r.latency_us, r.latency_min_us,
                                r.latency_max_us, r.plan_us, r.decode_TBps, r.prefill_TFLOPs, r.roofline_frac);
                }
    if (csv) fclose(csv);
    cudaStreamSynchronize(s);
    cleanup();
    *n_rows_out = row_idx;
    return result;
}
