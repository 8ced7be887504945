// Host work partitioner and the per-iteration run entry point.
//
// The partition depends on the logical lengths only (never on page ids), so a
// batch produces the same items, the same summation order and therefore the
// same output bits under any assignment of physical pages.
#include <algorithm>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <functional>
#include <iterator>
#include <atomic>
#include <mutex>
#include <new>
#include <unordered_map>
#include <utility>
#include <vector>

#include "common.cuh"

namespace ps {

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr int kDecodeUnitsPerWarp = 1;  // work units per resident warp (measured: 1 beats 2 and 3 on the decode-only batch)
// Smallest decode unit (pages) of a batch too small to give every warp its share: between 4 and 8, so that the
// longest row is cut into about 16 pieces at most.  Finer cuts spread a small batch over more warps (64 rows of
// 64 tokens: 13 us instead of 20; 8 rows of 512: 16 instead of 23), but every further piece of a row is one more
// partial result for the one warp that combines them (one row of 4096 tokens: 22 us at 32 pieces, 26 at 64).
constexpr int kDecodeMinPagesLo = 4, kDecodeMinPagesHi = 8, kDecodePiecesPerRow = 16;
constexpr int kPrefillKeyTile = 128;    // keys per tensor-core tile
// Measured on B200 (decode: bandwidth against the number of SMs the kernel runs on; prefill: time of one
// key-tile step of a q tile pair), used to split the SMs of a mixed batch between the two kernels.
constexpr double kDecodePeakBytesPerSec = 6.7e12;
constexpr double kDecodeSharedPeakBytesPerSec = 6.0e12;  // decode rows beside a running prefill kernel
constexpr double kDecodeBytesPerSecPerSm = 115e9;
constexpr double kDecodeAloneBytesPerSecPerSm = 135e9;  // per SM with the memory system to itself
constexpr double kPrefillStepSec = 2.5e-6;
constexpr double kKernelFloorSec = 12e-6;

// A chunk of a few tokens runs as that many decode rows (token i of the chunk is a row that sees prior + i + 1 keys
// of the same sequence) instead of bringing in the prefill kernel for one small item: its launch and pipeline fill
// cost more than re-reading a short context a few times.  Bounded by the bytes the rows re-read, and only in batches
// whose decode rows are few: beside a long decode kernel the prefill kernel of a small chunk is hidden anyway.
// (measured: a 2-token chunk on 2048 tokens beside 8 decode rows of 512: 23.8 us instead of 29.8; 8 tokens on 900
// alone 16.4 instead of 22.6; 4 tokens on 1500 beside 128 rows of 2048 would be 169 instead of 165)
constexpr int kTinyChunkTokens = 8;
constexpr double kTinyChunkBytes = 32e6;
constexpr double kTinyChunkMaxDecodeBytes = 128e6;
static inline bool runs_as_decode(const ps_shape& sh, bool tiny_as_rows, int prior, int q_len) {
    if (q_len == 1) return true;
    if (!tiny_as_rows || q_len > kTinyChunkTokens) return false;
    return (double)q_len * ((double)prior + q_len) * 2.0 * sh.n_kv_heads * sh.head_dim * 2.0 <= kTinyChunkBytes;
}

}  // namespace ps

using namespace ps;

namespace {

// Which plan last put a work list into a given workspace.  Two plans that take turns on one workspace (or on the
// built-in scratch of ps_attn_run_static) each keep their own record of the slots they have used; a plan that finds
// another plan's serial here orders its upload behind everything already on the caller's stream instead of trusting
// that record.
std::mutex g_ws_mu;
std::unordered_map<const void*, uint64_t> g_ws_owner;
constexpr size_t kWsOwnerCap = 4096;  // forgetting an entry only costs its next run one stream fence

uint64_t next_plan_serial() {
    static std::atomic<uint64_t> next{1};
    return next.fetch_add(1, std::memory_order_relaxed);
}

// true if `serial` was already the last user of `ws`; records it as the last user either way
bool claim_workspace(const void* ws, uint64_t serial) {
    std::lock_guard<std::mutex> lock(g_ws_mu);
    auto it = g_ws_owner.find(ws);
    if (it != g_ws_owner.end()) {
        const bool same = it->second == serial;
        it->second = serial;
        return same;
    }
    if (g_ws_owner.size() >= kWsOwnerCap) g_ws_owner.clear();
    g_ws_owner.emplace(ws, serial);
    return false;
}

void forget_plan(uint64_t serial) {
    std::lock_guard<std::mutex> lock(g_ws_mu);
    for (auto it = g_ws_owner.begin(); it != g_ws_owner.end();)
        it = it->second == serial ? g_ws_owner.erase(it) : std::next(it);
}

}  // namespace

struct ps_plan {
    ps_shape shape{};
    int32_t n = 0, max_pages = 0, num_sms = 0, device_sms = 0;
    // SMs given to each kernel: all of them when only one class of rows is present; in a mixed batch the
    // decode kernel (HBM-bound: a fraction of the SMs saturates the memory system) and the prefill kernel
    // (tensor-bound) run side by side on disjoint sets of SMs
    int32_t dec_sms = 0, pf_sms = 0;
    bool concurrent = false;
    bool tiny_as_rows = false;  // this batch runs its chunks of a few tokens as decode rows
    std::vector<DecodePiece> pieces;
    std::vector<DecodeUnit> units;
    std::vector<PrefillItem> prefill;
    std::vector<MergeEntry> merge;       // prefill q tile pairs cut into segments: combined by the merge kernel
    std::vector<DecodeMerge> dmerge;     // combined inside the decode kernel
    int64_t decode_merge_rows = 0;
    std::vector<int32_t> prefill_cta_start;  // static partition: CTA b runs items [start[b], start[b+1]); empty = dynamic queue
    std::vector<int32_t> prior;  // kept for item inspection
    ps_plan_info info{};
    // workspace layout: two image slots of slot_stride bytes each, then the partial rows.  The stride only ever
    // grows (with headroom), so that re-planning to another batch normally leaves the slots and the partial
    // buffers where the runs still in flight expect them.
    size_t off_pieces = 0, off_units = 0, off_prefill = 0, off_merge = 0, off_cta_start = 0, off_dmerge = 0, off_dmerge_cnt = 0, image_bytes = 0;
    size_t slot_stride = 0;
    size_t off_part_lse = 0, off_part_o = 0, ws_bytes = 0;
    bool layout_moved = false;  // slot_stride grew since the last run: the slots of earlier runs lie elsewhere
    uint64_t serial = 0;        // identifies this plan object among all that may share a workspace
    int64_t wait_limit_ns = kDefaultWaitLimitNs;  // bound of every device-side wait of this plan's kernels
    // pinned staging image of [0, image_bytes)
    char* pinned = nullptr;
    bool pinned_is_cuda = false;
    size_t pinned_cap = 0;
    // The work-list image is uploaded on a private stream into one of two slots at the head of the
    // workspace, so that the upload for run i+1 overlaps the kernels of run i.
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr};  // slot's upload finished (copy stream)
    cudaEvent_t ev_done[2] = {nullptr, nullptr};    // the run that used the slot finished (caller's stream)
    cudaEvent_t ev_fence = nullptr;                  // caller's stream position, when the workspace changed
    cudaStream_t side_stream = nullptr;              // decode kernel of a mixed batch (runs beside the prefill kernel)
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    bool done_valid[2] = {false, false};
    bool copy_pending = false;
    int last_slot = 0;
    unsigned run_no = 0;
    void* last_ws = nullptr;
    WsHeader* last_hdr = nullptr;
    // optional per-kernel timing: 6 events per recorded run (begin/end of prefill, decode, merge)
    bool timing = false;
    std::vector<cudaEvent_t> tev;
    int timed_runs = 0;
};

static int query_num_sms() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return sms;
}

static void plan_decode(ps_plan* pl, const int32_t* prior, const int32_t* q_len, const std::vector<int32_t>& q_start,
                        const ps_plan_opts* opts, int64_t* n_slots) {
    const int Hkv = pl->shape.n_kv_heads, G = pl->shape.n_q_heads / Hkv;
    int64_t total_pages = 0, longest = 0;
    for (int r = 0; r < pl->n; ++r)
        if (runs_as_decode(pl->shape, pl->tiny_as_rows, prior[r], q_len[r]))
            for (int i = 0; i < q_len[r]; ++i) {
                const int64_t pages = (prior[r] + i + 1 + kPage - 1) / kPage;
                total_pages += pages * Hkv;
                longest = std::max(longest, pages);
            }
    if (total_pages == 0) {
        pl->pieces.clear();
        pl->units.clear();
        pl->dmerge.clear();
        return;
    }
    const int64_t min_pages = std::min<int64_t>(kDecodeMinPagesHi, std::max<int64_t>(kDecodeMinPagesLo, (longest + kDecodePiecesPerRow - 1) / kDecodePiecesPerRow));
    int64_t per_unit;
    if (opts && opts->decode_segment_tokens > 0) {
        per_unit = std::max(1, opts->decode_segment_tokens / kPage);
    } else {
        const int64_t target = (int64_t)pl->dec_sms * decode_warps_per_sm() * kDecodeUnitsPerWarp;
        per_unit = std::max<int64_t>(min_pages, (total_pages + target - 1) / target);
    }
    pl->info.decode_segment_tokens = (int32_t)(per_unit * kPage);

    // Upper bounds on the counts (a piece ends where its row or its unit ends), so that the lists are filled
    // in place and trimmed once.
    int64_t n_rows = 0;
    for (int r = 0; r < pl->n; ++r) n_rows += runs_as_decode(pl->shape, pl->tiny_as_rows, prior[r], q_len[r]) ? (int64_t)q_len[r] * Hkv : 0;
    const size_t max_units = (size_t)((total_pages + per_unit - 1) / per_unit);
    pl->pieces.resize((size_t)n_rows + max_units);
    pl->units.resize(max_units);
    pl->dmerge.resize(std::min<size_t>((size_t)n_rows, max_units));
    DecodePiece* const pieces = pl->pieces.data();
    DecodeUnit* const units = pl->units.data();
    DecodeMerge* const dmerge = pl->dmerge.data();
    int32_t n_pieces = 0, n_units = 0, n_dmerge = 0;
    int64_t slots = *n_slots;
    int64_t room = 0;  // pages the open unit can still take
    for (int r = 0; r < pl->n; ++r) {
        if (!runs_as_decode(pl->shape, pl->tiny_as_rows, prior[r], q_len[r])) continue;
        for (int i = 0; i < q_len[r]; ++i) {  // one row per new token (a decode request has one)
            const int kv_len = prior[r] + i + 1;
            const int pages = (kv_len + kPage - 1) / kPage;
            const int32_t q_tok = q_start[r] + i;
            for (int g = 0; g < Hkv; ++g) {
                const int32_t first_piece = n_pieces;
                int pg = 0;
                while (pg < pages) {
                    if (room == 0) {
                        if (n_units > 0) units[n_units - 1].piece_end = n_pieces;
                        units[n_units++].piece_begin = n_pieces;
                        room = per_unit;
                    }
                    const int take = (int)std::min<int64_t>(room, pages - pg);
                    DecodePiece& pc = pieces[n_pieces++];
                    pc.req = r;
                    pc.kv_head = g;
                    pc.page_begin = pg;
                    pc.page_end = pg + take;
                    pc.q_tok = q_tok;
                    pc.part_slot = -1;
                    pc.kv_len = kv_len;
                    pc.merge_idx = 0;
                    pg += take;
                    room -= take;
                }
                const int32_t cnt = n_pieces - first_piece;
                if (cnt > 1) {
                    for (int32_t s = 0; s < cnt; ++s) {
                        pieces[first_piece + s].part_slot = (int32_t)(slots + (int64_t)s * G);
                        pieces[first_piece + s].merge_idx = n_dmerge;
                    }
                    dmerge[n_dmerge].base = (int32_t)slots;
                    dmerge[n_dmerge].n_seg = cnt;
                    ++n_dmerge;
                    slots += (int64_t)cnt * G;
                }
            }
        }
    }
    if (n_units > 0) units[n_units - 1].piece_end = n_pieces;
    pl->pieces.resize((size_t)n_pieces);
    pl->units.resize((size_t)n_units);
    pl->dmerge.resize((size_t)n_dmerge);
    pl->decode_merge_rows += (int64_t)n_dmerge * G;
    *n_slots = slots;
}

// Cost model of the prefill kernel in units of one 128-key tile step: an item pays a fixed
// overhead (pipeline fill, output) plus one unit per key tile.
// (fitted to per-CTA run times on B200: 2.2 us per step, about 3 us per item, 1.2 us more for a masked tile)
constexpr double kPrefillFixedCost = 1.5;
constexpr double kPrefillMaskedExtra = 0.5;  // the diagonal tile of an item takes the slower masked softmax
constexpr double kPrefillCutCost = 3.0;
constexpr double kPrefillWholeItemSlack = 1.12;  // uncut items are taken if the busiest CTA stays within this of an even split
constexpr double kPrefillMinCtaCost = 4.0;  // do not spread the work thinner than this per CTA (two key tiles)

static void plan_prefill(ps_plan* pl, const int32_t* prior, const int32_t* q_len, const std::vector<int32_t>& q_start,
                         const ps_plan_opts* opts, int64_t* n_slots) {
    const int Hkv = pl->shape.n_kv_heads, G = pl->shape.n_q_heads / Hkv;
    const int tile_tok = kPrefillRowsPerItem / G;
    struct Tile { int r, g, tok0, n_tok, first_pos, key_tiles; };
    std::vector<Tile> tiles;
    size_t n_tiles = 0;
    for (int r = 0; r < pl->n; ++r)
        if (!runs_as_decode(pl->shape, pl->tiny_as_rows, prior[r], q_len[r])) n_tiles += (size_t)((q_len[r] + tile_tok - 1) / tile_tok) * Hkv;
    tiles.reserve(n_tiles);
    int64_t total_key_tiles = 0;
    for (int r = 0; r < pl->n; ++r) {
        if (runs_as_decode(pl->shape, pl->tiny_as_rows, prior[r], q_len[r])) continue;
        for (int g = 0; g < Hkv; ++g)
            for (int t0 = 0; t0 < q_len[r]; t0 += tile_tok) {
                const int n_tok = std::min(tile_tok, q_len[r] - t0);
                const int first_pos = prior[r] + t0;
                const int kt = (first_pos + n_tok + kPrefillKeyTile - 1) / kPrefillKeyTile;
                tiles.push_back(Tile{r, g, t0, n_tok, first_pos, kt});
                total_key_tiles += kt;
            }
    }
    pl->prefill_cta_start.clear();
    if (tiles.empty()) return;

    // (tile, key-tile index) of every cut, ascending in both: tile i is cut into pieces at these key tiles
    // (exclusive of 0 and key_tiles)
    struct Cut { int tile, at; };
    std::vector<Cut> cuts;
    // owner CTA of the first piece of each tile and of each following piece, for the static partition
    bool static_partition = false, whole_items = false;
    if (opts && opts->prefill_segment_tokens > 0) {
        const int seg_tiles = std::max(1, opts->prefill_segment_tokens / kPrefillKeyTile);
        pl->info.prefill_segment_tokens = seg_tiles * kPrefillKeyTile;
        for (size_t i = 0; i < tiles.size(); ++i) {
            const int n_seg = (tiles[i].key_tiles + seg_tiles - 1) / seg_tiles;
            const int base_tiles = tiles[i].key_tiles / n_seg, extra = tiles[i].key_tiles % n_seg;
            int kt0 = 0;
            for (int s = 0; s + 1 < n_seg; ++s) {
                kt0 += base_tiles + (s < extra ? 1 : 0);
                cuts.push_back(Cut{(int)i, kt0});
            }
        }
    } else if ((int64_t)tiles.size() < 4LL * pl->pf_sms) {
        // Few items per SM: give every CTA an equal share of the flattened (item, key tile) cost
        // line, cutting items where a share ends.  Only the cut items need the merge.
        static_partition = true;
        double total = 0;
        for (const Tile& t : tiles) total += kPrefillFixedCost + t.key_tiles + kPrefillMaskedExtra;
        const int n_cta = (int)std::max<double>(1, std::min<double>(pl->pf_sms, total / kPrefillMinCtaCost));
        // Many short items (fresh prompts): whole items, longest first, each to the CTA with the least work so far.
        // If that comes within kPrefillWholeItemSlack of an even split, nothing is cut: no partial rows, no merge
        // kernel, no item paying its fixed cost twice.
        {
            std::vector<int> order(tiles.size());
            for (size_t i = 0; i < tiles.size(); ++i) order[i] = (int)i;
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return tiles[a].key_tiles > tiles[b].key_tiles; });
            // (least work so far, CTA): equal loads go to the lower CTA
            typedef std::pair<double, int> Slot;
            std::vector<Slot> heap((size_t)n_cta);
            for (int c = 0; c < n_cta; ++c) heap[c] = Slot(0.0, c);  // ascending: already a min-heap under greater<>
            std::vector<int> owner(tiles.size());
            std::vector<int32_t> count((size_t)n_cta + 1, 0);
            double makespan = 0;
            for (int i : order) {
                std::pop_heap(heap.begin(), heap.end(), std::greater<Slot>());
                Slot& least = heap.back();
                owner[i] = least.second;
                ++count[least.second + 1];
                least.first += kPrefillFixedCost + tiles[i].key_tiles + kPrefillMaskedExtra;
                makespan = std::max(makespan, least.first);
                std::push_heap(heap.begin(), heap.end(), std::greater<Slot>());
            }
            // (cutting is not free either: the merge kernel and the partial rows cost about kPrefillCutCost steps)
            if (makespan <= std::max(kPrefillWholeItemSlack * total / n_cta, total / n_cta + kPrefillCutCost)) {
                for (int c = 0; c < n_cta; ++c) count[c + 1] += count[c];
                pl->prefill_cta_start.assign(count.begin(), count.end());
                std::vector<Tile> sorted(tiles.size());
                for (int i : order) sorted[(size_t)count[owner[i]]++] = tiles[i];  // each CTA's items longest first
                tiles.swap(sorted);
                whole_items = true;
            }
        }
        if (!whole_items) {
        // CTA k ends where the running cost passes (k + 1) * quota (absolute marks, so rounding does not pile
        // up).  A share that ends inside an item makes the rest of that item pay the fixed cost again, and how
        // many shares do depends on the quota itself: bisect for the smallest quota that does not leave the
        // last CTA with more than a share.
        int n_items = 0;
        double q_lo = total / n_cta, q_hi = (total + (n_cta - 1) * kPrefillFixedCost) / n_cta + 0.5;
        for (int pass = 0; pass < 7; ++pass) {
            const double quota = pass == 6 ? q_hi : 0.5 * (q_lo + q_hi);  // the last pass keeps a quota known to fit
            pl->prefill_cta_start.assign(1, 0);
            cuts.clear();
            n_items = 0;
            int cta = 0;
            double cum = 0, cum_at_last = 0;  // cost handed out so far; and before the last CTA
            auto close_cta = [&]() {
                ++cta;
                pl->prefill_cta_start.push_back(n_items);
                if (cta == n_cta - 1) cum_at_last = cum;
            };
            for (size_t i = 0; i < tiles.size(); ++i) {
                const int kt = tiles[i].key_tiles;
                int kt0 = 0;
                for (;;) {
                    const double rest = kPrefillFixedCost + (kt - kt0) + kPrefillMaskedExtra;  // the item's remaining tiles as one piece
                    const double room = (cta + 1) * quota - cum;
                    const bool cta_has_work = pl->prefill_cta_start.back() < n_items;
                    const double fit = room - kPrefillFixedCost;
                    const int take = fit < 0.5 ? 0 : (int)(fit + 0.5);  // key tiles that fit, to the nearest
                    if (cta == n_cta - 1 || rest <= room + 0.5 || take >= kt - kt0 || (take < 1 && !cta_has_work)) {
                        cum += rest;
                        ++n_items;
                        break;
                    }
                    if (take >= 1) {
                        kt0 += take;
                        cuts.push_back(Cut{(int)i, kt0});
                        cum += kPrefillFixedCost + take;
                        ++n_items;
                    }
                    close_cta();  // (with take < 1: no room left for even one key tile; the item starts in the next CTA)
                }
                while (cta < n_cta - 1 && cum >= (cta + 1) * quota - 0.5) close_cta();
            }
            const bool fits = cta < n_cta - 1 || cum - cum_at_last <= quota + 0.5;
            if (fits) q_hi = quota; else q_lo = quota;
        }
        while ((int)pl->prefill_cta_start.size() < n_cta) pl->prefill_cta_start.push_back(n_items);  // CTAs left without work
        pl->prefill_cta_start.push_back(n_items);
        }
    }

    pl->prefill.reserve(tiles.size() + cuts.size());
    size_t next_cut = 0;
    for (size_t i = 0; i < tiles.size(); ++i) {
        const Tile& t = tiles[i];
        const size_t first_cut = next_cut;
        while (next_cut < cuts.size() && cuts[next_cut].tile == (int)i) ++next_cut;
        const int n_seg = (int)(next_cut - first_cut) + 1;
        const int visible = t.first_pos + t.n_tok;
        int32_t slot_base = -1;
        if (n_seg > 1) {
            slot_base = (int32_t)*n_slots;
            MergeEntry me{};
            me.q_tok = q_start[t.r] + t.tok0;
            me.n_tok = t.n_tok;
            me.kv_head = t.g;
            me.base = slot_base;
            me.n_seg = n_seg;
            me.seg_stride = t.n_tok * G;
            pl->merge.push_back(me);
            *n_slots += (int64_t)n_seg * t.n_tok * G;
        }
        for (int s = 0; s < n_seg; ++s) {
            const int kt0 = s == 0 ? 0 : cuts[first_cut + s - 1].at;
            const int kt1 = s == n_seg - 1 ? t.key_tiles : cuts[first_cut + s].at;
            PrefillItem it{};
            it.req = t.r;
            it.kv_head = t.g;
            it.key_begin = kt0 * kPrefillKeyTile;
            it.key_end = std::min(visible, kt1 * kPrefillKeyTile);
            it.q_tok = q_start[t.r] + t.tok0;
            it.n_tok = t.n_tok;
            it.part_slot = n_seg > 1 ? slot_base + s * t.n_tok * G : -1;
            it.first_pos = t.first_pos;
            pl->prefill.push_back(it);
        }
    }
    if (!static_partition) {
        // dynamic queue: longest first, so that it finishes with the short items
        std::stable_sort(pl->prefill.begin(), pl->prefill.end(), [](const PrefillItem& a, const PrefillItem& b) {
            return (a.key_end - a.key_begin) > (b.key_end - b.key_begin);
        });
    }
}

extern "C" {

ps_status ps_attn_plan(const ps_shape* shape, const int32_t* prior_host, const int32_t* q_len_host, int32_t n,
                       int32_t max_pages_per_seq, const ps_plan_opts* opts, ps_plan** plan_inout,
                       size_t* workspace_bytes_out) {
    ps_status st = check_shape(shape);
    if (st != PS_OK) return st;
    if (!prior_host || !q_len_host || !plan_inout || !workspace_bytes_out) return fail(PS_ERR_INVALID, "null argument");
    if (n < 1) return fail(PS_ERR_INVALID, "n=%d must be positive", n);
    if (max_pages_per_seq < 1) return fail(PS_ERR_INVALID, "max_pages_per_seq=%d must be positive", max_pages_per_seq);
    if (opts && (opts->decode_segment_tokens < 0 || opts->decode_segment_tokens % kPage != 0))
        return fail(PS_ERR_INVALID, "decode_segment_tokens must be a non-negative multiple of %d", kPage);
    if (opts && (opts->prefill_segment_tokens < 0 || opts->prefill_segment_tokens % kPrefillKeyTile != 0))
        return fail(PS_ERR_INVALID, "prefill_segment_tokens must be a non-negative multiple of %d", kPrefillKeyTile);
    std::vector<int32_t> q_start((size_t)n + 1);
    int64_t T = 0;
    for (int r = 0; r < n; ++r) {
        if (q_len_host[r] < 1) return fail(PS_ERR_INVALID, "request %d: q_len=%d must be >= 1", r, q_len_host[r]);
        if (prior_host[r] < 0) return fail(PS_ERR_INVALID, "request %d: prior=%d must be >= 0", r, prior_host[r]);
        if ((int64_t)prior_host[r] + q_len_host[r] > (int64_t)max_pages_per_seq * kPage)
            return fail(PS_ERR_INVALID, "request %d: kv_len=%lld exceeds max_pages_per_seq * page_size", r,
                        (long long)prior_host[r] + q_len_host[r]);
        if (shape->dtype == 1 && q_len_host[r] != 1)
            return fail(PS_ERR_UNSUPPORTED, "request %d: q_len=%d -- the FP8 cache variant serves decode rows (q_len = 1) only", r,
                        q_len_host[r]);
        q_start[r] = (int32_t)T;
        T += q_len_host[r];
        if (T > (1 << 24)) return fail(PS_ERR_INVALID, "more than 2^24 new tokens in one batch");
    }
    q_start[n] = (int32_t)T;

    ps_plan* pl = *plan_inout;
    const bool fresh = pl == nullptr;
    if (fresh) {
        pl = new (std::nothrow) ps_plan();
        if (!pl) return fail(PS_ERR_OOM, "host allocation failed");
        pl->serial = next_plan_serial();
    } else if (pl->copy_pending && pl->ev_copied[pl->last_slot]) {
        cudaError_t e = cudaEventSynchronize(pl->ev_copied[pl->last_slot]);
        if (e != cudaSuccess) return fail(PS_ERR_CUDA, "cudaEventSynchronize failed: %s", cudaGetErrorString(e));
        pl->copy_pending = false;
    }
    pl->shape = *shape;
    pl->n = n;
    pl->max_pages = max_pages_per_seq;
    if (opts && opts->num_sms > 0) {
        pl->num_sms = opts->num_sms;
    } else {
        if (pl->device_sms <= 0) pl->device_sms = query_num_sms();
        pl->num_sms = pl->device_sms;
    }
    if (pl->num_sms <= 0) {
        if (fresh) delete pl;
        return fail(PS_ERR_CUDA, "no CUDA device to plan for (pass opts->num_sms to plan without one)");
    }
    pl->prefill.clear();
    pl->merge.clear();
    pl->decode_merge_rows = 0;
    pl->prior.assign(prior_host, prior_host + n);
    pl->info = ps_plan_info{};
    {
        double true_dec_bytes = 0;
        for (int r = 0; r < n; ++r)
            if (q_len_host[r] == 1) true_dec_bytes += ((double)prior_host[r] + 1.0) * 2.0 * shape->n_kv_heads * shape->head_dim * 2.0;
        // (forced prefill segments: the caller wants every chunk on the prefill kernel)
        pl->tiny_as_rows = !(opts && opts->prefill_segment_tokens > 0) && true_dec_bytes <= kTinyChunkMaxDecodeBytes;
    }
    // ---- split the SMs between the two kernels of a mixed batch ----
    {
        double dec_bytes = 0, pf_steps = 0;  // KV bytes the decode rows stream; key-tile steps of the prefill items
        const int G = shape->n_q_heads / shape->n_kv_heads;
        const int tile_tok = kPrefillRowsPerItem / G;
        for (int r = 0; r < n; ++r) {
            if (runs_as_decode(*shape, pl->tiny_as_rows, prior_host[r], q_len_host[r])) {
                for (int i = 0; i < q_len_host[r]; ++i)
                    dec_bytes += ((double)prior_host[r] + i + 1.0) * 2.0 * shape->n_kv_heads * shape->head_dim * 2.0;
            } else {
                for (int t0 = 0; t0 < q_len_host[r]; t0 += tile_tok) {
                    const int n_tok = std::min(tile_tok, q_len_host[r] - t0);
                    pf_steps += (kPrefillFixedCost + (prior_host[r] + t0 + n_tok + kPrefillKeyTile - 1) / kPrefillKeyTile) * shape->n_kv_heads;
                }
            }
        }
        pl->dec_sms = pl->pf_sms = pl->num_sms;
        pl->concurrent = false;
        if (dec_bytes > 0 && pf_steps > 0 && pl->num_sms >= 16) {
            // time models (seconds): decode = bytes / min(side-by-side peak, n * per-SM rate); prefill = steps * step time / m
            auto t_dec = [&](int nd) { return dec_bytes / std::min(kDecodeSharedPeakBytesPerSec, nd * kDecodeBytesPerSecPerSm) + kKernelFloorSec; };
            auto t_pf = [&](int nd) { return pf_steps * kPrefillStepSec / (pl->num_sms - nd) + kKernelFloorSec; };
            int best_n = 0;
            double best_t = 1e30;
            for (int nd = 8; nd <= pl->num_sms - 8; nd += 4) {
                const double t = std::max(t_dec(nd), t_pf(nd));
                if (t < best_t) {
                    best_t = t;
                    best_n = nd;
                }
            }
            // Once the decode rows saturate HBM the modelled time is flat in n; measured step times keep
            // improving a little as the decode kernel gets more SMs, as long as the prefill kernel still ends
            // well before it.  Take the middle of that flat stretch.
            int hi = best_n;
            for (int nd = best_n; nd <= pl->num_sms - 8; nd += 4)
                if (std::max(t_dec(nd), t_pf(nd)) <= 1.015 * best_t && t_pf(nd) <= 0.8 * t_dec(nd)) hi = nd;
            best_n = (best_n + hi) / 2 / 4 * 4;
            const double t_seq = dec_bytes / kDecodePeakBytesPerSec + pf_steps * kPrefillStepSec / pl->num_sms + 2 * kKernelFloorSec;
            // The decode rows pay the shared rate only while the prefill kernel runs; once it has ended they stream
            // at the rate their CTAs reach alone.  A short chunk beside many decode rows is therefore cheaper than
            // the model above says, which matters for the choice against running the two one after the other.
            if (best_n > 0) {
                const double pf_work = pf_steps * kPrefillStepSec / (pl->num_sms - best_n);
                const double shared = std::min(kDecodeSharedPeakBytesPerSec, best_n * kDecodeBytesPerSecPerSm);
                const double alone = std::min(kDecodePeakBytesPerSec, best_n * kDecodeAloneBytesPerSecPerSm);
                const double dec_work = dec_bytes <= shared * pf_work ? dec_bytes / shared : pf_work + (dec_bytes - shared * pf_work) / alone;
                best_t = std::min(best_t, std::max(pf_work, dec_work) + kKernelFloorSec);
            }
            if (best_n > 0 && best_t < 0.95 * t_seq) {
                pl->dec_sms = best_n;
                pl->pf_sms = pl->num_sms - best_n;
                pl->concurrent = true;
            }
        }
    }
    int64_t n_slots = 0;
    plan_decode(pl, prior_host, q_len_host, q_start, opts, &n_slots);
    plan_prefill(pl, prior_host, q_len_host, q_start, opts, &n_slots);
    if (n_slots > 0x7fffffffLL) {
        if (fresh) delete pl;
        return fail(PS_ERR_UNSUPPORTED, "partial buffer would need %lld slots", (long long)n_slots);
    }

    const int d = shape->head_dim;
    size_t off = 256;  // WsHeader
    pl->off_pieces = off;   off = align_up(off + pl->pieces.size() * sizeof(DecodePiece), 256);
    pl->off_units = off;    off = align_up(off + pl->units.size() * sizeof(DecodeUnit), 256);
    pl->off_prefill = off;  off = align_up(off + pl->prefill.size() * sizeof(PrefillItem), 256);
    pl->off_merge = off;    off = align_up(off + pl->merge.size() * sizeof(MergeEntry), 256);
    pl->off_dmerge = off;   off = align_up(off + pl->dmerge.size() * sizeof(DecodeMerge), 256);
    pl->off_dmerge_cnt = off; off = align_up(off + pl->dmerge.size() * sizeof(int32_t), 256);
    pl->off_cta_start = off; off = align_up(off + pl->prefill_cta_start.size() * sizeof(int32_t), 256);
    pl->image_bytes = off;
    if (pl->image_bytes > pl->slot_stride) {
        // (re)size the slots with headroom: a batch of the next iterations that needs a somewhat longer work list
        // still fits, and the layout stays put
        pl->slot_stride = align_up(pl->image_bytes + pl->image_bytes / 2, 4096);
        pl->layout_moved = true;
    }
    off = 2 * pl->slot_stride;  // two image slots
    pl->off_part_lse = off; off = align_up(off + (size_t)n_slots * sizeof(float), 256);
    pl->off_part_o = off;   off = align_up(off + (size_t)n_slots * d * sizeof(float), 256);
    pl->ws_bytes = off;

    if (pl->pinned_cap < pl->image_bytes) {
        if (pl->pinned) { if (pl->pinned_is_cuda) cudaFreeHost(pl->pinned); else free(pl->pinned); }
        pl->pinned = nullptr;
        const size_t cap = std::max(pl->image_bytes * 2, (size_t)1 << 16);
        // Page-locked staging lets the work-list upload run asynchronously.  Without a CUDA
        // device (planning ahead of time on another host) plain memory holds the image.
        pl->pinned_is_cuda = cudaHostAlloc((void**)&pl->pinned, cap, cudaHostAllocDefault) == cudaSuccess;
        if (!pl->pinned_is_cuda) {
            (void)cudaGetLastError();
            pl->pinned = (char*)malloc(cap);
        }
        if (!pl->pinned) {
            pl->pinned_cap = 0;
            if (fresh) delete pl;
            return fail(PS_ERR_OOM, "cannot allocate %zu bytes of staging memory", cap);
        }
        pl->pinned_cap = cap;
    }
    if (!pl->copy_stream && pl->pinned_is_cuda) {
        bool ok = cudaStreamCreateWithFlags(&pl->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
        for (int b = 0; b < 2 && ok; ++b)
            ok = cudaEventCreateWithFlags(&pl->ev_copied[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&pl->ev_done[b], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&pl->ev_fence, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&pl->side_stream, cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&pl->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&pl->ev_join, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            (void)cudaGetLastError();
            if (pl->copy_stream) cudaStreamDestroy(pl->copy_stream);
            pl->copy_stream = nullptr;  // uploads then go on the caller's stream
            if (pl->side_stream) cudaStreamDestroy(pl->side_stream);
            pl->side_stream = nullptr;  // mixed batches then run their two kernels one after the other
        }
    }
    memset(pl->pinned, 0, 256);
    if (!pl->pieces.empty()) memcpy(pl->pinned + pl->off_pieces, pl->pieces.data(), pl->pieces.size() * sizeof(DecodePiece));
    if (!pl->units.empty()) memcpy(pl->pinned + pl->off_units, pl->units.data(), pl->units.size() * sizeof(DecodeUnit));
    if (!pl->prefill.empty()) memcpy(pl->pinned + pl->off_prefill, pl->prefill.data(), pl->prefill.size() * sizeof(PrefillItem));
    if (!pl->merge.empty()) memcpy(pl->pinned + pl->off_merge, pl->merge.data(), pl->merge.size() * sizeof(MergeEntry));
    if (!pl->dmerge.empty()) {
        memcpy(pl->pinned + pl->off_dmerge, pl->dmerge.data(), pl->dmerge.size() * sizeof(DecodeMerge));
        memset(pl->pinned + pl->off_dmerge_cnt, 0, pl->dmerge.size() * sizeof(int32_t));  // arrival counters start at zero
    }
    if (!pl->prefill_cta_start.empty())
        memcpy(pl->pinned + pl->off_cta_start, pl->prefill_cta_start.data(), pl->prefill_cta_start.size() * sizeof(int32_t));

    pl->info.n_decode_items = (int32_t)pl->pieces.size();
    pl->info.n_prefill_items = (int32_t)pl->prefill.size();
    int64_t merge_rows = pl->decode_merge_rows;
    for (const MergeEntry& me : pl->merge) merge_rows += (int64_t)me.n_tok * (shape->n_q_heads / shape->n_kv_heads);
    pl->info.n_merge_rows = (int32_t)merge_rows;
    pl->info.n_partial_slots = n_slots;
    pl->info.total_q_tokens = T;
    pl->info.decode_sms = pl->dec_sms;
    pl->info.prefill_sms = pl->pf_sms;
    pl->info.n_launches = (pl->concurrent && !pl->units.empty() && pl->prefill_cta_start.empty() && (int)pl->prefill.size() > pl->pf_sms ? 1 : 0) + (pl->units.empty() ? 0 : 1) + (pl->prefill.empty() ? 0 : 1) + (pl->merge.empty() ? 0 : 1);
    *plan_inout = pl;
    *workspace_bytes_out = pl->ws_bytes;
    return PS_OK;
}

ps_status ps_plan_free(ps_plan* pl) {
    if (!pl) return PS_OK;
    forget_plan(pl->serial);
    if (pl->copy_stream) {
        cudaStreamSynchronize(pl->copy_stream);
        cudaStreamDestroy(pl->copy_stream);
    }
    for (int b = 0; b < 2; ++b) {
        if (pl->ev_copied[b]) cudaEventDestroy(pl->ev_copied[b]);
        if (pl->ev_done[b]) cudaEventDestroy(pl->ev_done[b]);
    }
    if (pl->ev_fence) cudaEventDestroy(pl->ev_fence);
    if (pl->side_stream) {
        cudaStreamSynchronize(pl->side_stream);
        cudaStreamDestroy(pl->side_stream);
    }
    if (pl->ev_fork) cudaEventDestroy(pl->ev_fork);
    if (pl->ev_join) cudaEventDestroy(pl->ev_join);
    for (cudaEvent_t e : pl->tev) cudaEventDestroy(e);
    if (pl->pinned) { if (pl->pinned_is_cuda) cudaFreeHost(pl->pinned); else free(pl->pinned); }
    delete pl;
    return PS_OK;
}

ps_status ps_plan_get_info(const ps_plan* pl, ps_plan_info* info_out) {
    if (!pl || !info_out) return fail(PS_ERR_INVALID, "null argument");
    *info_out = pl->info;
    return PS_OK;
}

ps_status ps_plan_get_items(const ps_plan* pl, int32_t* decode_items_out, int64_t decode_capacity,
                            int32_t* prefill_items_out, int64_t prefill_capacity) {
    if (!pl) return fail(PS_ERR_INVALID, "null argument");
    if (decode_items_out) {
        if (decode_capacity < (int64_t)pl->pieces.size()) return fail(PS_ERR_INVALID, "decode capacity too small");
        for (size_t i = 0; i < pl->pieces.size(); ++i) {
            const DecodePiece& pc = pl->pieces[i];
            int32_t* o = decode_items_out + 8 * i;
            o[0] = pc.req;
            o[1] = pc.kv_head;
            o[2] = pc.page_begin * kPage;
            o[3] = std::min(pc.page_end * kPage, pc.kv_len);
            o[4] = pc.q_tok;
            o[5] = 1;
            o[6] = pc.part_slot;
            o[7] = pc.kv_len - 1;  // the row's own position
        }
    }
    if (prefill_items_out) {
        if (prefill_capacity < (int64_t)pl->prefill.size()) return fail(PS_ERR_INVALID, "prefill capacity too small");
        static_assert(sizeof(PrefillItem) == 32, "item record is 8 int32");
        if (!pl->prefill.empty()) memcpy(prefill_items_out, pl->prefill.data(), pl->prefill.size() * sizeof(PrefillItem));
    }
    return PS_OK;
}

ps_status ps_attn_run(ps_plan* pl, const ps_kv* kv, const void* q_dev, const int32_t* block_table_dev, void* out_dev,
                      float* lse_out_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!pl || !kv || !q_dev || !block_table_dev || !out_dev || !workspace_dev) return fail(PS_ERR_INVALID, "null argument");
    if (workspace_bytes < pl->ws_bytes)
        return fail(PS_ERR_WORKSPACE, "workspace has %zu bytes, the plan needs %zu", workspace_bytes, pl->ws_bytes);
    if ((uintptr_t)workspace_dev % 256 != 0) return fail(PS_ERR_INVALID, "workspace must be 256-byte aligned");
    if (((uintptr_t)q_dev | (uintptr_t)out_dev) % 16 != 0) return fail(PS_ERR_INVALID, "q and out must be 16-byte aligned");
    const KvPool& pool = pool_of(kv);
    if (memcmp(&pool.shape, &pl->shape, sizeof(ps_shape)) != 0) return fail(PS_ERR_INVALID, "plan and pool shapes differ");
    cudaStream_t s = (cudaStream_t)stream;
    char* const ws_base = (char*)workspace_dev;
    const int slot = (int)(pl->run_no & 1u);
    char* ws = ws_base + (size_t)slot * pl->slot_stride;  // this run's image slot; partials are addressed from ws_base
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    PS_CUDA_TRY(cudaStreamIsCapturing(s, &cap));
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    // The upload may run under the kernels of the previous run only if this plan's own record of the two slots is
    // all there is to know about the workspace: same memory as last time, slots where they were, and no other
    // plan's run on it since.
    const bool mine = claim_workspace(workspace_dev, pl->serial);
    const bool known = mine && pl->last_ws == workspace_dev && !pl->layout_moved;
    if (capturing) {
        // Inside a stream capture the upload is a node of the graph on the caller's stream: every replay copies the
        // staging image as it then stands.  Nothing recorded here may be waited for by a later call outside the
        // capture, so the slot bookkeeping starts afresh.
        PS_CUDA_TRY(cudaMemcpyAsync(ws, pl->pinned, pl->image_bytes, cudaMemcpyHostToDevice, s));
        pl->done_valid[0] = pl->done_valid[1] = false;
    } else if (pl->copy_stream) {
        cudaStream_t cs = pl->copy_stream;
        if (known && pl->done_valid[slot]) {
            // the slot is free once the run two calls ago has finished; the previous run reads the other slot and
            // the partial rows behind both
            PS_CUDA_TRY(cudaStreamWaitEvent(cs, pl->ev_done[slot], 0));
        } else {
            // First use of this memory, slots that have moved, or another plan's work list in it: the upload is
            // ordered after everything already on the caller's stream (every earlier run that shares this workspace
            // is on that stream, or ordered before this call by the caller).
            PS_CUDA_TRY(cudaEventRecord(pl->ev_fence, s));
            PS_CUDA_TRY(cudaStreamWaitEvent(cs, pl->ev_fence, 0));
            if (!known) pl->done_valid[0] = pl->done_valid[1] = false;
        }
        PS_CUDA_TRY(cudaMemcpyAsync(ws, pl->pinned, pl->image_bytes, cudaMemcpyHostToDevice, cs));
        PS_CUDA_TRY(cudaEventRecord(pl->ev_copied[slot], cs));
        PS_CUDA_TRY(cudaStreamWaitEvent(s, pl->ev_copied[slot], 0));
        pl->copy_pending = true;
        pl->last_slot = slot;
    } else {
        PS_CUDA_TRY(cudaMemcpyAsync(ws, pl->pinned, pl->image_bytes, cudaMemcpyHostToDevice, s));
        PS_CUDA_TRY(cudaStreamSynchronize(s));  // no event to guard the staging image: finish the copy now
    }
    // the upload is in place (or queued): only now does the run count
    ++pl->run_no;
    pl->layout_moved = false;
    pl->last_ws = workspace_dev;
    pl->last_hdr = (WsHeader*)ws;
    pl->done_valid[slot] = false;  // until this run's own completion event is recorded below

    RunArgs a{};
    a.shape = pl->shape;
    a.pool = pool.base;
    a.num_pages = pool.num_pages;
    a.q = (const __nv_bfloat16*)q_dev;
    a.block_table = block_table_dev;
    a.max_pages = pl->max_pages;
    a.out = (__nv_bfloat16*)out_dev;
    a.lse = lse_out_dev;
    a.stream = s;
    a.num_sms = pl->num_sms;
    a.dec_sms = pl->dec_sms;
    a.pf_sms = pl->pf_sms;
    a.total_q = (int32_t)pl->info.total_q_tokens;
    a.n_req = pl->n;
    a.wait_limit_ns = pl->wait_limit_ns;
    a.w.hdr = (WsHeader*)ws;
    a.w.pieces = (const DecodePiece*)(ws + pl->off_pieces);
    a.w.units = (const DecodeUnit*)(ws + pl->off_units);
    a.w.prefill = (const PrefillItem*)(ws + pl->off_prefill);
    a.w.merge = (const MergeEntry*)(ws + pl->off_merge);
    a.w.part_lse = (float*)(ws_base + pl->off_part_lse);
    a.w.part_o = (float*)(ws_base + pl->off_part_o);
    a.w.n_units = (int32_t)pl->units.size();
    a.w.n_prefill = (int32_t)pl->prefill.size();
    a.w.n_merge = (int32_t)pl->merge.size();
    a.w.n_dmerge = (int32_t)pl->dmerge.size();
    a.w.n_part_slots = pl->info.n_partial_slots;
    a.w.dmerge = (const DecodeMerge*)(ws + pl->off_dmerge);
    a.w.dmerge_cnt = (int32_t*)(ws + pl->off_dmerge_cnt);
    a.w.prefill_cta_start = (const int32_t*)(ws + pl->off_cta_start);
    a.w.n_prefill_ctas = pl->prefill_cta_start.empty() ? 0 : (int32_t)pl->prefill_cta_start.size() - 1;

    // events per recorded run: prefill begin/end, decode begin/end, merge begin/end
    const bool rec = !capturing && pl->timing && (size_t)(pl->timed_runs + 1) * 6 <= pl->tev.size();
    cudaEvent_t* ev = rec ? &pl->tev[(size_t)pl->timed_runs * 6] : nullptr;
    ps_status st = PS_OK;
    bool merged = false;  // the merge kernel has been launched already
    if (pl->concurrent && pl->side_stream) {
        // Mixed batch: the decode kernel runs on its share of the SMs on a second stream while the
        // prefill kernel runs on the rest.  Both need about 200 KB of shared memory per CTA, so each SM
        // holds one CTA of either kernel.
        cudaStream_t side = pl->side_stream;
        PS_CUDA_TRY(cudaEventRecord(pl->ev_fork, s));
        PS_CUDA_TRY(cudaStreamWaitEvent(side, pl->ev_fork, 0));
        // From here on the side stream belongs to this call (inside a capture: to the capture): whatever
        // fails below, it is joined back into the caller's stream before the call returns.
        if (rec) cudaEventRecord(ev[2], side);
        RunArgs ad = a;
        ad.stream = side;
        st = launch_decode(ad);
        if (rec && st == PS_OK) cudaEventRecord(ev[3], side);
        if (rec && st == PS_OK) cudaEventRecord(ev[0], s);
        if (st == PS_OK) st = launch_prefill(a);
        if (rec && st == PS_OK) cudaEventRecord(ev[1], s);
        const bool helpers = a.w.n_prefill_ctas == 0 && a.w.n_prefill > a.pf_sms;
        if (st == PS_OK && !helpers) {
            // Only this launch writes prefill partials: combine them right behind it, on the SMs it leaves, while
            // the decode kernel is still streaming (decode rows are combined inside the decode kernel).
            if (rec) cudaEventRecord(ev[4], s);
            st = launch_merge(a);
            if (rec) cudaEventRecord(ev[5], s);
            merged = true;
        }
        if (st == PS_OK && helpers) {
            // dynamic item queue: once the decode CTAs have left their SMs, as many more prefill CTAs
            // start there and help drain the same queue
            RunArgs ah = a;
            ah.stream = side;
            ah.pf_sms = a.dec_sms;
            st = launch_prefill(ah);
        }
        const cudaError_t ej = cudaEventRecord(pl->ev_join, side);
        const cudaError_t ew = ej == cudaSuccess ? cudaStreamWaitEvent(s, pl->ev_join, 0) : ej;
        if (st != PS_OK) return st;
        PS_CUDA_TRY(ew);
    } else {
        if (rec) cudaEventRecord(ev[0], s);
        st = launch_prefill(a);
        if (st != PS_OK) return st;
        if (rec) cudaEventRecord(ev[1], s);
        if (rec) cudaEventRecord(ev[2], s);
        st = launch_decode(a);
        if (st != PS_OK) return st;
        if (rec) cudaEventRecord(ev[3], s);
    }
    if (!merged) {
        if (rec) cudaEventRecord(ev[4], s);
        st = launch_merge(a);
        if (rec) cudaEventRecord(ev[5], s);
    }
    if (rec) ++pl->timed_runs;
    if (pl->copy_stream && st == PS_OK && !capturing) {
        PS_CUDA_TRY(cudaEventRecord(pl->ev_done[slot], s));
        pl->done_valid[slot] = true;
    }
    return st;
}

ps_status ps_plan_set_wait_limit(ps_plan* pl, int64_t limit_ns) {
    if (!pl) return fail(PS_ERR_INVALID, "null argument");
    if (limit_ns < 0 || limit_ns > kMaxWaitLimitNs)
        return fail(PS_ERR_INVALID, "limit_ns=%lld outside [0, %lld]", (long long)limit_ns, (long long)kMaxWaitLimitNs);
    pl->wait_limit_ns = limit_ns;
    return PS_OK;
}

ps_status ps_plan_set_timing(ps_plan* pl, int32_t max_runs) {
    if (!pl) return fail(PS_ERR_INVALID, "null argument");
    if (max_runs < 0 || max_runs > 4096) return fail(PS_ERR_INVALID, "max_runs=%d outside [0, 4096]", max_runs);
    pl->timed_runs = 0;
    pl->timing = max_runs > 0;
    while (pl->tev.size() < (size_t)max_runs * 6) {
        cudaEvent_t e;
        PS_CUDA_TRY(cudaEventCreate(&e));
        pl->tev.push_back(e);
    }
    return PS_OK;
}

ps_status ps_plan_get_timing(ps_plan* pl, void* stream, float* prefill_ms_out, float* decode_ms_out, float* merge_ms_out,
                             int32_t* n_runs_out) {
    if (!pl || !prefill_ms_out || !decode_ms_out || !merge_ms_out || !n_runs_out) return fail(PS_ERR_INVALID, "null argument");
    PS_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    double acc[3] = {0, 0, 0};
    for (int r = 0; r < pl->timed_runs; ++r)
        for (int k = 0; k < 3; ++k) {
            float ms = 0.f;
            PS_CUDA_TRY(cudaEventElapsedTime(&ms, pl->tev[(size_t)r * 6 + 2 * k], pl->tev[(size_t)r * 6 + 2 * k + 1]));
            acc[k] += ms;
        }
    const double n = pl->timed_runs > 0 ? pl->timed_runs : 1;
    *prefill_ms_out = (float)(acc[0] / n);
    *decode_ms_out = (float)(acc[1] / n);
    *merge_ms_out = (float)(acc[2] / n);
    *n_runs_out = pl->timed_runs;
    return PS_OK;
}

ps_status ps_plan_status(ps_plan* pl, void* stream) {
    if (!pl) return fail(PS_ERR_INVALID, "null argument");
    PS_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (!pl->last_hdr) return PS_OK;
    int32_t status = 0;
    PS_CUDA_TRY(cudaMemcpy(&status, &pl->last_hdr->status, sizeof status, cudaMemcpyDeviceToHost));
    if (status & kStatusTimeout) return fail(PS_ERR_TIMEOUT, "a bounded device-side wait expired; output is invalid");
    if (status & kStatusBounds) return fail(PS_ERR_BOUNDS, "a block-table entry pointed outside the pool");
    return PS_OK;
}

}  // extern "C"

namespace ps {
size_t plan_workspace_bytes(const ps_plan* pl) { return pl ? pl->ws_bytes : 0; }
}  // namespace ps
