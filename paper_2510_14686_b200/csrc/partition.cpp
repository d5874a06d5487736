// Work partition for the split-KV attention kernel (host only, no CUDA).
//
// The report's third layer of DP load balance works inside the attention kernel: instead of one
// request per compute core, requests are re-distributed so that every matrix unit sees about the
// same number of tokens, and very long sequences are split so that parts of them run next to short
// ones.  Here the "compute unit" is one persistent CTA per SM.  All (request, KV head, row group)
// units are laid out on one cost axis (tiles plus a fixed per-unit overhead) and the axis is cut into
// n_ctas equal runs; a cut that falls inside a unit splits that unit, and the pieces are merged later
// by the log-sum-exp combine kernel.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "xllm_internal.h"

namespace xllm {

namespace {
struct Unit {
    int32_t req, kv_head;
    int16_t q_tok0, n_q_tok, g0, n_g;
    int32_t n_tiles;  // tiles that hold keys visible to the unit's last row
    int32_t max_cut;  // largest tile boundary at which a split may start so that the first row still sees a key
};
struct Cut {
    int32_t unit, tile;
};
}  // namespace

int plan_partition(int32_t n_req, const int64_t *kv_lens, const int32_t *q_lens, int32_t n_q_heads,
                   int32_t n_kv_heads, int32_t n_ctas, const PlanTuning &tune, std::vector<xllm_work_item> &items,
                   std::vector<int32_t> &cta_begin, int32_t *n_units_out, int32_t *n_partials_out) {
    if (n_req < 1 || n_ctas < 1 || n_kv_heads < 1 || n_q_heads < n_kv_heads || n_q_heads % n_kv_heads) return -1;
    const int32_t G = n_q_heads / n_kv_heads;
    const int32_t T = XLLM_TILE_TOKENS;
    std::vector<Unit> units;
    units.reserve(static_cast<size_t>(n_req) * n_kv_heads);
    for (int32_t r = 0; r < n_req; ++r) {
        const int64_t kv = kv_lens[r];
        const int32_t ql = q_lens ? q_lens[r] : 1;
        if (ql < 1 || kv < ql || kv > INT32_MAX) return -1;
        for (int32_t h = 0; h < n_kv_heads; ++h) {
            if (G <= kMaxRows) {
                const int32_t per = std::max(1, kMaxRows / G);  // query tokens per row group
                for (int32_t t0 = 0; t0 < ql; t0 += per) {
                    const int32_t nt = std::min(per, ql - t0);
                    const int64_t vis_last = kv - ql + t0 + nt;  // keys visible to the last row
                    const int64_t vis_first = kv - ql + t0 + 1;  // keys visible to the first row
                    Unit u{r, h, (int16_t)t0, (int16_t)nt, 0, (int16_t)G, (int32_t)((vis_last + T - 1) / T),
                           (int32_t)((vis_first - 1) / T)};
                    units.push_back(u);
                }
            } else {
                for (int32_t t0 = 0; t0 < ql; ++t0) {
                    const int64_t vis = kv - ql + t0 + 1;
                    for (int32_t g0 = 0; g0 < G; g0 += kMaxRows) {
                        Unit u{r, h, (int16_t)t0, 1, (int16_t)g0, (int16_t)std::min(kMaxRows, G - g0),
                               (int32_t)((vis + T - 1) / T), (int32_t)((vis - 1) / T)};
                        units.push_back(u);
                    }
                }
            }
        }
    }
    const int32_t U = static_cast<int32_t>(units.size());
    // cost axis: start position of every unit
    std::vector<int64_t> start(static_cast<size_t>(U) + 1);
    start[0] = 0;
    for (int32_t u = 0; u < U; ++u)
        start[u + 1] = start[u] + tune.unit_overhead + (int64_t)tune.tile_cost * units[u].n_tiles;
    const int64_t total = start[U];

    std::vector<Cut> cuts(static_cast<size_t>(n_ctas) + 1);
    cuts[0] = {0, 0};
    cuts[n_ctas] = {U, 0};
    int32_t u = 0;
    for (int32_t c = 1; c < n_ctas; ++c) {
        const int64_t pos = (total * c) / n_ctas;
        while (u < U && start[u + 1] <= pos) ++u;
        if (u >= U) {
            cuts[c] = {U, 0};
            continue;
        }
        const Unit &un = units[u];
        int64_t b = (pos - start[u] - tune.unit_overhead + tune.tile_cost / 2) / tune.tile_cost;  // nearest tile
        if (pos - start[u] < tune.unit_overhead) b = 0;
        b = std::max<int64_t>(0, std::min<int64_t>(b, un.n_tiles));
        if (b > un.max_cut) b = un.max_cut;                      // every row of a piece must see a key
        if (b < tune.min_piece_tiles) b = 0;                     // no sliver at the front ...
        else if (un.n_tiles - b < tune.min_piece_tiles) b = un.n_tiles;  // ... nor at the back
        Cut cut = (b >= un.n_tiles) ? Cut{u + 1, 0} : Cut{u, (int32_t)b};
        // cuts never move backwards
        const Cut &prev = cuts[c - 1];
        if (cut.unit < prev.unit || (cut.unit == prev.unit && cut.tile < prev.tile)) cut = prev;
        cuts[c] = cut;
    }

    items.clear();
    cta_begin.assign(static_cast<size_t>(n_ctas) + 1, 0);
    int32_t n_partials = 0;
    for (int32_t c = 0; c < n_ctas; ++c) {
        cta_begin[c] = static_cast<int32_t>(items.size());
        Cut a = cuts[c];
        const Cut b = cuts[c + 1];
        while (a.unit < U && (a.unit < b.unit || (a.unit == b.unit && a.tile < b.tile))) {
            const Unit &un = units[a.unit];
            const int32_t te = (a.unit == b.unit) ? b.tile : un.n_tiles;
            if (te > a.tile) {
                xllm_work_item it;
                it.req = un.req;
                it.kv_head = un.kv_head;
                it.tile_begin = a.tile;
                it.tile_end = te;
                it.q_tok0 = un.q_tok0;
                it.n_q_tok = un.n_q_tok;
                it.g0 = un.g0;
                it.n_g = un.n_g;
                it.partial_idx = (a.tile == 0 && te == un.n_tiles) ? -1 : n_partials++;
                it.unit = a.unit;
                items.push_back(it);
            }
            if (a.unit == b.unit) break;
            a = {a.unit + 1, 0};
        }
    }
    cta_begin[n_ctas] = static_cast<int32_t>(items.size());
    if (n_units_out) *n_units_out = U;
    if (n_partials_out) *n_partials_out = n_partials;
    return 0;
}

}  // namespace xllm
