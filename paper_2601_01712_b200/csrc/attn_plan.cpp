// Host side of the tensor-core attention: the list of work items (and of split-KV merges) of one launch.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "forward.hpp"

namespace relaygr {

// ---- tensor-core attention work items: one per (user, head, 128-row tile[, KV split]) of the rows in `seqs` ------------------
// The kernel runs one item per CTA, two CTAs per SM, handed out in list order as CTAs retire.  The list is therefore
// ordered costliest first, and the plan decides how finely to split the key ranges so that the last wave is not a few
// whole items running on an otherwise idle GPU.  Cost model, in units of one 64-key block of one tile (about 0.7 us):
// an item costs kItemFixed (launch, Q and first K loads, first S, epilogue) plus its key blocks; `slots` items run at a
// time.  Every item is split `ns` ways; the items left over after the last full wave (the cheapest ones, at the end of
// the list) are split `nst` times finer still, so that their pieces spread over all slots.  ns is the value with the
// smallest estimated makespan; a split piece keeps at least kMinSplitBlocks key blocks.
void build_attention_worklist(const std::vector<SeqDesc> &seqs, int n_heads, int n_sms, int64_t max_split_tiles,
                              std::vector<AttnItem> &items, std::vector<AttnMerge> &merges)
{
    constexpr double kItemFixed = 8.0, kMergeCost = 5.0;
    constexpr int kMinSplitBlocks = 4, kMaxSplit = 16;
    items.clear();
    merges.clear();
    struct Tile { int seq, q0, n_q, nb; };
    std::vector<Tile> tiles;
    int64_t sum_nb = 0;
    for (int u = 0; u < (int)seqs.size(); ++u) {
        const SeqDesc &sd = seqs[(size_t)u];
        const int nPB = (sd.n_paged + 63) / 64, nLB = (sd.n_lin + 63) / 64;      // key blocks of 64 (one page each)
        for (int q0 = 0; q0 < sd.n_q; q0 += 128) {
            const int n_q = std::min(128, sd.n_q - q0);
            const int tp1 = sd.q_pos0 + q0 + n_q - 1;
            const int kmax = tp1 < sd.causal_end ? tp1 : sd.causal_end - 1;      // last key position any row of the tile sees
            int nb = 0;
            if (kmax >= 0) {
                const int pb = sd.n_paged > 0 ? std::min(nPB, kmax / 64 + 1) : 0;
                int lb = 0;
                if (pb == nPB && sd.n_lin > 0 && kmax >= sd.lin_pos0) lb = std::min(nLB, (kmax - sd.lin_pos0) / 64 + 1);
                nb = pb + lb;
            }
            tiles.push_back({u, q0, n_q, nb});
            sum_nb += nb;
        }
    }
    if (tiles.empty()) return;
    // costliest first (key blocks x softmax warps with live rows); ties keep a user's tiles together (they share K / V through L2)
    std::sort(tiles.begin(), tiles.end(), [](const Tile &x, const Tile &y) {
        const int64_t cx = (int64_t)x.nb * ((x.n_q + 31) / 32), cy = (int64_t)y.nb * ((y.n_q + 31) / 32);
        if (cx != cy) return cx > cy;
        if (x.seq != y.seq) return x.seq < y.seq;
        return x.q0 < y.q0;
    });

    const int64_t slots = 2 * (int64_t)std::max(1, n_sms);
    const int64_t base = (int64_t)tiles.size() * n_heads;
    const double mean_nb = (double)sum_nb / (double)tiles.size();
    // tail_of(ns): how many items (of the unsplit list) do not fit the full waves, and how much finer they are split
    auto tail_of = [&](int ns, int64_t &tail_items, int &nst) {
        const int64_t waves = base * ns / slots;
        tail_items = base - waves * slots / ns;
        nst = 1;
        if (tail_items > 0) {
            const int room = (int)std::min<int64_t>(kMaxSplit, slots / (tail_items * ns));
            const int most = (int)(mean_nb / ns / kMinSplitBlocks);
            nst = std::max(1, std::min(room, most));
        }
        return waves;
    };
    int best_ns = 1;
    double best_est = 0;
    const int ns_most = std::max(1, std::min(kMaxSplit, (int)(mean_nb / kMinSplitBlocks)));
    for (int ns = 1; ns <= ns_most; ++ns) {
        if (ns > 1 && base * ns > max_split_tiles) break;
        int64_t tail_items;
        int nst;
        const int64_t waves = tail_of(ns, tail_items, nst);
        double est = (double)waves * (kItemFixed + mean_nb / ns);
        if (tail_items > 0) est += kItemFixed + mean_nb / (ns * nst);
        if (ns * nst > 1) est += kMergeCost;
        if (ns == 1 || est < best_est) { best_est = est; best_ns = ns; }
    }
    int64_t tail_items;
    int nst;
    tail_of(best_ns, tail_items, nst);

    int64_t idx = 0;
    int part_slot = 0;
    for (const Tile &t : tiles) {
        const bool has_cand = seqs[(size_t)t.seq].q_pos0 + t.q0 + t.n_q > seqs[(size_t)t.seq].causal_end;
        for (int h = 0; h < n_heads; ++h, ++idx) {
            const int want = idx >= base - tail_items ? best_ns * nst : best_ns;
            int ns = std::max(1, std::min(want, t.nb / kMinSplitBlocks));
            if (ns > 1 && part_slot + ns > max_split_tiles) ns = 1;
            if (ns == 1) {
                items.push_back({t.seq, h, t.q0, t.n_q, 0, t.nb, -1, has_cand ? 1 : 0});
            } else {
                merges.push_back({t.seq, h, t.q0, t.n_q, part_slot, ns});
                for (int i = 0; i < ns; ++i) {
                    const int b0 = (int)((int64_t)t.nb * i / ns), b1 = (int)((int64_t)t.nb * (i + 1) / ns);
                    items.push_back({t.seq, h, t.q0, t.n_q, b0, b1, part_slot + i, (i == 0 && has_cand) ? 1 : 0});
                }
                part_slot += ns;
            }
        }
    }
}

}  // namespace relaygr
