// Builds the prepared layer image (format: include/vptq.h, "prepared layer image") from the canonical index
// streams.  Plain host code: a set-up step that runs once per layer, not on the timed path.
#include <string.h>

#include <algorithm>
#include <thread>
#include <vector>

#include "common.cuh"
#include "prepared.cuh"

namespace vptq {

namespace {

// What one partition contributes: its warps' blocks, in warp order.
struct PartImage {
    std::vector<uint32_t> hdr;          // one word per block
    std::vector<uint32_t> entries;      // 128 words per block
    uint32_t warp_blocks[PREP_WARPS];   // blocks of every warp
};

// A quarter block: four steps of eight lanes (one lane per residue of the main index mod 8) in one vector row.
struct QuarterBlock {
    uint32_t e[8][4];
    uint32_t row;
};

void build_partition(const PreparedGeometry &g, const uint8_t *idx1, long long stride1, const uint8_t *idx2,
                     long long stride2, int part, PartImage *out)
{
    const PreparedPart pp = prepared_part(g.R, g.n_buckets, g.n_parts, g.n_split, part);
    const int r0 = pp.r0, r1 = pp.r1;          // the partition's rows, and of their entries those of the buckets [b0, b1)
    const int n_rows = r1 - r0, nb8 = g.n_buckets * 8;
    const uint32_t pad = (uint32_t)g.N << 17;

    // every row's entries sorted by (bucket, residue of the main index mod 8); the column of an entry is the
    // stored column (the main columns follow the outlier columns)
    std::vector<uint32_t> sorted((size_t)n_rows * g.Nc);
    std::vector<int> count((size_t)n_rows * nb8, 0), start((size_t)n_rows * nb8);
    std::vector<int32_t> row1((size_t)g.Nc), row2((size_t)g.Nc, 0);
    for (int r = r0; r < r1; r++) {
        unpack_host(idx1 + (long long)r * stride1, 1, g.Nc, g.k1, row1.data());
        if (idx2) unpack_host(idx2 + (long long)r * stride2, 1, g.Nc, g.k2, row2.data());
        int *cnt = &count[(size_t)(r - r0) * nb8], *st = &start[(size_t)(r - r0) * nb8];
        for (int c = 0; c < g.Nc; c++) {
            if (row1[c] >= g.k1) row1[c] = g.k1 - 1;                       // clamp, as every kernel does
            if (g.k2 > 0 && row2[c] >= g.k2) row2[c] = g.k2 - 1;
            cnt[(row1[c] >> 12) * 8 + (row1[c] & 7)]++;
        }
        int at = 0;
        for (int i = 0; i < nb8; i++) { st[i] = at; at += cnt[i]; }
        std::vector<int> fill(st, st + nb8);
        uint32_t *dst = &sorted[(size_t)(r - r0) * g.Nc];
        for (int c = 0; c < g.Nc; c++) {
            const uint32_t id = (uint32_t)row1[c], id2 = (uint32_t)row2[c];
            dst[fill[(id >> 12) * 8 + (id & 7)]++] = ((id & 0xFFFu) >> 3) | (id2 << 9) | ((uint32_t)(g.n_out + c) << 17);
        }
    }

    // Per bucket, the four quarters of a warp run four STREAMS of rows side by side: a quarter changes its row
    // as rarely as if it had the warp to itself, while the 32 lanes of a step draw their columns from four rows.  That
    // matters for the activation lookups (bank = bits 1..5 of the column): the order of a lane's entries is
    // free, and every step is a matching of lanes to banks (a lane can take a bank when its row and residue
    // class still have an entry there), found with augmenting paths; lanes left unmatched take any entry of
    // theirs.  One row's 512 or so entries per bucket fill the banks too unevenly for that to work; four do.
    std::vector<std::vector<QuarterBlock>> qb(g.n_buckets);       // [bucket][4 * warp block + quarter]
    std::vector<uint32_t> stack[4][8][32];
    for (int b = pp.b0; b < pp.b1; b++) {
        // The bucket's quarter blocks, row after row, are cut into four streams of equal length; a row that
        // lies across a cut becomes two segments, each with its share of every class's entries.
        struct Segment { int row, nq, first[8], n[8]; };       // entries [first[c], first[c] + n[c]) of the row's class lists
        std::vector<Segment> seg_of[4];
        std::vector<int> nq_of((size_t)n_rows);
        int total_q = 0;
        for (int r = 0; r < n_rows; r++) {
            int steps = 0;
            for (int c = 0; c < 8; c++) steps = std::max(steps, count[(size_t)r * nb8 + b * 8 + c]);
            nq_of[r] = (steps + 3) / 4;
            total_q += nq_of[r];
        }
        const int nblk = (total_q + 3) / 4;                      // warp blocks of the bucket = length of a stream
        {
            int k = 0, room = nblk;
            for (int r = 0; r < n_rows; r++) {
                int todo = nq_of[r], given[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                while (todo > 0) {
                    if (room == 0) { k++; room = nblk; }
                    Segment sg;
                    sg.row = r;
                    sg.nq = std::min(todo, room);
                    for (int c = 0; c < 8; c++) {
                        const int cnt = count[(size_t)r * nb8 + b * 8 + c] - given[c];      // what the row has left
                        // its share by length, at most what fits here, at least what would not fit in the rest
                        int take = (int)(((long long)cnt * sg.nq + todo - 1) / todo);
                        take = std::max(take, cnt - 4 * (todo - sg.nq));
                        take = std::min(std::min(take, cnt), 4 * sg.nq);
                        sg.first[c] = given[c];
                        sg.n[c] = take;
                        given[c] += take;
                    }
                    seg_of[k].push_back(sg);
                    todo -= sg.nq;
                    room -= sg.nq;
                }
            }
        }
        QuarterBlock idle;
        idle.row = 63;
        for (int c = 0; c < 8; c++)
            for (int s = 0; s < 4; s++) idle.e[c][s] = pad;
        qb[b].assign((size_t)nblk * 4, idle);
        int cur[4] = {-1, -1, -1, -1}, togo[4] = {0, 0, 0, 0}, left[4][8];      // stream state: row, its blocks to go
        int steps_left[4] = {0, 0, 0, 0};                                        // steps the segment still has in its quarter
        size_t next[4] = {0, 0, 0, 0};
        for (int j = 0; j < nblk; j++) {
            for (int k = 0; k < 4; k++) {
                if (togo[k] == 0) {
                    cur[k] = -1;
                    if (next[k] < seg_of[k].size()) {
                        const Segment &sg = seg_of[k][next[k]++];
                        const int r = sg.row;
                        cur[k] = r;
                        togo[k] = sg.nq;
                        steps_left[k] = 4 * sg.nq;
                        for (int c = 0; c < 8; c++) {
                            for (int q = 0; q < 32; q++) stack[k][c][q].clear();
                            const uint32_t *list = &sorted[(size_t)r * g.Nc + start[(size_t)r * nb8 + b * 8 + c] + sg.first[c]];
                            left[k][c] = sg.n[c];
                            for (int i = 0; i < left[k][c]; i++) stack[k][c][(list[i] >> 18) & 31u].push_back(list[i]);
                        }
                    }
                }
                if (cur[k] >= 0) { qb[b][(size_t)j * 4 + k].row = (uint32_t)cur[k]; togo[k]--; }
            }
            for (int s = 0; s < 4; s++) {
                // Lanes that have entries left.  A row has as many steps as its fullest class needs (rounded up to
                // whole blocks), so the other classes' lanes have steps to spare: a lane MUST take an entry now
                // only when it has as many left as the row has steps; otherwise it may sit a step out when all its
                // banks are taken.  The lanes without an entry then all name the same one of the columns N .. N+63,
                // one whose bank is still free (the kernel holds zeros there).
                int lane_k[32], lane_c[32], slack[32], n_lanes = 0;
                for (int k = 0; k < 4; k++) {
                    if (cur[k] < 0) continue;
                    for (int c = 0; c < 8; c++)
                        if (left[k][c] > 0) {
                            int at = n_lanes++;                   // kept sorted by slack: the tightest lanes are matched first
                            const int sl = steps_left[k] - left[k][c];
                            for (; at > 0 && slack[at - 1] > sl; at--) {
                                lane_k[at] = lane_k[at - 1]; lane_c[at] = lane_c[at - 1]; slack[at] = slack[at - 1];
                            }
                            lane_k[at] = k; lane_c[at] = c; slack[at] = sl;
                        }
                    steps_left[k]--;
                }
                int bank_of[32], lane_at[32];                     // lane -> bank, bank -> lane; -1 = none
                for (int i = 0; i < 32; i++) { bank_of[i] = -1; lane_at[i] = -1; }
                // a lane tries its banks fullest first, so that what is left towards the end of a row is spread
                // over many banks
                uint8_t pref[32][32];
                for (int l = 0; l < n_lanes; l++) {
                    const std::vector<uint32_t> *st = stack[lane_k[l]][lane_c[l]];
                    for (int q = 0; q < 32; q++) pref[l][q] = (uint8_t)q;
                    std::stable_sort(pref[l], pref[l] + 32, [&](uint8_t x, uint8_t y) { return st[x].size() > st[y].size(); });
                }
                bool seen[32];
                auto augment = [&](auto &&self, int l) -> bool {
                    const std::vector<uint32_t> *st = stack[lane_k[l]][lane_c[l]];
                    for (int i = 0; i < 32; i++) {
                        const int q = pref[l][i];
                        if (st[q].empty()) break;
                        if (seen[q]) continue;
                        seen[q] = true;
                        if (lane_at[q] == -1 || self(self, lane_at[q])) { lane_at[q] = l; bank_of[l] = q; return true; }
                    }
                    return false;
                };
                for (int l = 0; l < n_lanes; l++) {
                    for (int q = 0; q < 32; q++) seen[q] = false;
                    augment(augment, l);
                }
                uint32_t used = 0;                                // banks the step's entries read
                for (int pass = 0; pass < 2; pass++)              // matched lanes first: their entries are spoken for
                    for (int l = 0; l < n_lanes; l++) {
                        std::vector<uint32_t> *st = stack[lane_k[l]][lane_c[l]];
                        int q = bank_of[l];
                        if ((q < 0) != (pass == 1)) continue;
                        if (q < 0 && slack[l] > 0) continue;      // sits this step out
                        if (q < 0) {                              // no free bank and no step to spare: the fullest stack
                            q = 0;
                            for (int i = 1; i < 32; i++)
                                if (st[i].size() > st[q].size()) q = i;
                        }
                        qb[b][(size_t)j * 4 + lane_k[l]].e[lane_c[l]][s] = st[q].back();
                        st[q].pop_back();
                        left[lane_k[l]][lane_c[l]]--;
                        used |= 1u << q;
                    }
                uint32_t none = pad;
                for (int d = 0; d < PREP_PAD_COLS; d++)
                    if (!((used >> (((g.N + d) >> 1) & 31)) & 1u)) { none = (uint32_t)(g.N + d) << 17; break; }
                for (int k = 0; k < 4; k++) {
                    if (cur[k] < 0) continue;
                    for (int c = 0; c < 8; c++) {
                        uint32_t &e = qb[b][(size_t)j * 4 + k].e[c][s];
                        if ((e >> 17) >= (uint32_t)g.N) e = none;
                    }
                }
            }
        }
    }
    // A warp block is four consecutive quarter blocks of a bucket's list (one of each stream).  A bucket's warp
    // blocks go to the warps in order, floor(n / warps) each, and the remainder one each to the warps that have
    // had the least work so far: the kernel lets a warp run one bucket ahead of the slowest, so what has to be
    // even is the running total, not every bucket by itself.
    std::vector<std::vector<uint32_t>> w_hdr(PREP_WARPS), w_ent(PREP_WARPS);
    long long done[PREP_WARPS] = {0};
    for (int b = pp.b0; b < pp.b1; b++) {
        const long long Q = (long long)qb[b].size(), nblk = (Q + 3) / 4;
        long long share[PREP_WARPS];
        int order[PREP_WARPS];
        for (int w = 0; w < PREP_WARPS; w++) { share[w] = nblk / PREP_WARPS; order[w] = w; }
        std::stable_sort(order, order + PREP_WARPS, [&](int a, int c) { return done[a] < done[c]; });
        for (int i = 0; i < (int)(nblk % PREP_WARPS); i++) share[order[i]]++;
        long long j = 0;
        for (int w = 0; w < PREP_WARPS; w++) {
            for (const long long j1 = j + share[w]; j < j1; j++) {
                uint32_t h = (uint32_t)(b - pp.b0) << 24;            // counted from the partition's first bucket
                const size_t base = w_ent[w].size();
                w_ent[w].resize(base + 128, pad);
                for (int k = 0; k < 4; k++) {
                    if (4 * j + k >= Q) { h |= 63u << (6 * k); continue; }
                    const QuarterBlock &q = qb[b][(size_t)(4 * j + k)];
                    h |= q.row << (6 * k);
                    if (q.row == 63) continue;
                    for (int c = 0; c < 8; c++)
                        for (int s = 0; s < 4; s++) w_ent[w][base + 4 * (8 * k + c) + s] = q.e[c][s];
                }
                w_hdr[w].push_back(h);
            }
            done[w] += share[w];
        }
    }
    for (int w = 0; w < PREP_WARPS; w++) {
        out->warp_blocks[w] = (uint32_t)w_hdr[w].size();
        out->hdr.insert(out->hdr.end(), w_hdr[w].begin(), w_hdr[w].end());
        out->entries.insert(out->entries.end(), w_ent[w].begin(), w_ent[w].end());
    }
}

}  // namespace

int prepare_host(const PreparedGeometry &g, const uint8_t *idx1, const uint8_t *idx2, void *image, size_t image_bytes,
                 size_t *used_bytes)
{
    const long long stride1 = row_bytes(g.Nc, g.k1), stride2 = g.k2 ? row_bytes(g.Nc, g.k2) : 0;
    std::vector<PartImage> parts((size_t)g.n_parts);
    unsigned n_threads = std::thread::hardware_concurrency();
    if (n_threads < 1) n_threads = 1;
    if (n_threads > 32) n_threads = 32;
    if (n_threads > (unsigned)g.n_parts) n_threads = (unsigned)g.n_parts;
    std::vector<std::thread> pool;
    for (unsigned t = 0; t < n_threads; t++)
        pool.emplace_back([&, t]() {
            for (int p = (int)t; p < g.n_parts; p += (int)n_threads)
                build_partition(g, idx1, stride1, g.k2 ? idx2 : nullptr, stride2, p, &parts[(size_t)p]);
        });
    for (auto &th : pool) th.join();

    unsigned long long n_blocks = 0;
    for (const PartImage &pi : parts) n_blocks += pi.hdr.size();
    const PreparedLayout lay = prepared_layout(g.n_parts, n_blocks);
    if (used_bytes) *used_bytes = (size_t)lay.total;
    if (n_blocks > 0xFFFFFFFFull || lay.total > image_bytes) return VPTQ_E_WORKSPACE;

    uint8_t *img = reinterpret_cast<uint8_t *>(image);
    memset(img, 0, 256);
    uint32_t *head = reinterpret_cast<uint32_t *>(img);
    head[0] = VPTQ_PREPARED_MAGIC; head[1] = 2; head[2] = (uint32_t)g.M; head[3] = (uint32_t)g.N;
    head[4] = (uint32_t)g.k1; head[5] = (uint32_t)g.k2; head[6] = (uint32_t)g.n_parts; head[7] = PREP_WARPS;
    head[8] = (uint32_t)g.n_buckets; head[9] = (uint32_t)n_blocks;
    head[10] = (uint32_t)lay.off_woff; head[11] = (uint32_t)lay.off_hdr; head[12] = (uint32_t)lay.off_entries;
    head[13] = (uint32_t)lay.total; head[14] = (uint32_t)((unsigned long long)g.R * g.Nc);
    head[15] = (uint32_t)g.n_split; head[16] = (uint32_t)g.v; head[17] = (uint32_t)g.n_out;
    uint32_t *woff = reinterpret_cast<uint32_t *>(img + lay.off_woff);
    uint32_t *hdr = reinterpret_cast<uint32_t *>(img + lay.off_hdr);
    uint32_t *ent = reinterpret_cast<uint32_t *>(img + lay.off_entries);
    // zero the alignment gaps so that the image is a function of its inputs alone
    memset(img + 256, 0, (size_t)(lay.off_entries - 256));
    uint32_t at = 0;
    for (int p = 0; p < g.n_parts; p++) {
        const PartImage &pi = parts[(size_t)p];
        for (int w = 0; w < PREP_WARPS; w++) {
            woff[p * PREP_WARPS + w] = at;
            at += pi.warp_blocks[w];
        }
        const uint32_t first = woff[p * PREP_WARPS];
        if (!pi.hdr.empty()) {
            memcpy(hdr + first, pi.hdr.data(), pi.hdr.size() * 4);
            memcpy(ent + (size_t)first * 128, pi.entries.data(), pi.entries.size() * 4);
        }
    }
    woff[g.n_parts * PREP_WARPS] = at;
    memset(img + lay.off_entries + (size_t)n_blocks * 512, 0, (size_t)(lay.total - lay.off_entries - n_blocks * 512));
    return VPTQ_OK;
}

}  // namespace vptq
