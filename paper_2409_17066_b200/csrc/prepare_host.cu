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
    const uint32_t pad = (uint32_t)g.N << 17;
    std::vector<std::vector<QuarterBlock>> qb(g.n_buckets);
    std::vector<uint32_t> sorted((size_t)g.N);                  // the row's entries, by (bucket, residue)
    std::vector<int> count((size_t)g.n_buckets * 8), start((size_t)g.n_buckets * 8 + 1);
    for (int r = r0; r < r1; r++) {
        const uint16_t *row1 = reinterpret_cast<const uint16_t *>(idx1 + (long long)r * stride1);
        const uint8_t *row2 = idx2 ? idx2 + (long long)r * stride2 : nullptr;
        std::fill(count.begin(), count.end(), 0);
        for (int n = 0; n < g.N; n++) {
            uint32_t id = row1[n];
            if (id >= (uint32_t)g.k1) id = (uint32_t)g.k1 - 1;             // clamp, as every kernel does
            count[(id >> 12) * 8 + (id & 7)]++;
        }
        start[0] = 0;
        for (size_t i = 0; i < count.size(); i++) start[i + 1] = start[i] + count[i];
        std::vector<int> fill(start.begin(), start.end() - 1);
        for (int n = 0; n < g.N; n++) {
            uint32_t id = row1[n];
            if (id >= (uint32_t)g.k1) id = (uint32_t)g.k1 - 1;
            uint32_t id2 = row2 ? row2[n] : 0u;
            if (g.k2 > 0 && id2 >= (uint32_t)g.k2) id2 = (uint32_t)g.k2 - 1;
            sorted[(size_t)fill[(id >> 12) * 8 + (id & 7)]++] = ((id & 0xFFFu) >> 3) | (id2 << 9) | ((uint32_t)n << 17);
        }
        for (int b = pp.b0; b < pp.b1; b++) {
            int steps = 0;
            for (int c = 0; c < 8; c++) steps = std::max(steps, count[b * 8 + c]);
            // The order of a lane's entries is free.  It is chosen so that the 32 lanes of a warp step look their
            // activations up in different shared-memory banks where possible (bank = bits 1..5 of the column):
            // quarter blocks that will share a warp block are filled together, step by step, each lane taking
            // an entry of its residue class whose bank no lane of the step has taken yet.
            const int nq = (steps + 3) / 4;
            const size_t q_first = qb[b].size();
            qb[b].resize(q_first + (size_t)nq);
            int left[8];
            for (int c = 0; c < 8; c++) left[c] = count[b * 8 + c];
            for (int lq0 = 0; lq0 < nq;) {
                int lq1 = lq0 + 1;                                        // quarter blocks [lq0, lq1) share a warp block
                while (lq1 < nq && (q_first + (size_t)lq1) / 4 == (q_first + (size_t)lq0) / 4) lq1++;
                for (int lq = lq0; lq < lq1; lq++) qb[b][q_first + (size_t)lq].row = (uint32_t)(r - r0);
                for (int s = 0; s < 4; s++) {
                    uint32_t taken = 0;
                    for (int lq = lq0; lq < lq1; lq++)
                        for (int c = 0; c < 8; c++) {
                            uint32_t *list = &sorted[(size_t)start[b * 8 + c]];
                            uint32_t e = pad;
                            if (left[c] > 0) {
                                int pick = 0;
                                for (int i = 0; i < left[c]; i++)
                                    if (!((taken >> ((list[i] >> 18) & 31u)) & 1u)) { pick = i; break; }
                                e = list[pick];
                                list[pick] = list[--left[c]];
                                taken |= 1u << ((e >> 18) & 31u);
                            }
                            qb[b][q_first + (size_t)lq].e[c][s] = e;
                        }
                }
                lq0 = lq1;
            }
        }
    }
    // A warp block is four consecutive quarter blocks of a bucket's list (the last one filled up with idle
    // quarters).  A bucket's warp blocks go to the warps in order, floor(n / warps) each, and the remainder one
    // each to the warps that have had the least work so far: the kernel lets a warp run one bucket ahead of
    // the slowest, so what has to be even is the running total, not every bucket by itself.
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
                uint32_t h = (uint32_t)b << 24;
                const size_t base = w_ent[w].size();
                w_ent[w].resize(base + 128, pad);
                for (int k = 0; k < 4; k++) {
                    if (4 * j + k >= Q) { h |= 63u << (6 * k); continue; }
                    const QuarterBlock &q = qb[b][(size_t)(4 * j + k)];
                    h |= q.row << (6 * k);
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
    const long long stride1 = row_bytes(g.N, g.k1), stride2 = g.k2 ? row_bytes(g.N, g.k2) : 0;
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
    head[13] = (uint32_t)lay.total; head[14] = (uint32_t)((unsigned long long)g.R * g.N);
    head[15] = (uint32_t)g.n_split;
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
