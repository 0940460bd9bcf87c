// Host side of libalcs: the grouped-CSR packer (paper, Section 3.2.2, storage-format paragraph),
// its inverse, the serialised blob, and the launch schedules derived from a packed matrix.
// No CUDA in this file.
#include <algorithm>
#include <climits>
#include <cstring>
#include <limits>
#include <new>
#include <numeric>

#include "alcs_internal.h"

namespace {

constexpr uint32_t kMagic = 0x53434C41u;  // "ALCS" little-endian
constexpr uint32_t kBlobVersion = 1;

struct BlobHeader {
    uint32_t magic, version;
    int32_t cout, cin, g, dtype, rows, nb;
};

thread_local const char* g_cuda_err = "";

}  // namespace

namespace alcs {

void set_cuda_error_text(const char* s) { g_cuda_err = s ? s : ""; }

float bfloat16_bits_to_float(uint16_t h)
{
    // bfloat16 -> binary32, exact: the upper half of the binary32 pattern
    const uint32_t bits = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

float half_bits_to_float(uint16_t h)
{
    // binary16 -> binary32, exact.  Handles zeros, subnormals, infinities and NaNs.
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t ex = (h >> 10) & 0x1fu;
    uint32_t man = h & 0x3ffu;
    uint32_t bits;
    if (ex == 0) {
        if (man == 0) {
            bits = sign;
        } else {
            int shift = 0;
            while (!(man & 0x400u)) { man <<= 1; ++shift; }
            man &= 0x3ffu;
            bits = sign | ((uint32_t)(127 - 15 - shift + 1) << 23) | (man << 13);
        }
    } else if (ex == 31) {
        bits = sign | 0x7f800000u | (man << 13);
    } else {
        bits = sign | ((ex + 127 - 15) << 23) | (man << 13);
    }
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

static int rec_bytes(int g) { return g == 1 ? 16 : 16 + 8 * g; }
int pair_record_bytes(int g) { return rec_bytes(g); }

// Pair records, slices and row headers for the row map already in `out` (n_rg groups of rpg local rows).
// part[rg*rpg + t] / nparts[...]: local row t multiplies only the blocks of its block row whose position in
// the row is congruent to part modulo nparts (empty vectors: every local row takes its whole row).
static void emit_pair_records(const alcs_packed& p, int kc, bool with_records, Schedule& out,
                              const std::vector<int>& part = std::vector<int>(),
                              const std::vector<int>& nparts = std::vector<int>())
{
    const int R = p.rows, g = p.g;
    const int n_rg = out.n_rg, rpg = out.rpg;
    const int nch = (p.cin + kc - 1) / kc;
    const int REC = rec_bytes(g);
    out.kc = kc; out.nch = nch;
    out.h_slice.assign((size_t)n_rg * nch + 1, 0);
    const int ros = rpg * 4;                     // one int4 {offset, first two columns, pair count} per local row
    out.ros = ros;
    out.h_rowoff.assign((size_t)n_rg * nch * ros, 0);
    out.h_rec.clear();
    std::vector<int> cursor((size_t)rpg);           // per local row: next block of its block row to look at
    std::vector<int> mine;                          // blocks of the current segment
    int rec_count = 0, wcap = 0;
    auto value = [&](int k, int j) -> float {
        const size_t vi = (size_t)k * g + j;
        float v;
        if (p.dt == ALCS_F32) {
            std::memcpy(&v, &p.vals[vi * 4], 4);
        } else {
            uint16_t hb;
            std::memcpy(&hb, &p.vals[vi * 2], 2);
            v = p.dt == ALCS_F16 ? half_bits_to_float(hb) : bfloat16_bits_to_float(hb);
        }
        return v;
    };
    for (int rg = 0; rg < n_rg; ++rg) {
        for (int t = 0; t < rpg; ++t) {
            const int r = out.h_rowmap[(size_t)rg * rpg + t];
            if (r >= 0) cursor[t] = p.row_ptr[r];
        }
        for (int c = 0; c < nch; ++c) {
            out.h_slice[(size_t)rg * nch + c] = rec_count;
            int* roff = &out.h_rowoff[((size_t)rg * nch + c) * ros];
            const int lim = (c + 1) * kc;
            const int c0 = c * kc;
            int local = 0;
            for (int t = 0; t < rpg; ++t) {
                int* hd = roff + 4 * t;                 // {segment start (16-byte units), c0, c1, pairs}
                hd[0] = local; hd[1] = hd[2] = hd[3] = 0;
                const int r = out.h_rowmap[(size_t)rg * rpg + t];
                if (r < 0) continue;
                const int np = nparts.empty() ? 1 : nparts[(size_t)rg * rpg + t];
                const int pt = part.empty() ? 0 : part[(size_t)rg * rpg + t];
                const int kend = p.row_ptr[r + 1];
                int k1 = cursor[t];
                mine.clear();
                for (; k1 < kend && p.col_idx[k1] < lim; ++k1)
                    if ((k1 - p.row_ptr[r]) % np == pt) mine.push_back(k1);
                cursor[t] = k1;
                const int nblk = (int)mine.size();
                const int npair = (nblk + 1) / 2;
                const int seg16 = npair * (REC / 16);
                auto cols_of = [&](int q, int* c) {       // chunk-local columns of pair q
                    const int ka = mine[2 * q];
                    const int kb = 2 * q + 1 < nblk ? mine[2 * q + 1] : ka;    // padding repeats the column
                    c[0] = p.col_idx[ka] - c0;
                    c[1] = p.col_idx[kb] - c0;
                };
                if (npair) cols_of(0, hd + 1);
                hd[3] = npair;
                if (with_records && npair) {
                    const size_t base = out.h_rec.size();
                    out.h_rec.resize(base + (size_t)seg16 * 16, 0);
                    for (int q = 0; q < npair; ++q) {
                        unsigned char* rec = &out.h_rec[base + (size_t)q * REC];
                        const int ka = mine[2 * q];
                        const bool has_b = 2 * q + 1 < nblk;
                        int hdr[4] = {0, 0, 0, 0};
                        if (q + 1 < npair) cols_of(q + 1, hdr);       // columns of the next pair
                        float* w = reinterpret_cast<float*>(rec + (g == 1 ? 8 : 16));
                        for (int j = 0; j < g; ++j) {
                            w[j] = value(ka, j);
                            w[g + j] = has_b ? value(mine[2 * q + 1], j) : 0.0f;
                        }
                        std::memcpy(rec, hdr, g == 1 ? 8 : 16);
                    }
                }
                local += seg16;
            }
            rec_count += local;
            wcap = std::max(wcap, local);
        }
    }
    out.h_slice[(size_t)n_rg * nch] = rec_count;
    out.n_rec = rec_count;
    out.wcap = wcap;
    (void)R;
}


void build_schedule(const alcs_packed& p, int kc, int n_rg, bool with_records, Schedule& out)
{
    if (kc <= 0 || kc > p.cin) kc = p.cin;
    const int R = p.rows;
    n_rg = std::max(1, std::min(n_rg, R));
    const int rpg = (R + n_rg - 1) / n_rg;
    out.n_rg = n_rg; out.rpg = rpg;

    // rows by descending kept-block count, dealt to the row groups in serpentine order
    std::vector<int> order(R);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        return p.row_ptr[a + 1] - p.row_ptr[a] > p.row_ptr[b + 1] - p.row_ptr[b];
    });
    out.h_rowmap.assign((size_t)n_rg * rpg, -1);
    for (int i = 0; i < R; ++i) {
        const int t = i / n_rg, j = i % n_rg;
        const int rg = (t & 1) ? n_rg - 1 - j : j;
        out.h_rowmap[(size_t)rg * rpg + t] = order[i];
    }

    emit_pair_records(p, kc, with_records, out);
}

// Local row of (consumer warp w, accumulator set s) in a kernel with nw consumer warps: the kernel's
// own mapping (tier s, warps in serpentine order).
int local_row_of(int w, int s, int nw) { return s * nw + ((s & 1) ? nw - 1 - w : w); }

// Word that tells a consumer warp what the unit in one of its accumulator sets is: role 0 = a whole
// block row, 1 = the primary part of a split row (adds `count` partial sums found in exchange slots
// slot, slot+1, ... and stores the row), 2 = a secondary part (writes its partial sums to exchange slot
// `slot` and stores nothing).
int unit_word(int role, int slot, int count) { return role | (slot << 4) | (count << 16); }
constexpr int kMaxExchange = 6;     // secondary units per row group (each costs an exchange tile in shared memory)
constexpr int kMaxParts = 7;        // parts one block row may be split into

// Balanced flavour of the pair-record schedule: see the comment on Schedule.
void build_schedule_balanced(const alcs_packed& p, int kc, int n_rg, int nw, int rw, bool with_records, Schedule& out,
                             bool allow_split)
{
    if (kc <= 0 || kc > p.cin) kc = p.cin;
    const int R = p.rows;
    const int cap = nw * rw;                             // block rows one work item can hold
    n_rg = std::max(std::max(1, (R + cap - 1) / cap), std::min(n_rg, R));
    out.n_rg = n_rg; out.rpg = cap; out.mma = 0; out.balanced = 1;
    out.nwg = nw; out.rw = rw;
    out.max_x = 0;

    // Sizes of the row groups: whole multiples of 4 where the capacity allows it, so that the four
    // schedulers of an SM can be given the same number of rows; otherwise as even as possible.
    std::vector<int> size(n_rg, 0);
    {
        const int quads = (R + 3) / 4;
        bool ok = true;
        int left = R;
        for (int i = 0; i < n_rg; ++i) {
            const int q = quads / n_rg + (i < quads % n_rg ? 1 : 0);
            size[i] = std::min(4 * q, left);
            left -= size[i];
            if (size[i] > cap) ok = false;
        }
        if (!ok || left > 0) {
            for (int i = 0; i < n_rg; ++i) size[i] = R / n_rg + (i < R % n_rg ? 1 : 0);
        }
    }

    // rows by descending kept-block count, dealt to the row groups in serpentine order (skipping full ones)
    std::vector<int> order(R);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        return p.row_ptr[a + 1] - p.row_ptr[a] > p.row_ptr[b + 1] - p.row_ptr[b];
    });
    std::vector<std::vector<int>> members(n_rg);
    {
        int pos = 0, dir = 1, i = 0;
        while (i < R) {
            if ((int)members[pos].size() < size[pos]) members[pos].push_back(order[i++]);
            if (pos + dir < 0 || pos + dir >= n_rg) dir = -dir; else pos += dir;
        }
    }

    // Inside a row group: "units" are dealt to the (warp, accumulator set) pairs.  A unit is a whole block
    // row, or, for a row far longer than the others, one of nparts parts of it (the blocks whose position
    // in the row is congruent to `part` modulo nparts, so that every chunk's share is split as well); the
    // spare (warp, set) pairs of the row group pay for the extra units.  Part 0 is the row's primary unit
    // (it adds the others' partial sums, handed over through shared memory, and stores the row); at most
    // kMaxExchange secondary units per row group.  Units, largest first, go in serpentine order to the
    // schedulers (scheduler of consumer warp w = w mod 4), then, per scheduler, to its warps; the t-th
    // unit a warp receives becomes its accumulator set t.
    struct Unit { int row, part, nparts, blocks; };
    const size_t nloc = (size_t)n_rg * cap;
    out.h_rowmap.assign(2 * nloc + n_rg, -1);
    std::fill(out.h_rowmap.begin() + nloc, out.h_rowmap.end(), 0);
    std::vector<int> part(nloc, 0), nparts(nloc, 1);
    int* unit_info = out.h_rowmap.data() + nloc;         // per local row, see unit_word()
    int* rg_exchange = out.h_rowmap.data() + 2 * nloc;   // per row group: secondary units (0: no hand-over)
    out.max_x = 0;
    const int nsched = std::min(4, nw);
    for (int rg = 0; rg < n_rg; ++rg) {
        std::vector<Unit> units;
        long long blocks_total = 0;
        for (int r : members[rg]) {
            const int len = p.row_ptr[r + 1] - p.row_ptr[r];
            units.push_back({r, 0, 1, len});
            blocks_total += len;
        }
        // split while a row's parts are still much larger than the average unit and a spare pair is left
        int spare = cap - (int)members[rg].size(), exchange = 0;
        std::vector<int> parts_of(members[rg].size(), 1);
        while (allow_split && spare > 0 && exchange < kMaxExchange && !units.empty()) {
            size_t best = 0;
            double best_load = -1;
            for (size_t i = 0; i < members[rg].size(); ++i) {
                const int len = p.row_ptr[members[rg][i] + 1] - p.row_ptr[members[rg][i]];
                const double load = (double)len / parts_of[i];
                if (load > best_load) { best_load = load; best = i; }
            }
            const double avg = (double)blocks_total / (double)(members[rg].size() + exchange);
            if (best_load <= std::max(1.5 * avg, 16.0) || parts_of[best] >= kMaxParts) break;
            ++parts_of[best];
            ++exchange;
            --spare;
        }
        if (exchange > 0) {
            units.clear();
            for (size_t i = 0; i < members[rg].size(); ++i) {
                const int r = members[rg][i];
                const int len = p.row_ptr[r + 1] - p.row_ptr[r];
                for (int q = 0; q < parts_of[i]; ++q)
                    units.push_back({r, q, parts_of[i], (len - q + parts_of[i] - 1) / parts_of[i]});
            }
            std::stable_sort(units.begin(), units.end(), [](const Unit& a, const Unit& b) { return a.blocks > b.blocks; });
        }
        rg_exchange[rg] = exchange;
        out.max_x = std::max(out.max_x, exchange);

        std::vector<std::vector<Unit>> per(nsched);
        std::vector<int> room(nsched, 0);
        for (int w = 0; w < nw; ++w) room[w % nsched] += rw;
        {
            int pos = 0, dir = 1;
            size_t i = 0;
            while (i < units.size()) {
                if ((int)per[pos].size() < room[pos]) per[pos].push_back(units[i++]);
                if (pos + dir < 0 || pos + dir >= nsched) dir = -dir; else pos += dir;
            }
        }
        // exchange slots: the secondary units of a row take consecutive slots, rows in order of appearance
        std::vector<int> first_slot(members[rg].size(), -1);
        {
            int next = 0;
            for (size_t i = 0; i < members[rg].size(); ++i)
                if (parts_of[i] > 1) { first_slot[i] = next; next += parts_of[i] - 1; }
        }
        auto index_of = [&](int row) {
            for (size_t i = 0; i < members[rg].size(); ++i)
                if (members[rg][i] == row) return i;
            return (size_t)0;
        };
        for (int k = 0; k < nsched; ++k) {
            std::vector<int> warps;
            for (int w = k; w < nw; w += nsched) warps.push_back(w);
            std::vector<int> fill(warps.size(), 0);
            int pos = 0, dir = 1;
            size_t i = 0;
            while (i < per[k].size()) {
                if (fill[pos] < rw) {
                    const Unit& u = per[k][i++];
                    const size_t at = (size_t)rg * cap + local_row_of(warps[pos], fill[pos], nw);
                    out.h_rowmap[at] = u.row;
                    part[at] = u.part;
                    nparts[at] = u.nparts;
                    if (u.nparts > 1) {
                        const int fs = first_slot[index_of(u.row)];
                        unit_info[at] = u.part == 0 ? unit_word(1, fs, u.nparts - 1) : unit_word(2, fs + u.part - 1, 0);
                    }
                    ++fill[pos];
                }
                if (pos + dir < 0 || pos + dir >= (int)warps.size()) dir = -dir; else pos += dir;
            }
        }
    }
    emit_pair_records(p, kc, with_records, out, part, nparts);
}

// Tensor-core flavour of the schedule (fp16 weights): see the comment on Schedule.
void build_schedule_mma(const alcs_packed& p, int kc, int n_rg, bool with_records, Schedule& out)
{
    if (kc <= 0 || kc > p.cin) kc = p.cin;
    const int R = p.rows, g = p.g;
    const int gp = g < 8 ? 8 : g;                 // output channels per block after padding to an 8-wide tile
    n_rg = std::max(1, std::min(n_rg, R));
    const int nch = (p.cin + kc - 1) / kc;
    const int rpg = (R + n_rg - 1) / n_rg;
    const int REC = step_record_bytes(g);
    out.kc = kc; out.nch = nch; out.n_rg = n_rg; out.rpg = rpg; out.mma = 1;

    std::vector<int> order(R);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
        return p.row_ptr[a + 1] - p.row_ptr[a] > p.row_ptr[b + 1] - p.row_ptr[b];
    });
    out.h_rowmap.assign((size_t)n_rg * rpg, -1);
    for (int i = 0; i < R; ++i) {
        const int t = i / n_rg, j = i % n_rg;
        const int rg = (t & 1) ? n_rg - 1 - j : j;
        out.h_rowmap[(size_t)rg * rpg + t] = order[i];
    }

    out.h_slice.assign((size_t)n_rg * nch + 1, 0);
    const int ros = rpg * 4;
    out.ros = ros;
    out.h_rowoff.assign((size_t)n_rg * nch * ros, 0);
    out.h_rec.clear();
    std::vector<int> cursor(R);
    int rec_count = 0, wcap = 0;
    std::vector<int> slot;                         // slot -> index into col_idx, or -1 - column for padding
    for (int rg = 0; rg < n_rg; ++rg) {
        for (int t = 0; t < rpg; ++t) {
            const int r = out.h_rowmap[(size_t)rg * rpg + t];
            if (r >= 0) cursor[r] = p.row_ptr[r];
        }
        for (int c = 0; c < nch; ++c) {
            out.h_slice[(size_t)rg * nch + c] = rec_count;
            int* roff = &out.h_rowoff[((size_t)rg * nch + c) * ros];
            const int c0 = c * kc;
            const int lim = c0 + kc;
            const int nrows = std::min(kc, p.cin - c0);      // channels present in this chunk
            int local = 0;
            for (int t = 0; t < rpg; ++t) {
                int* hd = roff + 4 * t;                      // {segment start (16-byte units), steps, 0, 0}
                hd[0] = local; hd[1] = hd[2] = hd[3] = 0;
                const int r = out.h_rowmap[(size_t)rg * rpg + t];
                if (r < 0) continue;
                const int k = cursor[r];
                const int kend = p.row_ptr[r + 1];
                int k1 = k;
                while (k1 < kend && p.col_idx[k1] < lim) ++k1;
                const int nblk = k1 - k;
                const int nstep = (nblk + 15) / 16;
                hd[1] = nstep;
                cursor[r] = k1;
                if (!nstep) continue;
                if (with_records) {
                    // deal the blocks to the 2*nstep half steps: members of one residue class (column
                    // modulo 8) are spread over the half steps as evenly as the room allows
                    const int noct = 2 * nstep;
                    slot.assign((size_t)noct * 8, 0);
                    std::vector<int> fill(noct, 0);
                    std::vector<int> has((size_t)noct * 8, 0);            // [half step][residue] count
                    std::vector<int> cls[8];
                    for (int kk = k; kk < k1; ++kk) cls[(p.col_idx[kk] - c0) & 7].push_back(kk);
                    int cord[8] = {0, 1, 2, 3, 4, 5, 6, 7};
                    std::stable_sort(cord, cord + 8, [&](int a, int b) { return cls[a].size() > cls[b].size(); });
                    for (int ci = 0; ci < 8; ++ci) {
                        const int res = cord[ci];
                        for (int kk : cls[res]) {
                            int best = -1;
                            for (int o = 0; o < noct; ++o) {
                                if (fill[o] >= 8) continue;
                                if (best < 0 || has[(size_t)o * 8 + res] < has[(size_t)best * 8 + res] ||
                                    (has[(size_t)o * 8 + res] == has[(size_t)best * 8 + res] && fill[o] < fill[best]))
                                    best = o;
                            }
                            slot[(size_t)best * 8 + fill[best]++] = kk;
                            ++has[(size_t)best * 8 + res];
                        }
                    }
                    for (int o = 0; o < noct; ++o) {
                        while (fill[o] < 8) {       // padding: a zero-weight block on a column whose residue is free
                            int col = 0;
                            for (int res = 0; res < 8; ++res)
                                if (!has[(size_t)o * 8 + res] && res < nrows) { col = res; break; }
                            ++has[(size_t)o * 8 + (col & 7)];
                            slot[(size_t)o * 8 + fill[o]++] = -1 - col;
                        }
                    }
                    const size_t base = out.h_rec.size();
                    out.h_rec.resize(base + (size_t)nstep * REC, 0);
                    for (int s = 0; s < nstep; ++s) {
                        unsigned char* rec = &out.h_rec[base + (size_t)s * REC];
                        uint16_t cols[16];
                        uint16_t wv[16][16];                 // [column of the step][output channel of the block]
                        std::memset(wv, 0, sizeof wv);
                        for (int i = 0; i < 16; ++i) {
                            const int e = slot[(size_t)s * 16 + i];
                            if (e < 0) { cols[i] = (uint16_t)(-1 - e); continue; }
                            cols[i] = (uint16_t)(p.col_idx[e] - c0);
                            std::memcpy(wv[i], &p.vals[(size_t)e * g * 2], (size_t)g * 2);
                        }
                        std::memcpy(rec, cols, 32);
                        // B operand of m16n8k16, per tile of 8 output channels: lane l = 4*n + t holds
                        // W[2t][n], W[2t+1][n], W[2t+8][n], W[2t+9][n]
                        for (int nb = 0; nb < gp / 8; ++nb) {
                            uint16_t* frag = reinterpret_cast<uint16_t*>(rec + 32 + nb * 256);
                            for (int l = 0; l < 32; ++l) {
                                const int n = nb * 8 + (l >> 2), tq = l & 3;
                                frag[l * 4 + 0] = wv[2 * tq][n];
                                frag[l * 4 + 1] = wv[2 * tq + 1][n];
                                frag[l * 4 + 2] = wv[2 * tq + 8][n];
                                frag[l * 4 + 3] = wv[2 * tq + 9][n];
                            }
                        }
                    }
                }
                local += nstep * (REC / 16);
            }
            rec_count += local;
            wcap = std::max(wcap, local);
        }
    }
    out.h_slice[(size_t)n_rg * nch] = rec_count;
    out.n_rec = rec_count;
    out.wcap = wcap;
}

}  // namespace alcs

extern "C" {

ALCS_API int alcs_schedule_selfcheck(const alcs_packed* p, int chunk_channels, int row_groups, int warps, int slots,
                                     int64_t* stats)
{
    if (!p || warps < 1 || warps > 32 || slots < 1 || slots > 15) return ALCS_ERR_INVALID_ARG;
    alcs::Schedule sc;
    try {
        alcs::build_schedule_balanced(*p, chunk_channels, row_groups, warps, slots, true, sc);
    } catch (const std::bad_alloc&) {
        return ALCS_ERR_ALLOC;
    }
    const int g = p->g, cap = warps * slots;
    const int REC = alcs::pair_record_bytes(g);
    if (sc.rpg != cap || sc.ros != 4 * cap) return ALCS_ERR_CORRUPT;
    // every block row exactly once in the row map
    // every block row stored by exactly one unit (a whole row or the primary part of a split row), and the
    // exchange slots of a row group used exactly once each
    const size_t nloc = (size_t)sc.n_rg * cap;
    if (sc.h_rowmap.size() != 2 * nloc + sc.n_rg) return ALCS_ERR_CORRUPT;
    std::vector<int> seen(p->rows, 0);
    int64_t secondaries = 0;
    for (int rg = 0; rg < sc.n_rg; ++rg) {
        const int nx = sc.h_rowmap[2 * nloc + rg];
        if (nx < 0 || nx > sc.max_x) return ALCS_ERR_CORRUPT;
        std::vector<int> written(nx, 0), read(nx, 0);
        for (int t = 0; t < cap; ++t) {
            const int v = sc.h_rowmap[(size_t)rg * cap + t];
            const int uw = sc.h_rowmap[nloc + (size_t)rg * cap + t];
            const int role = uw & 15, slot = (uw >> 4) & 0xfff, count = uw >> 16;
            if (v < 0) { if (uw != 0) return ALCS_ERR_CORRUPT; continue; }
            if (v >= p->rows || role > 2) return ALCS_ERR_CORRUPT;
            if (role != 2) ++seen[v];
            if (role == 2) { if (slot >= nx) return ALCS_ERR_CORRUPT; ++written[slot]; ++secondaries; }
            if (role == 1) {
                if (count < 1 || slot + count > nx) return ALCS_ERR_CORRUPT;
                for (int i = 0; i < count; ++i) {
                    ++read[slot + i];
                    // the slot must be written by a part of the same row
                    bool found = false;
                    for (int t2 = 0; t2 < cap; ++t2) {
                        const int uw2 = sc.h_rowmap[nloc + (size_t)rg * cap + t2];
                        if ((uw2 & 15) == 2 && ((uw2 >> 4) & 0xfff) == slot + i && sc.h_rowmap[(size_t)rg * cap + t2] == v) found = true;
                    }
                    if (!found) return ALCS_ERR_CORRUPT;
                }
            }
        }
        for (int i = 0; i < nx; ++i)
            if (written[i] != 1 || read[i] != 1) return ALCS_ERR_CORRUPT;
    }
    for (int r = 0; r < p->rows; ++r)
        if (seen[r] != 1) return ALCS_ERR_CORRUPT;
    // walk every (warp, accumulator set) the way a consumer warp does and rebuild the dense matrix
    std::vector<float> dense((size_t)p->rows * g * p->cin, 0.0f);
    std::vector<uint8_t> hit((size_t)p->rows * p->cin, 0);
    int64_t pairs = 0, max_sched = 0, min_sched = LLONG_MAX, max_rows = 0, min_rows = LLONG_MAX;
    const int nsched = std::min(4, warps);
    for (int rg = 0; rg < sc.n_rg; ++rg) {
        std::vector<int64_t> per_sched(nsched, 0), rows_sched(nsched, 0);
        for (int w = 0; w < warps; ++w)
            for (int s = 0; s < slots; ++s)
                if (sc.h_rowmap[(size_t)rg * cap + alcs::local_row_of(w, s, warps)] >= 0) ++rows_sched[w % nsched];
        for (int c = 0; c < sc.nch; ++c) {
            const size_t slice0 = (size_t)sc.h_slice[(size_t)rg * sc.nch + c] * 16;
            const size_t slice1 = (size_t)sc.h_slice[(size_t)rg * sc.nch + c + 1] * 16;
            const int* hdrs = &sc.h_rowoff[((size_t)rg * sc.nch + c) * sc.ros];
            for (int w = 0; w < warps; ++w) {
                for (int s = 0; s < slots; ++s) {
                    const int lrow = alcs::local_row_of(w, s, warps);
                    const int* hd = hdrs + 4 * lrow;       // {segment start, c0, c1, pairs}
                    const int row = sc.h_rowmap[(size_t)rg * cap + lrow];
                    if (hd[3] < 0 || (row < 0 && hd[3] != 0)) return ALCS_ERR_CORRUPT;
                    int c0 = hd[1], c1 = hd[2];
                    size_t rp = slice0 + (size_t)hd[0] * 16;
                    for (int q = 0; q < hd[3]; ++q) {
                        if (rp + REC > slice1) return ALCS_ERR_CORRUPT;
                        const unsigned char* rec = &sc.h_rec[rp];
                        int h[2];
                        std::memcpy(h, rec, 8);
                        const float* wv = reinterpret_cast<const float*>(rec + (g == 1 ? 8 : 16));
                        const int cols[2] = {c0 + c * sc.kc, c1 + c * sc.kc};
                        for (int b = 0; b < 2; ++b) {
                            if (cols[b] < 0 || cols[b] >= p->cin || cols[b] >= (c + 1) * sc.kc) return ALCS_ERR_CORRUPT;
                            for (int j = 0; j < g; ++j) dense[((size_t)row * g + j) * p->cin + cols[b]] += wv[b * g + j];
                            if (b == 0 || cols[1] != cols[0]) ++hit[(size_t)row * p->cin + cols[b]];
                        }
                        per_sched[w % nsched] += 2;
                        ++pairs;
                        c0 = h[0]; c1 = h[1];
                        rp += REC;
                    }
                }
            }
        }
        for (int k = 0; k < nsched; ++k) {
            max_sched = std::max(max_sched, per_sched[k]); min_sched = std::min(min_sched, per_sched[k]);
            max_rows = std::max(max_rows, rows_sched[k]); min_rows = std::min(min_rows, rows_sched[k]);
        }
    }
    // compare with the canonical storage
    for (int r = 0; r < p->rows; ++r) {
        int k = p->row_ptr[r];
        for (int c = 0; c < p->cin; ++c) {
            const bool kept = k < p->row_ptr[r + 1] && p->col_idx[k] == c;
            if ((hit[(size_t)r * p->cin + c] != 0) != kept) return ALCS_ERR_CORRUPT;
            if (kept && hit[(size_t)r * p->cin + c] != 1) return ALCS_ERR_CORRUPT;
            for (int j = 0; j < g; ++j) {
                float v = 0.0f;
                if (kept) {
                    if (p->dt == ALCS_F32) std::memcpy(&v, &p->vals[((size_t)k * g + j) * 4], 4);
                    else {
                        uint16_t hb;
                        std::memcpy(&hb, &p->vals[((size_t)k * g + j) * 2], 2);
                        v = p->dt == ALCS_F16 ? alcs::half_bits_to_float(hb) : alcs::bfloat16_bits_to_float(hb);
                    }
                }
                const float d = dense[((size_t)r * g + j) * p->cin + c];
                if (std::memcmp(&d, &v, 4) != 0 && !(d == v)) return ALCS_ERR_CORRUPT;
            }
            if (kept) ++k;
        }
    }
    if (stats) {
        stats[0] = sc.n_rg; stats[1] = max_sched; stats[2] = min_sched == LLONG_MAX ? 0 : min_sched;
        stats[3] = pairs; stats[4] = p->nb;
        stats[5] = max_rows; stats[6] = min_rows == LLONG_MAX ? 0 : min_rows;
        stats[7] = secondaries;
    }
    return ALCS_OK;
}

ALCS_API const char* alcs_strerror(int status)
{
    switch (status) {
        case ALCS_OK: return "ALCS_OK";
        case ALCS_ERR_INVALID_ARG: return "ALCS_ERR_INVALID_ARG: null, negative, misaligned or overlapping argument";
        case ALCS_ERR_SHAPE: return "ALCS_ERR_SHAPE: sizes do not fit together or exceed int32 indexing";
        case ALCS_ERR_UNSUPPORTED: return "ALCS_ERR_UNSUPPORTED: group size, dtype or option not implemented";
        case ALCS_ERR_ALLOC: return "ALCS_ERR_ALLOC: allocation failed";
        case ALCS_ERR_CUDA: return "ALCS_ERR_CUDA: CUDA runtime call failed";
        case ALCS_ERR_CORRUPT: return "ALCS_ERR_CORRUPT: serialized blob failed validation";
        case ALCS_ERR_STATE: return "ALCS_ERR_STATE: object not in the required state";
        case ALCS_ERR_TOO_LARGE: return "ALCS_ERR_TOO_LARGE: the problem needs more scratch than alcs_spconv1x1_noalloc has (ALCS_NOALLOC_SCRATCH_BYTES)";
        default: return "unknown ALCS status";
    }
}

ALCS_API const char* alcs_last_cuda_error(void) { return g_cuda_err; }

ALCS_API int alcs_version(void) { return ALCS_VERSION; }

ALCS_API int alcs_pack(const void* w, const uint8_t* block_mask, int cout, int cin, int g, alcs_dtype dt,
              alcs_packed** out)
{
    if (!w || !block_mask || !out) return ALCS_ERR_INVALID_ARG;
    *out = nullptr;
    if (g < 1 || g > 64) return ALCS_ERR_INVALID_ARG;
    if (dt != ALCS_F32 && dt != ALCS_F16 && dt != ALCS_BF16) return ALCS_ERR_UNSUPPORTED;
    if (cout <= 0 || cin <= 0) return ALCS_ERR_SHAPE;
    const int rows = (cout + g - 1) / g;
    // count kept blocks first so that overflow is detected before anything is allocated
    uint64_t nb64 = 0;
    for (size_t i = 0, e = (size_t)rows * cin; i < e; ++i) nb64 += block_mask[i] != 0;
    // the launch schedules pad every (row, 16-channel chunk) segment by at most one block and
    // index values as block * g with int32
    const uint64_t worst = (nb64 + ((uint64_t)rows + 4) * (uint64_t)((cin + 15) / 16)) * (uint64_t)g;
    if (worst >= (uint64_t)std::numeric_limits<int32_t>::max()) return ALCS_ERR_SHAPE;
    alcs_packed* p = new (std::nothrow) alcs_packed();
    if (!p) return ALCS_ERR_ALLOC;
    try {
        p->cout = cout; p->cin = cin; p->g = g; p->rows = rows; p->dt = dt; p->nb = (int)nb64;
        const size_t es = p->elt();
        p->row_ptr.assign(rows + 1, 0);
        p->col_idx.resize(nb64);
        p->vals.assign((size_t)nb64 * g * es, 0);
        const uint8_t* wb = static_cast<const uint8_t*>(w);
        int k = 0;
        for (int r = 0; r < rows; ++r) {
            p->row_ptr[r] = k;
            for (int c = 0; c < cin; ++c) {
                if (!block_mask[(size_t)r * cin + c]) continue;
                p->col_idx[k] = c;
                for (int j = 0; j < g; ++j) {
                    const int co = r * g + j;
                    if (co < cout)
                        std::memcpy(&p->vals[((size_t)k * g + j) * es], wb + ((size_t)co * cin + c) * es, es);
                }
                ++k;
            }
        }
        p->row_ptr[rows] = k;
    } catch (const std::bad_alloc&) {
        delete p;
        return ALCS_ERR_ALLOC;
    }
    *out = p;
    return ALCS_OK;
}

ALCS_API int alcs_unpack(const alcs_packed* p, void* w_out, uint8_t* mask_out)
{
    if (!p) return ALCS_ERR_INVALID_ARG;
    const size_t es = p->elt();
    if (w_out) std::memset(w_out, 0, (size_t)p->cout * p->cin * es);
    if (mask_out) std::memset(mask_out, 0, (size_t)p->rows * p->cin);
    uint8_t* wb = static_cast<uint8_t*>(w_out);
    for (int r = 0; r < p->rows; ++r) {
        for (int k = p->row_ptr[r]; k < p->row_ptr[r + 1]; ++k) {
            const int c = p->col_idx[k];
            if (mask_out) mask_out[(size_t)r * p->cin + c] = 1;
            if (!wb) continue;
            for (int j = 0; j < p->g; ++j) {
                const int co = r * p->g + j;
                if (co < p->cout)
                    std::memcpy(wb + ((size_t)co * p->cin + c) * es, &p->vals[((size_t)k * p->g + j) * es], es);
            }
        }
    }
    return ALCS_OK;
}

ALCS_API int alcs_packed_view(const alcs_packed* p, int* cout, int* cin, int* g, alcs_dtype* dt, int* nb,
                     const int32_t** row_ptr, const int32_t** col_idx, const void** vals)
{
    if (!p) return ALCS_ERR_INVALID_ARG;
    if (cout) *cout = p->cout;
    if (cin) *cin = p->cin;
    if (g) *g = p->g;
    if (dt) *dt = p->dt;
    if (nb) *nb = p->nb;
    if (row_ptr) *row_ptr = p->row_ptr.data();
    if (col_idx) *col_idx = p->col_idx.data();
    if (vals) *vals = p->vals.data();
    return ALCS_OK;
}

ALCS_API int alcs_packed_serialize(const alcs_packed* p, void* buf, size_t* nbytes)
{
    if (!p || !nbytes) return ALCS_ERR_INVALID_ARG;
    const size_t need = sizeof(BlobHeader) + p->row_ptr.size() * 4 + p->col_idx.size() * 4 + p->vals.size();
    if (!buf) { *nbytes = need; return ALCS_OK; }
    if (*nbytes < need) { *nbytes = need; return ALCS_ERR_SHAPE; }
    BlobHeader h{kMagic, kBlobVersion, p->cout, p->cin, p->g, (int32_t)p->dt, p->rows, p->nb};
    uint8_t* o = static_cast<uint8_t*>(buf);
    std::memcpy(o, &h, sizeof h); o += sizeof h;
    std::memcpy(o, p->row_ptr.data(), p->row_ptr.size() * 4); o += p->row_ptr.size() * 4;
    if (!p->col_idx.empty()) std::memcpy(o, p->col_idx.data(), p->col_idx.size() * 4);
    o += p->col_idx.size() * 4;
    if (!p->vals.empty()) std::memcpy(o, p->vals.data(), p->vals.size());
    *nbytes = need;
    return ALCS_OK;
}

ALCS_API int alcs_packed_deserialize(const void* buf, size_t nbytes, alcs_packed** out)
{
    if (!buf || !out) return ALCS_ERR_INVALID_ARG;
    *out = nullptr;
    if (nbytes < sizeof(BlobHeader)) return ALCS_ERR_CORRUPT;
    BlobHeader h;
    std::memcpy(&h, buf, sizeof h);
    if (h.magic != kMagic || h.version != kBlobVersion) return ALCS_ERR_CORRUPT;
    if (h.cout <= 0 || h.cin <= 0 || h.g < 1 || h.g > 64 || h.nb < 0) return ALCS_ERR_CORRUPT;
    if (h.dtype != ALCS_F32 && h.dtype != ALCS_F16 && h.dtype != ALCS_BF16) return ALCS_ERR_CORRUPT;
    if (h.rows != (h.cout + h.g - 1) / h.g) return ALCS_ERR_CORRUPT;
    if ((uint64_t)h.nb > (uint64_t)h.rows * (uint64_t)h.cin) return ALCS_ERR_CORRUPT;
    const size_t es = h.dtype == ALCS_F32 ? 4 : 2;
    const size_t need = sizeof h + ((size_t)h.rows + 1) * 4 + (size_t)h.nb * 4 + (size_t)h.nb * h.g * es;
    if (nbytes != need) return ALCS_ERR_CORRUPT;
    alcs_packed* p = new (std::nothrow) alcs_packed();
    if (!p) return ALCS_ERR_ALLOC;
    try {
        p->cout = h.cout; p->cin = h.cin; p->g = h.g; p->rows = h.rows; p->nb = h.nb;
        p->dt = (alcs_dtype)h.dtype;
        const uint8_t* in = static_cast<const uint8_t*>(buf) + sizeof h;
        p->row_ptr.resize((size_t)h.rows + 1);
        std::memcpy(p->row_ptr.data(), in, p->row_ptr.size() * 4); in += p->row_ptr.size() * 4;
        p->col_idx.resize(h.nb);
        if (h.nb) std::memcpy(p->col_idx.data(), in, (size_t)h.nb * 4);
        in += (size_t)h.nb * 4;
        p->vals.resize((size_t)h.nb * h.g * es);
        if (!p->vals.empty()) std::memcpy(p->vals.data(), in, p->vals.size());
    } catch (const std::bad_alloc&) {
        delete p;
        return ALCS_ERR_ALLOC;
    }
    bool ok = p->row_ptr[0] == 0 && p->row_ptr[h.rows] == h.nb;
    for (int r = 0; ok && r < h.rows; ++r) {
        const int a = p->row_ptr[r], b = p->row_ptr[r + 1];
        if (a > b || b > h.nb || a < 0) { ok = false; break; }
        for (int k = a; k < b; ++k) {
            const int c = p->col_idx[k];
            if (c < 0 || c >= h.cin || (k > a && c <= p->col_idx[k - 1])) { ok = false; break; }
        }
    }
    if (!ok) { delete p; return ALCS_ERR_CORRUPT; }
    *out = p;
    return ALCS_OK;
}

}  // extern "C"
