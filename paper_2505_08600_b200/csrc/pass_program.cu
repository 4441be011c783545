// Builds and checks the static schedule of the persistent streaming kernel (host code only).
#include "pass_program.h"

#include <string.h>

#include <algorithm>

namespace sd {

namespace {

struct Range { int a, b; };

struct MatPlan {
    int n_tiles = 0, kb_per_tile = 0;
    std::vector<std::vector<int>> wave_tiles;     // tiles of each wave
    std::vector<Range> chunk_kb;                  // k blocks of each chunk
    std::vector<int> chunk_dep, chunk_need;       // word and count a chunk waits for (-1: nothing)
    bool dep_prev = false;
    int chunk_major = 0;
};

std::vector<Range> natural_ranges(int n, int parts) {
    parts = std::max(1, std::min(parts, n));
    std::vector<Range> r;
    for (int a = 0; a < parts; ++a) r.push_back({(int)((long long)a * n / parts), (int)((long long)(a + 1) * n / parts)});
    return r;
}

struct Builder {
    const PassShape& S;
    const PassTuning& T;
    int G;
    MatPlan mp[N_MAT];
    int arrive_base[N_MAT] = {0, 0, 0, 0, 0};
    int done_base = 0;
    std::vector<Range> att_waves;                 // kv heads of each attention wave
    int rows_per_block = 1, n_blocks = 1;
    // output
    std::vector<std::vector<PassSeg>> segs[2];
    std::vector<std::vector<PassTask>> tasks[2];
    std::vector<std::vector<std::pair<int, int>>> task_key[2];     // (ready key, order) of each task, for sorting
    std::vector<std::vector<uint16_t>> pieces;
    int slots[2] = {0, 0};
    int rot = 0, rr = 0, block_seq = 0;
    std::string error;

    Builder(const PassShape& s, const PassTuning& t) : S(s), T(t), G(s.grid) {
        for (int k = 0; k < 2; ++k) { segs[k].resize(G); tasks[k].resize(G); task_key[k].resize(G); }
        pieces.resize(G);
    }

    int S_n_acc() const { const int m_pad = (S.m_tok + 15) & ~15; return std::max(2, std::min(16, 512 / m_pad)); }
    int done_word(int mat, int wave) const { return done_base + mat * PASS_MAX_WAVES + wave; }

    void plan() {
        const int d = S.d, hd = S.hd, H = S.H, Hkv = S.Hkv, grp = H / Hkv, F = S.F;
        const int n_qkv = (H + 2 * Hkv) * hd;
        mp[MAT_QKV].n_tiles = (n_qkv + 127) / 128; mp[MAT_QKV].kb_per_tile = d / 64;
        mp[MAT_WO].n_tiles = (d + 127) / 128;      mp[MAT_WO].kb_per_tile = H * hd / 64;
        mp[MAT_GU].n_tiles = 2 * F / 128;          mp[MAT_GU].kb_per_tile = d / 64;
        mp[MAT_DN].n_tiles = (d + 127) / 128;      mp[MAT_DN].kb_per_tile = F / 64;
        mp[MAT_LM].n_tiles = (S.V + 127) / 128;    mp[MAT_LM].kb_per_tile = d / 64;
        int w = 0;
        for (int m = 0; m < 4; ++m) { arrive_base[m] = w; w += mp[m].n_tiles; }
        arrive_base[MAT_LM] = 0;                                  // the tail has words of its own
        done_base = w;
        for (int m = 0; m < N_MAT; ++m) mp[m].chunk_major = T.chunk_major[m];

        // ---- waves
        // QKV: by groups of kv heads, so that a wave holds the query, key and value rows of whole heads
        const int align = std::max(1, 128 / hd);                  // kv heads per 128-row tile
        int wq = std::max(1, std::min(T.waves[MAT_QKV], PASS_MAX_WAVES));
        const bool exact = Hkv % align == 0 && (H * hd) % 128 == 0 && (Hkv * hd) % 128 == 0 && n_qkv % 128 == 0;
        if (!exact) wq = 1;
        const int units = exact ? Hkv / align : 1;
        wq = std::min(wq, units);
        att_waves.clear();
        for (int j = 0; j < wq; ++j)
            att_waves.push_back(exact ? Range{align * (int)((long long)j * units / wq), align * (int)((long long)(j + 1) * units / wq)} : Range{0, Hkv});
        mp[MAT_QKV].wave_tiles.assign(wq, {});
        for (int j = 0; j < wq; ++j) {
            auto& v = mp[MAT_QKV].wave_tiles[j];
            if (!exact) { for (int t = 0; t < mp[MAT_QKV].n_tiles; ++t) v.push_back(t); break; }
            const int g0 = att_waves[j].a, g1 = att_waves[j].b;
            for (int t = g0 * grp * hd / 128; t < g1 * grp * hd / 128; ++t) v.push_back(t);
            for (int part = 0; part < 2; ++part) {
                const int row0 = H * hd + part * Hkv * hd;
                for (int t = (row0 + g0 * hd) / 128; t < (row0 + g1 * hd) / 128; ++t) v.push_back(t);
            }
        }
        for (int m : {MAT_WO, MAT_GU, MAT_DN, MAT_LM}) {
            const auto r = natural_ranges(mp[m].n_tiles, std::min(T.waves[m], PASS_MAX_WAVES));
            mp[m].wave_tiles.assign(r.size(), {});
            for (size_t a = 0; a < r.size(); ++a) for (int t = r[a].a; t < r[a].b; ++t) mp[m].wave_tiles[a].push_back(t);
        }

        // ---- chunks: the k blocks that each wave of the producing step makes available
        auto from_d_tiles = [&](int consumer, int producer, bool prev) {      // producer tiles are 128 columns of a d-wide row
            MatPlan& c = mp[consumer];
            const MatPlan& p = mp[producer];
            c.dep_prev = prev;
            for (size_t a = 0; a < p.wave_tiles.size(); ++a) {
                const int t0 = p.wave_tiles[a].front(), t1 = p.wave_tiles[a].back() + 1;
                c.chunk_kb.push_back({std::min(2 * t0, c.kb_per_tile), std::min(2 * t1, c.kb_per_tile)});
                c.chunk_dep.push_back(done_word(producer, (int)a));
                c.chunk_need.push_back((int)p.wave_tiles[a].size());
            }
        };
        from_d_tiles(MAT_QKV, MAT_DN, true);
        from_d_tiles(MAT_GU, MAT_WO, false);
        from_d_tiles(MAT_LM, MAT_DN, true);
        {   // down projection: tile t of gate/up makes k block t of the activation
            MatPlan& c = mp[MAT_DN];
            const MatPlan& p = mp[MAT_GU];
            for (size_t a = 0; a < p.wave_tiles.size(); ++a) {
                c.chunk_kb.push_back({p.wave_tiles[a].front(), p.wave_tiles[a].back() + 1});
                c.chunk_dep.push_back(done_word(MAT_GU, (int)a));
                c.chunk_need.push_back((int)p.wave_tiles[a].size());
            }
        }
        rows_per_block = std::max(1, std::min(S.rows_per_seq, 16 / grp));
        const int bps = (S.rows_per_seq + rows_per_block - 1) / rows_per_block;
        n_blocks = (S.m_tok / S.rows_per_seq) * bps;
        {   // Wo: the heads of an attention wave are consecutive columns of its input
            MatPlan& c = mp[MAT_WO];
            for (size_t j = 0; j < att_waves.size(); ++j) {
                c.chunk_kb.push_back({att_waves[j].a * grp * hd / 64, att_waves[j].b * grp * hd / 64});
                c.chunk_dep.push_back(done_word(4, (int)j));
                c.chunk_need.push_back((att_waves[j].b - att_waves[j].a) * n_blocks);
            }
        }
    }

    // Splits the blocks of one matrix over the CTAs; kind 0 = layer body, 1 = tail.
    void emit_matrix(int m, int kind) {
        MatPlan& P = mp[m];
        const int W = (int)P.wave_tiles.size(), C = (int)P.chunk_kb.size();
        std::vector<std::vector<uint16_t>> tile_pieces(P.n_tiles);
        std::vector<int> wave_last_block(W, 0), wave_rot(W, -1);
        int next_slot = 0;
        std::vector<size_t> seg0(G);
        for (int c = 0; c < G; ++c) seg0[c] = segs[kind][c].size();
        // ---- pass 1: the blocks in ring order, each split evenly over the CTAs.  The chunks of a wave are cut at the same
        //      places, so that a CTA meets the same tiles again in the wave's next chunk and keeps accumulating.
        for (int idx = 0; idx < W * C; ++idx) {
            const int a = P.chunk_major ? idx % W : idx / C, j = P.chunk_major ? idx / W : idx % C;
            const auto& tl = P.wave_tiles[a];
            const int nk = P.chunk_kb[j].b - P.chunk_kb[j].a;
            const long long Tb = (long long)tl.size() * nk;
            wave_last_block[a] = block_seq;
            ++block_seq;
            if (Tb == 0) continue;
            if (wave_rot[a] < 0) { wave_rot[a] = rot; rot = (int)((rot + (Tb % G) * C) % G); }
            const long long base = Tb / G;
            const int rem = (int)(Tb % G);
            for (int pos = 0; pos < G; ++pos) {
                const int cta = (pos + wave_rot[a]) % G;
                const long long u0 = pos * base + std::min(pos, rem), u1 = u0 + base + (pos < rem ? 1 : 0);
                for (long long u = u0; u < u1;) {
                    const int ti = (int)(u / nk), k0 = (int)(u % nk);
                    const int n = (int)std::min<long long>(nk - k0, u1 - u);
                    PassSeg sg;
                    memset(&sg, 0, sizeof(sg));
                    sg.tile = (uint16_t)tl[ti]; sg.kb0 = (uint16_t)(P.chunk_kb[j].a + k0); sg.n_kb = (uint16_t)n; sg.mat = (uint8_t)m;
                    sg.flags = (uint8_t)((P.chunk_dep[j] >= 0 ? SEG_DEP : 0) | (P.dep_prev ? SEG_DEP_PREV : 0));
                    sg.dep = (uint16_t)std::max(0, P.chunk_dep[j]); sg.dep_need = (uint16_t)P.chunk_need[j];
                    sg.arrive = (uint16_t)(arrive_base[m] + tl[ti]);
                    segs[kind][cta].push_back(sg);
                    u += n;
                }
            }
        }
        // ---- pass 2: accumulators.  A CTA's segments of one tile share one accumulator in tensor memory from the first
        //      to the last of them; only the last one leaves a piece in the workspace.
        for (int c = 0; c < G; ++c) {
            std::vector<PassSeg>& v = segs[kind][c];
            std::vector<int> last_of(P.n_tiles, -1), acc_of(P.n_tiles, -1);
            for (size_t i = seg0[c]; i < v.size(); ++i) last_of[v[i].tile] = (int)i;
            std::vector<int> free_acc;
            for (int k = 0; k < S_n_acc(); ++k) free_acc.push_back(k);
            for (size_t i = seg0[c]; i < v.size(); ++i) {
                const int t = v[i].tile;
                if (acc_of[t] < 0) {
                    if (free_acc.empty()) { error = "a CTA would hold more accumulators than tensor memory has room for"; return; }
                    acc_of[t] = free_acc.front(); free_acc.erase(free_acc.begin());
                    v[i].flags |= SEG_FIRST;
                }
                v[i].flags |= (uint8_t)(acc_of[t] << 4);
                if (last_of[t] == (int)i) {
                    v[i].flags |= SEG_LAST;
                    if (next_slot >= 65535) { error = "too many workspace slots"; return; }
                    v[i].slot = (uint16_t)next_slot;
                    tile_pieces[t].push_back((uint16_t)next_slot);
                    ++next_slot;
                    free_acc.push_back(acc_of[t]);        // reused last: the epilogue has long drained it by then
                }
            }
        }
        slots[m & 1] = std::max(slots[m & 1], next_slot);
        // the tasks that sum the pieces of a tile and apply the step after the GEMM, wave by wave
        for (int a = 0; a < W; ++a)
            for (int t : P.wave_tiles[a]) {
                const int cta = rr++ % G;
                PassTask tk;
                memset(&tk, 0, sizeof(tk));
                tk.item = (uint32_t)t; tk.kind = TASK_REDUCE; tk.mat = (uint16_t)m;
                tk.wait_word = (uint16_t)(arrive_base[m] + t); tk.wait_need = (uint16_t)tile_pieces[t].size();
                tk.done_word = m == MAT_LM ? NO_WORD : (uint16_t)done_word(m, a);
                tk.piece0 = (uint32_t)pieces[cta].size(); tk.n_pieces = (uint16_t)tile_pieces[t].size();
                for (uint16_t s : tile_pieces[t]) pieces[cta].push_back(s);
                task_key[kind][cta].push_back({2 * wave_last_block[a], (int)tasks[kind][cta].size()});
                tasks[kind][cta].push_back(tk);
            }
        if (m == MAT_QKV) {
            // attention items of a wave become ready once the wave's query / key / value tiles are reduced
            for (int j = 0; j < W; ++j)
                for (int b = 0; b < n_blocks; ++b)
                    for (int kvh = att_waves[j].a; kvh < att_waves[j].b; ++kvh)
                        for (int sp = 0; sp < S.n_splits; ++sp) {
                            const int cta = rr++ % G;
                            PassTask tk;
                            memset(&tk, 0, sizeof(tk));
                            tk.item = (uint32_t)((b * S.Hkv + kvh) * S.n_splits + sp); tk.kind = TASK_ATTENTION; tk.mat = MAT_ATT;
                            tk.wait_word = (uint16_t)done_word(MAT_QKV, j); tk.wait_need = (uint16_t)P.wave_tiles[j].size();
                            tk.done_word = (uint16_t)done_word(4, j);
                            task_key[0][cta].push_back({2 * wave_last_block[j] + 1, (int)tasks[0][cta].size()});
                            tasks[0][cta].push_back(tk);
                        }
        }
    }

    void sort_tasks(int kind) {
        for (int c = 0; c < G; ++c) {
            auto& k = task_key[kind][c];
            std::vector<int> order(k.size());
            for (size_t i = 0; i < k.size(); ++i) order[i] = (int)i;
            std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return k[x].first < k[y].first; });
            std::vector<PassTask> t2;
            for (int i : order) t2.push_back(tasks[kind][c][i]);
            tasks[kind][c] = t2;
        }
    }
};

}  // namespace

PassTuning default_pass_tuning(const PassShape& s) {
    (void)s;
    PassTuning t;
    const int w[N_MAT] = {2, 1, 4, 1, 2};              // measured best on the 7B shape (QKV and gate/up in waves, the thin Wo and down whole)
    for (int m = 0; m < N_MAT; ++m) { t.waves[m] = w[m]; t.chunk_major[m] = 0; }
    return t;
}

bool pass_shape_supported(const PassShape& s) {
    if (s.n_layers < 1 || s.grid < 1 || s.m_tok < 1 || s.m_tok > 256 || s.rows_per_seq < 1 || s.m_tok % s.rows_per_seq) return false;
    if (s.hd != 64 && s.hd != 128) return false;
    if (s.H % s.Hkv || s.H / s.Hkv > 16) return false;
    if (s.d % 64 || s.F % 64 || (s.H * s.hd) % 64 || s.d > 128 * 64) return false;
    if (s.n_splits < 1 || s.n_splits > 32) return false;
    return true;
}

PassProgram build_pass_program(const PassShape& s, const PassTuning& t) {
    PassProgram out;
    out.words_per_layer = out.total_words = out.max_seg = out.max_section = 0;
    out.slots[0] = out.slots[1] = 0;
    out.rows_per_block = out.n_blocks = 1;
    out.units_per_layer = 0;
    if (!pass_shape_supported(s)) { out.error = "shape not supported"; return out; }
    Builder B(s, t);
    B.plan();
    for (int m = 0; m < 4 && B.error.empty(); ++m) B.emit_matrix(m, 0);
    if (s.want_logits && B.error.empty()) { B.block_seq = 0; B.emit_matrix(MAT_LM, 1); }
    if (!B.error.empty()) { out.error = B.error; return out; }
    B.sort_tasks(0); B.sort_tasks(1);
    out.words_per_layer = B.done_base + 5 * PASS_MAX_WAVES;
    out.total_words = s.n_layers * out.words_per_layer + (s.want_logits ? B.mp[MAT_LM].n_tiles : 0);
    if (out.words_per_layer >= 65535) { out.error = "too many words per layer"; return out; }
    out.slots[0] = B.slots[0]; out.slots[1] = B.slots[1];
    out.rows_per_block = B.rows_per_block; out.n_blocks = B.n_blocks;
    for (int m = 0; m < 4; ++m) out.units_per_layer += (int64_t)B.mp[m].n_tiles * B.mp[m].kb_per_tile;
    const int G = s.grid;
    std::vector<uint32_t> off(G + 1, 0);
    std::vector<std::vector<uint8_t>> sections(G);
    for (int c = 0; c < G; ++c) {
        PassCtaHeader h;
        memset(&h, 0, sizeof(h));
        std::vector<uint8_t>& sec = sections[c];
        sec.resize(sizeof(h));
        auto append = [&](const void* p, size_t n) { const size_t o = sec.size(); sec.resize(o + ((n + 15) & ~(size_t)15)); memcpy(sec.data() + o, p, n); return (uint32_t)o; };
        for (int k = 0; k < 2; ++k) {
            h.n_seg[k] = (uint32_t)B.segs[k][c].size(); h.n_task[k] = (uint32_t)B.tasks[k][c].size();
            h.seg_off[k] = append(B.segs[k][c].data(), B.segs[k][c].size() * sizeof(PassSeg));
            h.task_off[k] = append(B.tasks[k][c].data(), B.tasks[k][c].size() * sizeof(PassTask));
            out.max_seg = std::max(out.max_seg, (int)h.n_seg[k]);
        }
        h.piece_off = append(B.pieces[c].data(), B.pieces[c].size() * sizeof(uint16_t));
        h.bytes = (uint32_t)sec.size();
        memcpy(sec.data(), &h, sizeof(h));
        out.max_section = std::max(out.max_section, (int)sec.size());
        off[c + 1] = off[c] + (uint32_t)sec.size();
    }
    const size_t table = ((size_t)(G + 1) * 4 + 15) & ~(size_t)15;
    out.blob.resize(table + off[G]);
    for (int c = 0; c <= G; ++c) { const uint32_t v = (uint32_t)table + off[c]; memcpy(out.blob.data() + 4 * c, &v, 4); }
    for (int c = 0; c < G; ++c) memcpy(out.blob.data() + table + off[c], sections[c].data(), sections[c].size());
    const std::string chk = check_pass_program(s, out);
    if (!chk.empty()) out.error = chk;
    return out;
}

std::string check_pass_program(const PassShape& s, const PassProgram& p) {
    const int G = s.grid, L = s.n_layers, WPL = p.words_per_layer;
    const int n_it = L + (s.want_logits ? 1 : 0);
    std::vector<uint32_t> words((size_t)p.total_words + 1, 0);
    struct Cta { const PassCtaHeader* h; const uint8_t* base; int it_s = 0, si = 0, it_t = 0, ti = 0; };
    std::vector<Cta> ctas(G);
    for (int c = 0; c < G; ++c) {
        uint32_t o;
        memcpy(&o, p.blob.data() + 4 * c, 4);
        ctas[c].base = p.blob.data() + o;
        ctas[c].h = reinterpret_cast<const PassCtaHeader*>(ctas[c].base);
    }
    // coverage of one layer and of the tail: every (tile, k block) exactly once
    const int kbpt[N_MAT] = {s.d / 64, s.H * s.hd / 64, s.d / 64, s.F / 64, s.d / 64};
    const int nt[N_MAT] = {((s.H + 2 * s.Hkv) * s.hd + 127) / 128, (s.d + 127) / 128, 2 * s.F / 128, (s.d + 127) / 128, (s.V + 127) / 128};
    for (int m = 0; m < N_MAT; ++m) {
        if (m == MAT_LM && !s.want_logits) continue;
        std::vector<uint8_t> seen((size_t)nt[m] * kbpt[m], 0);
        for (int c = 0; c < G; ++c) {
            const int k = m == MAT_LM ? 1 : 0;
            const PassSeg* sg = reinterpret_cast<const PassSeg*>(ctas[c].base + ctas[c].h->seg_off[k]);
            for (uint32_t i = 0; i < ctas[c].h->n_seg[k]; ++i) {
                if (sg[i].mat != m) continue;
                if (sg[i].tile >= nt[m] || sg[i].kb0 + sg[i].n_kb > kbpt[m] || sg[i].n_kb == 0) return "segment out of range";
                if ((sg[i].flags & SEG_LAST) && (int)sg[i].slot >= p.slots[m & 1]) return "slot out of range";
                for (int j = 0; j < sg[i].n_kb; ++j) {
                    uint8_t& b = seen[(size_t)sg[i].tile * kbpt[m] + sg[i].kb0 + j];
                    if (b) return "a weight block is scheduled twice";
                    b = 1;
                }
            }
        }
        for (uint8_t b : seen) if (!b) return "a weight block is not scheduled";
    }
    // replay
    auto word_of = [&](int it, uint16_t w, bool prev) { return (size_t)(prev ? it - 1 : it) * WPL + w; };
    bool progress = true;
    long long remaining = 0;
    const int rpb = std::max(1, std::min(s.rows_per_seq, 16 / (s.H / s.Hkv)));
    const int n_items = (s.m_tok / s.rows_per_seq) * ((s.rows_per_seq + rpb - 1) / rpb) * s.Hkv;
    std::vector<int> slices_in((size_t)n_it * n_items, 0);       // slices of each attention item that have delivered
    for (int c = 0; c < G; ++c)
        remaining += (long long)L * (ctas[c].h->n_seg[0] + ctas[c].h->n_task[0]) + (s.want_logits ? ctas[c].h->n_seg[1] + ctas[c].h->n_task[1] : 0);
    while (progress && remaining > 0) {
        progress = false;
        for (int c = 0; c < G; ++c) {
            Cta& A = ctas[c];
            for (;;) {                                    // the ring: segments in order
                if (A.it_s >= n_it) break;
                const int k = A.it_s == L ? 1 : 0;
                if (A.si >= (int)A.h->n_seg[k]) { ++A.it_s; A.si = 0; continue; }
                const PassSeg& sg = reinterpret_cast<const PassSeg*>(A.base + A.h->seg_off[k])[A.si];
                const bool prev = sg.flags & SEG_DEP_PREV;
                if ((sg.flags & SEG_DEP) && !(prev && A.it_s == 0) && words[word_of(A.it_s, sg.dep, prev)] < sg.dep_need) break;
                if (sg.flags & SEG_LAST) words[word_of(A.it_s, sg.arrive, false)] += 1;
                ++A.si; --remaining; progress = true;
            }
            for (;;) {                                    // the task warps: tasks in order
                if (A.it_t >= n_it) break;
                const int k = A.it_t == L ? 1 : 0;
                if (A.ti >= (int)A.h->n_task[k]) { ++A.it_t; A.ti = 0; continue; }
                const PassTask& tk = reinterpret_cast<const PassTask*>(A.base + A.h->task_off[k])[A.ti];
                const uint32_t have = words[word_of(A.it_t, tk.wait_word, false)];
                if (have < tk.wait_need) break;
                if (tk.kind == TASK_REDUCE && have != tk.wait_need) return "a tile received more pieces than its task expects";
                bool counts = tk.done_word != NO_WORD;
                if (tk.kind == TASK_ATTENTION) {
                    // an item's slice 0 merges the others: it finishes (and the item counts) only when they have all delivered
                    if (tk.item / (uint32_t)s.n_splits >= (uint32_t)n_items) return "attention item out of range";
                    int& in = slices_in[(size_t)A.it_t * n_items + tk.item / (uint32_t)s.n_splits];
                    if (tk.item % (uint32_t)s.n_splits == 0u) { if (in < s.n_splits - 1) break; }
                    else { ++in; counts = false; }
                }
                if (counts) words[word_of(A.it_t, tk.done_word, false)] += 1;
                ++A.ti; --remaining; progress = true;
            }
        }
    }
    if (remaining > 0) return "the schedule cannot complete: a wait is never satisfied";
    for (int c = 0; c < G; ++c)                               // every wait expects exactly what is delivered
        for (int k = 0; k < (s.want_logits ? 2 : 1); ++k) {
            const PassSeg* sg = reinterpret_cast<const PassSeg*>(ctas[c].base + ctas[c].h->seg_off[k]);
            const int it = k == 1 ? L : (L > 1 ? 1 : 0);
            for (uint32_t i = 0; i < ctas[c].h->n_seg[k]; ++i) {
                const bool prev = sg[i].flags & SEG_DEP_PREV;
                if (!(sg[i].flags & SEG_DEP) || (prev && it == 0)) continue;
                if (words[word_of(it, sg[i].dep, prev)] != sg[i].dep_need) return "a chunk waits for a count other than the one delivered";
            }
        }
    return "";
}

}  // namespace sd
