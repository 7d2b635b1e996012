// Layout planner: compiles (model spec, flat source layout, rollout layout, tp, rank) into the
// segment table the gather/cast kernel walks.  Host only.
#include <algorithm>
#include <cstdlib>
#include <cstring>

#include "dr_internal.h"

namespace dr {
namespace {

struct Param {  // one parameter of the training-side flat buffer
    uint64_t rows, cols, off;
};

struct Builder {
    const dr_model_spec& s;
    uint64_t A;
    uint64_t next = 0;
    explicit Builder(const dr_model_spec& spec, uint64_t align) : s(spec), A(align) {}
    Param take(uint64_t rows, uint64_t cols)
    {
        uint64_t off = (next + A - 1) / A * A;
        next = off + rows * cols;
        return Param{rows, cols, off};
    }
};

// The linear weights that DR_FP8_E4M3_B128 quantises; everything else stays bf16.
bool is_linear_weight(const std::string& name)
{
    size_t dot = name.rfind('.');
    std::string leaf = dot == std::string::npos ? name : name.substr(dot + 1);
    return leaf == "qkv" || leaf == "o" || leaf == "gate_up" || leaf == "down" || leaf == "w13" || leaf == "w2";
}

struct Emit {
    dr_plan* p;
    uint64_t arena = 0;
    uint32_t group = 0;  // group of the tensors begun from now on
    uint64_t align_up(uint64_t x) const
    {
        uint64_t a = p->dst.arena_align_bytes;
        return (x + a - 1) / a * a;
    }
    // Close the tensor being built: a quantised tensor is followed by its block scales.
    void finish()
    {
        if (p->tensors.empty()) return;
        Tensor& t = p->tensors.back();
        if (!t.quant || t.alias_of >= 0) return;
        QTensor& q = p->qtensors.back();
        q.rows = (uint32_t)t.rows;
        q.nbc = (uint32_t)((t.cols + 127) / 128);
        q.n_parts = (uint32_t)p->qparts.size() - q.part0;
        t.scale_off = align_up(t.arena_off + t.rows * t.cols);
        q.scale_off = t.scale_off;
        arena = t.scale_off + ((t.rows + 127) / 128) * q.nbc * 4;
    }
    void begin(const std::string& name, uint64_t cols)
    {
        finish();
        Tensor t;
        t.name = name;
        t.cols = cols;
        t.group = group;
        t.quant = p->fp8 && is_linear_weight(name);
        t.es = t.quant ? 1 : p->elem_size;
        arena = align_up(arena);
        t.arena_off = arena;
        p->tensors.push_back(t);
        if (t.quant) {
            QTensor q{};
            q.payload_off = t.arena_off;
            q.cols = (uint32_t)cols;
            q.part0 = (uint32_t)p->qparts.size();
            q.aligned = (cols % 8 == 0 && t.arena_off % 8 == 0) ? 1 : 0;
            p->qtensors.push_back(q);
        }
    }
    // Append rows [r0, r0+nr) x cols [c0, c0+cols) of parameter q below what the tensor already holds.
    void block(const Param& q, uint64_t r0, uint64_t c0, uint64_t nr)
    {
        Tensor& t = p->tensors.back();
        if (t.quant) {  // recorded as a row-block part of a quantised tensor, not as a copy segment
            if (nr) {
                QPart qp{};
                qp.src_off = q.off + r0 * q.cols + c0;
                qp.dst_row0 = (uint32_t)t.rows;
                qp.rows = (uint32_t)nr;
                qp.src_stride = (uint32_t)q.cols;
                if (qp.src_off % 8 || q.cols % 8) p->qtensors.back().aligned = 0;
                p->qparts.push_back(qp);
            }
            t.rows += nr;
            arena = t.arena_off + t.rows * t.cols;
            return;
        }
        HostSeg g{};
        g.dst_off = t.arena_off + t.rows * t.cols * p->elem_size;
        g.src_off = q.off + r0 * q.cols + c0;
        g.tensor = (uint32_t)(p->tensors.size() - 1);
        g.group = t.group;
        if (t.cols == q.cols) {  // whole rows: one contiguous run
            g.rows = 1;
            g.row_len = nr * t.cols;
            g.src_stride = g.dst_stride = g.row_len;
        } else {
            g.rows = nr;
            g.row_len = t.cols;
            g.src_stride = q.cols;
            g.dst_stride = t.cols;
        }
        if (g.rows != 0 && g.row_len != 0) p->segs.push_back(g);
        t.rows += nr;
        arena = t.arena_off + t.rows * t.cols * p->elem_size;
    }
    // The tensor owns `rows` rows in the arena even if fewer have a source (vocabulary padding).
    void pad_rows(uint64_t rows)
    {
        Tensor& t = p->tensors.back();
        if (rows > t.rows) t.rows = rows;
        arena = t.arena_off + t.rows * t.cols * p->elem_size;
    }
};

bool contiguous(const HostSeg& g) { return g.rows == 1; }

// Merge runs that are adjacent on both sides (q|k|v at tp = 1, gate_e|up_e, ...).
void merge_adjacent(std::vector<HostSeg>& v, uint32_t es)
{
    std::vector<HostSeg> out;
    for (const HostSeg& g : v) {
        if (!out.empty()) {
            HostSeg& b = out.back();
            if (b.group == g.group && contiguous(b) && contiguous(g) && b.src_off + b.row_len == g.src_off &&
                b.dst_off + b.row_len * es == g.dst_off) {
                b.row_len += g.row_len;
                b.src_stride = b.dst_stride = b.row_len;
                continue;
            }
        }
        out.push_back(g);
    }
    v.swap(out);
}

// Keep only the part of every segment whose source lies in [lo, hi); rebase sources to lo.
void clip_to_shard(std::vector<HostSeg>& v, uint64_t lo, uint64_t hi, uint32_t es)
{
    std::vector<HostSeg> out;
    auto run = [&](const HostSeg& g, uint64_t s0, uint64_t s1, uint64_t row) {  // source range of one row
        uint64_t a = std::max(s0, lo), b = std::min(s1, hi);
        if (a >= b) return;
        HostSeg c = g;
        c.rows = 1;
        c.row_len = b - a;
        c.src_stride = c.dst_stride = c.row_len;
        c.src_off = a - lo;
        c.dst_off = g.dst_off + (row * g.dst_stride + (a - s0)) * es;
        out.push_back(c);
    };
    for (const HostSeg& g : v) {
        if (contiguous(g)) {
            run(g, g.src_off, g.src_off + g.row_len, 0);
            continue;
        }
        uint64_t i = 0;
        while (i < g.rows) {
            uint64_t s0 = g.src_off + i * g.src_stride, s1 = s0 + g.row_len;
            if (s1 <= lo) {  // rows wholly below the shard: skip them all at once
                uint64_t skip = (lo - s1) / g.src_stride + 1;
                i += std::min(skip, g.rows - i);
                continue;
            }
            if (s0 >= hi) break;
            if (s0 >= lo && s1 <= hi) {  // a block of rows wholly inside the shard
                uint64_t n = std::min(g.rows - i, (hi - s1) / g.src_stride + 1);
                HostSeg c = g;
                c.rows = n;
                c.src_off = s0 - lo;
                c.dst_off = g.dst_off + i * g.dst_stride * es;
                out.push_back(c);
                i += n;
            } else {  // a row cut by a shard boundary
                run(g, s0, s1, i);
                ++i;
            }
        }
    }
    v.swap(out);
}

uint32_t vec_class(uint64_t src_off, uint64_t dst_off, uint32_t es, uint64_t arena_unit)
{
    if (dst_off % arena_unit) return 0;
    (void)es;
    if (src_off % 8 == 0) return kSegVec32;
    if (src_off % 4 == 0) return kSegVec16;
    return 0;
}

// Split every segment into pieces the kernel can treat uniformly: a vector body whose rows all start
// on aligned addresses and hold a multiple of 8 elements, and scalar head/tail runs around it.
void classify(std::vector<HostSeg>& v, uint32_t es)
{
    const uint64_t arena_unit = 8ull * es;  // bytes of 8 rollout elements: 16 (bf16) or 32 (fp32)
    std::vector<HostSeg> out;
    auto emit_run = [&](HostSeg c, uint64_t src, uint64_t dst, uint64_t n, uint32_t flags) {
        while (n) {
            uint64_t take = std::min(n, kMaxSegElems);
            c.rows = 1;
            c.row_len = take;
            c.src_stride = c.dst_stride = take;
            c.src_off = src;
            c.dst_off = dst;
            c.flags = flags | kSegContiguous;
            out.push_back(c);
            src += take;
            dst += take * es;
            n -= take;
        }
    };
    for (const HostSeg& g : v) {
        if (contiguous(g)) {
            // head: elements until the arena address reaches a unit boundary
            uint64_t mis = g.dst_off % arena_unit;
            uint64_t head = mis ? (arena_unit - mis) / es : 0;
            if (mis % es) head = g.row_len;  // arena offset not even element-aligned: all scalar
            head = std::min(head, g.row_len);
            uint64_t body = (g.row_len - head) / 8 * 8;
            uint32_t cls = body ? vec_class(g.src_off + head, g.dst_off + head * es, es, arena_unit) : 0;
            if (!cls) {
                emit_run(g, g.src_off, g.dst_off, g.row_len, 0);
                continue;
            }
            uint64_t tail = g.row_len - head - body;
            if (head) emit_run(g, g.src_off, g.dst_off, head, 0);
            emit_run(g, g.src_off + head, g.dst_off + head * es, body, cls);
            if (tail) emit_run(g, g.src_off + head + body, g.dst_off + (head + body) * es, tail, 0);
        } else {
            HostSeg c = g;
            uint32_t cls = vec_class(g.src_off, g.dst_off, es, arena_unit);
            bool ok = cls && g.row_len % 8 == 0 && g.dst_stride % 8 == 0;
            if (ok && g.src_stride % 8 != 0) cls = (g.src_stride % 4 == 0) ? (uint32_t)kSegVec16 : 0u;
            c.flags = (ok && cls) ? cls : 0;
            out.push_back(c);
        }
    }
    v.swap(out);
}

}  // namespace

// Device table, tile prefix and hint table for a list of classified segments.
int build_tables(const std::vector<HostSeg>& segs, Tables* out)
{
    uint64_t tiles = 0, moved = 0;
    out->segs.clear();
    out->segs.reserve(segs.size());
    for (const HostSeg& g : segs) {
        DevSeg d{};
        d.dst_off = g.dst_off;
        d.src_off = g.src_off;
        d.tile0 = tiles;
        d.units_per_row = (uint32_t)((g.row_len + kUnitElems - 1) / kUnitElems);
        uint64_t units = g.rows * d.units_per_row;
        if (units > 0xFFFFFFFFull || g.src_stride > 0xFFFFFFFFull || g.dst_stride > 0xFFFFFFFFull) {
            set_error("segment too large for the 32-bit unit index");
            return DR_ERR_UNSUPPORTED;
        }
        d.n_units = (uint32_t)units;
        d.row_len = (uint32_t)g.row_len;
        d.src_stride = (uint32_t)g.src_stride;
        d.dst_stride = (uint32_t)g.dst_stride;
        d.flags = g.flags;
        out->segs.push_back(d);
        tiles += (units + kTileUnits - 1) / kTileUnits;
        moved += g.rows * g.row_len;
    }
    // hint table: segment of every (1 << hint_shift)-th tile
    out->hint_shift = 0;
    while (((tiles + (1ull << out->hint_shift) - 1) >> out->hint_shift) > kMaxHints) ++out->hint_shift;
    const uint64_t n_hints = (tiles + (1ull << out->hint_shift) - 1) >> out->hint_shift;
    out->hints.assign(n_hints ? n_hints : 1, 0);
    uint32_t si = 0;
    for (uint64_t h = 0; h < n_hints; ++h) {
        const uint64_t tile = h << out->hint_shift;
        while (si + 1 < out->segs.size() && out->segs[si + 1].tile0 <= tile) ++si;
        out->hints[h] = si;
    }
    out->n_tiles = tiles;
    out->elems = moved;
    return DR_OK;
}

// The part of a plan whose source elements lie in [lo, hi), with sources rebased to lo: what one chunk of
// a streamed source can produce on its own.
std::vector<HostSeg> window_segments(const std::vector<HostSeg>& segs, uint64_t lo, uint64_t hi, uint32_t es)
{
    std::vector<HostSeg> v;
    for (const HostSeg& g : segs) {  // cheap reject before the exact clip
        uint64_t a = g.src_off, b = g.src_off + (g.rows - 1) * g.src_stride + g.row_len;
        if (b > lo && a < hi) v.push_back(g);
    }
    clip_to_shard(v, lo, hi, es);
    classify(v, es);
    return v;
}

// Arena byte ranges the plan writes, ascending, touching ranges merged.
std::vector<dr_range> plan_ranges(const dr_plan* p)
{
    const uint64_t es = p->elem_size;
    std::vector<dr_range> v;
    for (const HostSeg& g : p->segs) {
        if (g.rows == 1 || g.dst_stride == g.row_len) {  // rows are adjacent in the arena: one range
            v.push_back(dr_range{g.dst_off, g.rows * g.row_len * es});
        } else {
            for (uint64_t i = 0; i < g.rows; ++i) v.push_back(dr_range{g.dst_off + i * g.dst_stride * es, g.row_len * es});
        }
    }
    std::sort(v.begin(), v.end(), [](const dr_range& a, const dr_range& b) { return a.off < b.off; });
    std::vector<dr_range> out;
    for (const dr_range& r : v) {
        if (r.bytes == 0) continue;
        if (!out.empty() && out.back().off + out.back().bytes == r.off) out.back().bytes += r.bytes;
        else out.push_back(r);
    }
    return out;
}

int compile_plan(dr_plan* p)
{
    const dr_model_spec& s = p->spec;
    const uint64_t T = p->tp, t = p->tp_rank, H = s.hidden, hd = s.head_dim;
    const uint64_t nq = s.n_q_heads, nkv = s.n_kv_heads, F = s.ffn, V = s.vocab, E = s.n_experts, Fm = s.moe_ffn;
    const uint32_t es = p->elem_size;
    Builder flat(s, p->src.align_elems);
    Emit out{p};
    char nm[64];

    // layout variants
    const dr_dst_layout& L = p->dst;
    const uint64_t Vp = L.vocab_pad ? (V + L.vocab_pad - 1) / L.vocab_pad * L.vocab_pad : V;
    const uint64_t v_lo = t * (Vp / T), v_hi = (t + 1) * (Vp / T);
    const uint64_t v_real = v_lo >= V ? 0 : std::min(v_hi, V) - v_lo;  // rows of this rank that exist
    const bool kv_rep = L.kv_replicate && T > nkv;
    const uint64_t kv_rows = kv_rep ? hd : (nkv / T) * hd;
    const uint64_t kv_row0 = kv_rep ? (t / (T / nkv)) * hd : t * (nkv / T) * hd;
    const uint64_t EP = L.moe_ep ? L.moe_ep : 1, E_loc = E / EP, e_first = L.moe_ep_rank * E_loc;
    const uint64_t MT = L.moe_tp > 1 ? T : 1, mt = L.moe_tp > 1 ? t : 0;

    Param embed = flat.take(V, H);
    out.begin("embed", H);
    out.block(embed, v_lo, 0, v_real);
    out.pad_rows(Vp / T);
    const int64_t embed_index = 0;

    for (uint32_t l = 0; l < s.n_layers; ++l) {
        auto name = [&](const char* leaf) {
            snprintf(nm, sizeof nm, "layers.%u.%s", l, leaf);
            return std::string(nm);
        };
        out.group = l + 1;
        Param in_norm = flat.take(1, H);
        Param q = flat.take(nq * hd, H), k = flat.take(nkv * hd, H), v = flat.take(nkv * hd, H);
        Param q_norm{}, k_norm{};
        if (s.qk_norm) {
            q_norm = flat.take(1, hd);
            k_norm = flat.take(1, hd);
        }
        Param o = flat.take(H, nq * hd);
        Param post_norm = flat.take(1, H);

        out.begin(name("in_norm"), H);
        out.block(in_norm, 0, 0, 1);
        out.begin(name("qkv"), H);
        out.block(q, t * (nq / T) * hd, 0, (nq / T) * hd);
        out.block(k, kv_row0, 0, kv_rows);
        out.block(v, kv_row0, 0, kv_rows);
        if (s.qk_norm) {
            out.begin(name("q_norm"), hd);
            out.block(q_norm, 0, 0, 1);
            out.begin(name("k_norm"), hd);
            out.block(k_norm, 0, 0, 1);
        }
        out.begin(name("o"), nq * hd / T);
        out.block(o, 0, t * (nq * hd / T), H);
        out.begin(name("post_norm"), H);
        out.block(post_norm, 0, 0, 1);
        if (E == 0) {
            Param gate = flat.take(F, H), up = flat.take(F, H), down = flat.take(H, F);
            out.begin(name("gate_up"), H);
            out.block(gate, t * (F / T), 0, F / T);
            out.block(up, t * (F / T), 0, F / T);
            out.begin(name("down"), F / T);
            out.block(down, 0, t * (F / T), H);
        } else {
            Param router = flat.take(E, H);
            std::vector<Param> ge(E), ue(E), de(E);
            for (uint64_t e = 0; e < E; ++e) {  // experts interleaved: gate_e, up_e, down_e
                ge[e] = flat.take(Fm, H);
                ue[e] = flat.take(Fm, H);
                de[e] = flat.take(H, Fm);
            }
            out.begin(name("router"), H);
            out.block(router, 0, 0, E);
            const uint64_t Fs = Fm / MT;  // expert width kept by this rank
            out.begin(name("w13"), H);
            for (uint64_t e = e_first; e < e_first + E_loc; ++e) {
                out.block(ge[e], mt * Fs, 0, Fs);
                out.block(ue[e], mt * Fs, 0, Fs);
            }
            out.begin(name("w2"), Fs);
            for (uint64_t e = e_first; e < e_first + E_loc; ++e) out.block(de[e], 0, mt * Fs, H);
        }
    }
    out.group = s.n_layers + 1;
    Param final_norm = flat.take(1, H);
    out.begin("final_norm", H);
    out.block(final_norm, 0, 0, 1);
    if (s.tied_embeddings) {
        Tensor a;
        a.name = "lm_head";
        a.alias_of = embed_index;
        a.arena_off = p->tensors[embed_index].arena_off;
        a.rows = p->tensors[embed_index].rows;
        a.cols = H;
        a.group = out.group;
        p->tensors.push_back(a);
    } else {
        Param lm_head = flat.take(V, H);
        out.begin("lm_head", H);
        out.block(lm_head, v_lo, 0, v_real);
        out.pad_rows(Vp / T);
    }

    out.finish();
    const uint64_t N = flat.next, W = p->src.world, S = (N + W - 1) / W;
    merge_adjacent(p->segs, es);
    if (!p->src.gathered) clip_to_shard(p->segs, (uint64_t)p->src.rank * S, (uint64_t)(p->src.rank + 1) * S, es);
    classify(p->segs, es);

    Tables tb;
    int trc = build_tables(p->segs, &tb);
    if (trc) return trc;
    p->dev_segs.swap(tb.segs);
    p->hints.swap(tb.hints);
    p->hint_shift = tb.hint_shift;
    const uint64_t tiles = tb.n_tiles, moved = tb.elems;
    // tile range, tensors and element count of every group (segments are in group order)
    p->groups.assign(s.n_layers + 2, Group{});
    for (size_t i = 0; i < p->tensors.size(); ++i) {
        Group& G = p->groups[p->tensors[i].group];
        if (G.n_tensors == 0) G.first_tensor = (uint32_t)i;
        G.n_tensors++;
    }
    {
        uint64_t at = 0;
        for (Group& G : p->groups) G.tile_lo = G.tile_hi = 0;
        std::vector<bool> seen(p->groups.size(), false);
        for (size_t i = 0; i < p->segs.size(); ++i) {
            Group& G = p->groups[p->segs[i].group];
            const uint64_t t0 = p->dev_segs[i].tile0;
            const uint64_t t1 = i + 1 < p->segs.size() ? p->dev_segs[i + 1].tile0 : tiles;
            if (!seen[p->segs[i].group]) {
                G.tile_lo = t0;
                seen[p->segs[i].group] = true;
            }
            G.tile_hi = t1;
            G.elems += p->segs[i].rows * p->segs[i].row_len;
            at = t1;
        }
        (void)at;
    }

    // fp8: block prefix per quantised tensor and a block -> tensor hint table
    uint64_t qblocks = 0, qelems = 0;
    {
        size_t qi = 0;  // quantised tensors appear in p->qtensors in tensor order
        for (const Tensor& t : p->tensors) {
            if (!t.quant || t.alias_of >= 0) continue;
            QTensor& q = p->qtensors[qi++];
            Group& G = p->groups[t.group];
            q.block0 = qblocks;
            if (G.qblock_hi == G.qblock_lo) G.qblock_lo = qblocks;
            qblocks += (uint64_t)((q.rows + 127) / 128) * q.nbc;
            G.qblock_hi = qblocks;
            G.qelems += (uint64_t)q.rows * q.cols;
            qelems += (uint64_t)q.rows * q.cols;
        }
    }
    if (p->fp8) {
        p->qhint_shift = 0;
        while (((qblocks + (1ull << p->qhint_shift) - 1) >> p->qhint_shift) > kMaxHints) ++p->qhint_shift;
        const uint64_t n_hints = (qblocks + (1ull << p->qhint_shift) - 1) >> p->qhint_shift;
        p->qhints.assign(n_hints ? n_hints : 1, 0);
        uint32_t qi = 0;
        for (uint64_t h = 0; h < n_hints; ++h) {
            const uint64_t b = h << p->qhint_shift;
            while (qi + 1 < p->qtensors.size() && p->qtensors[qi + 1].block0 <= b) ++qi;
            p->qhints[h] = qi;
        }
    }

    {   // forward launches go through the bulk-copy kernel when under 2 % of the plan's elements sit in strided
        // segments and the plan has 2^28 elements or more (below that the register kernel's shorter tile latency wins)
        uint64_t strided = 0;
        for (const HostSeg& g : p->segs)
            if (g.rows > 1) strided += g.rows * g.row_len;
        p->bulk_forward = strided * 50 <= moved && moved >= (1ull << 28);
        // DR_FORWARD_KERNEL = bulk | register overrides the choice (for measurements; both give the same bytes)
        if (const char* e = std::getenv("DR_FORWARD_KERNEL")) {
            if (!std::strcmp(e, "bulk")) p->bulk_forward = true;
            else if (!std::strcmp(e, "register")) p->bulk_forward = false;
        }
    }
    dr_plan_info& I = p->info;
    I.flat_elems = N;
    I.shard_elems = S;
    I.src_bytes = 4 * (p->src.gathered ? W * S : S);
    I.dst_bytes = out.arena;
    I.n_tensors = p->tensors.size();
    I.n_segments = p->segs.size();
    I.n_tiles = tiles;
    I.elems_moved = moved + qelems;
    I.bytes_moved_fwd = moved * (4 + es) + qelems * 5 + qblocks * 4;
    I.bytes_moved_inv = moved * (4 + es) + qelems * 5 + qblocks * 4;
    I.n_groups = p->groups.size();
    I.quant_elems = qelems;
    I.quant_blocks = qblocks;
    I.bulk_forward = p->bulk_forward ? 1 : 0;

    // Every access the kernels will make is checked here, so a launch cannot leave its buffers.
    const uint64_t src_elems = I.src_bytes / 4;
    for (const HostSeg& g : p->segs) {
        uint64_t src_end = g.src_off + (g.rows - 1) * g.src_stride + g.row_len;
        uint64_t dst_end = g.dst_off + ((g.rows - 1) * g.dst_stride + g.row_len) * es;
        if (src_end > src_elems || dst_end > I.dst_bytes) {
            set_error("planner produced a segment outside its buffers");
            return DR_ERR_INVALID;
        }
    }
    return DR_OK;
}

}  // namespace dr
