/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, single-threaded CPU statement of the per-GPU state transform
 * that a Training<->Rollout role switch needs (dropping the old role's
 * parameters and taking in the new role's weights and optimizer state, paper
 * Sec. 1 challenge 2; bringing in the state the new topology asks for,
 * Sec. 3.3) and of the bounded
 * chunked host staging of Sec. 3.3.  The paper gives no formula for the
 * layout map, so the definitions D1-D6 below are the ones this repository
 * adopts; every one is written out element by element, with no segment
 * table, no blocking, no vector tricks and no code shared with the CUDA
 * library.  Only tests, the smoke check and the bench's CPU-baseline leg
 * may call it.
 *
 * Parity pins: every function here is pinned by the CPU test-suite
 * (closed-form counts, torch-CPU narrow/cat reconstruction, exhaustive cast
 * check against an exact-arithmetic definition, hand tie table, inverse and
 * shard-union invariants, byte-level staging invariants).  Nothing is
 * "parity unpinned".
 *
 * Notation: L layers, hidden H, nq query heads, nkv kv heads, head dim hd,
 * FFN width F, vocab V, E experts (0 = dense) of width Fm; FSDP-style flat
 * source with world W, rank r, per-parameter alignment A; rollout layout at
 * tensor-parallel degree T, rank t.  All matrices are [out, in] row-major.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    uint32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    uint32_t n_experts, moe_ffn, tied, qk_norm;
} orc_spec;

/* One tensor of the training-side flat buffer (D1, D2). */
typedef struct {
    char name[64];
    uint64_t rows, cols;
    uint64_t flat_off; /* element offset inside the flat buffer */
} orc_src;

/* A row-block of a rollout tensor: rows x cols elements taken from source
 * tensor `src` starting at (src_row0, src_col0), placed at rollout rows
 * [dst_row0, dst_row0 + rows). */
typedef struct {
    int64_t src;
    uint64_t src_row0, src_col0, rows, dst_row0;
} orc_part;

/* One tensor of the rollout arena (D3). */
typedef struct {
    char name[64];
    uint64_t rows, cols;
    uint64_t arena_off; /* byte offset inside the arena */
    int64_t alias_of;   /* >= 0: shares storage with that rollout tensor, owns no bytes */
    uint64_t n_parts;
    orc_part *parts;
} orc_dst;

/* Rollout layout variants beyond the base definition (all off / 1 by default):
 *   kv_replicate  tp may exceed the kv heads (tp % n_kv_heads == 0): rank t holds the one kv head
 *                 t / (tp / n_kv_heads), i.e. each kv head is replicated on tp / n_kv_heads ranks
 *   vocab_pad     embed / lm_head rows are padded up to a multiple of vocab_pad before slicing; the
 *                 padding rows exist in the arena but have no source element (never written)
 *   moe_tp        1: experts unsliced; == tp: expert FFN width sliced like the dense MLP
 *   moe_ep, moe_ep_rank   expert parallelism: the rank keeps the contiguous block of
 *                 n_experts / moe_ep experts number moe_ep_rank */
typedef struct {
    uint32_t kv_replicate, vocab_pad, moe_tp, moe_ep, moe_ep_rank;
} orc_opts;

typedef struct {
    orc_spec spec;
    orc_opts opt;
    uint64_t align, world, tp, tp_rank, elem_size, arena_align;
    uint64_t n_src, n_dst;
    orc_src *src;
    orc_dst *dst;
    uint64_t *layer_first; /* index of the first source tensor of each layer */
    uint64_t flat_elems;   /* N  */
    uint64_t shard_elems;  /* S = ceil(N / W) */
    uint64_t arena_bytes;
} orc_model;

static uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

/* ---- D5: the cast --------------------------------------------------------
 * fp32 -> bf16, round to nearest, ties to even, on the bit pattern u.
 * NaN (exponent all ones, mantissa non-zero) -> canonical 0x7FFF.
 * Otherwise add 0x7FFF plus the lowest kept bit and drop the low half; this
 * rounds subnormals (no flush), carries into the exponent, and lets values
 * above the largest finite bf16 round to infinity.  The sign bit rides along
 * because the addition cannot carry out of bit 30 for a non-NaN input.
 */
uint16_t orc_cast_bf16(uint32_t u)
{
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FFF;
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

/* The same cast over an array: the scalar function, one element at a time. */
void orc_cast_bf16_many(const uint32_t *u, uint16_t *out, uint64_t n)
{
    uint64_t i;
    for (i = 0; i < n; ++i) out[i] = orc_cast_bf16(u[i]);
}

/* bf16 -> fp32 is exact: the 16 bits become the high half. */
uint32_t orc_widen_bf16(uint16_t b) { return (uint32_t)b << 16; }

/* ---- D1 + D2: canonical tensor order and flat offsets -------------------- */
static void push_src(orc_model *m, uint64_t *cap, const char *name, uint64_t rows, uint64_t cols)
{
    orc_src *s;
    if (m->n_src == *cap) {
        *cap = *cap ? *cap * 2 : 64;
        m->src = (orc_src *)realloc(m->src, *cap * sizeof(orc_src));
    }
    s = &m->src[m->n_src];
    memset(s, 0, sizeof *s);
    snprintf(s->name, sizeof s->name, "%s", name);
    s->rows = rows;
    s->cols = cols;
    if (m->n_src == 0) {
        s->flat_off = 0;
    } else {
        const orc_src *p = &m->src[m->n_src - 1];
        s->flat_off = align_up(p->flat_off + p->rows * p->cols, m->align);
    }
    m->n_src++;
}

static void enumerate_src(orc_model *m)
{
    const orc_spec *c = &m->spec;
    uint64_t cap = 0, H = c->hidden, hd = c->head_dim;
    char nm[64];
    uint32_t l, e;
    m->layer_first = (uint64_t *)calloc(c->n_layers + 1, sizeof(uint64_t));
    push_src(m, &cap, "embed", c->vocab, H);
    for (l = 0; l < c->n_layers; ++l) {
        m->layer_first[l] = m->n_src;
#define P(suffix, r, cc) (snprintf(nm, sizeof nm, "layers.%u." suffix, l), push_src(m, &cap, nm, (r), (cc)))
        P("in_norm", 1, H);
        P("q", (uint64_t)c->n_q_heads * hd, H);
        P("k", (uint64_t)c->n_kv_heads * hd, H);
        P("v", (uint64_t)c->n_kv_heads * hd, H);
        if (c->qk_norm) {
            P("q_norm", 1, hd);
            P("k_norm", 1, hd);
        }
        P("o", H, (uint64_t)c->n_q_heads * hd);
        P("post_norm", 1, H);
        if (c->n_experts == 0) {
            P("gate", c->ffn, H);
            P("up", c->ffn, H);
            P("down", H, c->ffn);
        } else {
            P("router", c->n_experts, H);
            for (e = 0; e < c->n_experts; ++e) {
#define PE(suffix, r, cc) \
    (snprintf(nm, sizeof nm, "layers.%u.experts.%u." suffix, l, e), push_src(m, &cap, nm, (r), (cc)))
                PE("gate", c->moe_ffn, H);
                PE("up", c->moe_ffn, H);
                PE("down", H, c->moe_ffn);
#undef PE
            }
        }
#undef P
    }
    m->layer_first[c->n_layers] = m->n_src;
    push_src(m, &cap, "final_norm", 1, H);
    if (!c->tied) push_src(m, &cap, "lm_head", c->vocab, H);
    {
        const orc_src *p = &m->src[m->n_src - 1];
        m->flat_elems = p->flat_off + p->rows * p->cols;
    }
    m->shard_elems = (m->flat_elems + m->world - 1) / m->world;
}

/* Index of source tensor `name`; layer >= 0 restricts the search to that layer's tensors. */
static int64_t find_src(const orc_model *m, int64_t layer, const char *name)
{
    uint64_t lo = 0, hi = m->n_src, i;
    if (layer >= 0) {
        lo = m->layer_first[layer];
        hi = m->layer_first[layer + 1];
    }
    for (i = lo; i < hi; ++i)
        if (strcmp(m->src[i].name, name) == 0) return (int64_t)i;
    fprintf(stderr, "dr_oracle: source tensor %s not found\n", name);
    abort();
}

/* ---- D3: rollout layout at (T, t) ---------------------------------------- */
static orc_dst *push_dst(orc_model *m, uint64_t *cap, const char *name, uint64_t cols)
{
    orc_dst *d;
    if (m->n_dst == *cap) {
        *cap = *cap ? *cap * 2 : 64;
        m->dst = (orc_dst *)realloc(m->dst, *cap * sizeof(orc_dst));
    }
    d = &m->dst[m->n_dst++];
    memset(d, 0, sizeof *d);
    snprintf(d->name, sizeof d->name, "%s", name);
    d->cols = cols;
    d->alias_of = -1;
    return d;
}

/* Append to rollout tensor d the block rows x d->cols of source tensor s at (row0, col0). */
static void add_part(orc_dst *d, int64_t s, uint64_t row0, uint64_t col0, uint64_t rows)
{
    orc_part *p;
    d->parts = (orc_part *)realloc(d->parts, (d->n_parts + 1) * sizeof(orc_part));
    p = &d->parts[d->n_parts++];
    p->src = s;
    p->src_row0 = row0;
    p->src_col0 = col0;
    p->rows = rows;
    p->dst_row0 = d->rows;
    d->rows += rows;
}

static void build_dst(orc_model *m)
{
    const orc_spec *c = &m->spec;
    const uint64_t T = m->tp, t = m->tp_rank, H = c->hidden, hd = c->head_dim;
    const uint64_t nq = c->n_q_heads, nkv = c->n_kv_heads, F = c->ffn, V = c->vocab;
    uint64_t cap = 0, i, off = 0;
    char nm[64], sn[64];
    uint32_t l, e;
    orc_dst *d;
    int64_t embed_index;

    /* vocabulary rows of this rank: [t Vp/T, (t+1) Vp/T) of the matrix padded to Vp rows; only rows < V exist */
    const uint64_t Vp = m->opt.vocab_pad ? align_up(V, m->opt.vocab_pad) : V;
    const uint64_t v_lo = t * (Vp / T), v_hi = (t + 1) * (Vp / T);
    const uint64_t v_real = v_lo >= V ? 0 : (v_hi <= V ? v_hi - v_lo : V - v_lo);
    /* kv heads of this rank: nkv / T of them, or with replication the single head t / (T / nkv) */
    const int kv_rep = m->opt.kv_replicate && T > nkv;
    const uint64_t kv_rows = kv_rep ? hd : (nkv / T) * hd;
    const uint64_t kv_row0 = kv_rep ? (t / (T / nkv)) * hd : t * (nkv / T) * hd;
    /* experts of this rank and their width */
    const uint64_t EP = m->opt.moe_ep ? m->opt.moe_ep : 1, E_loc = c->n_experts / EP, e0 = m->opt.moe_ep_rank * E_loc;
    const uint64_t MT = m->opt.moe_tp > 1 ? T : 1, mt = m->opt.moe_tp > 1 ? t : 0;

    /* embed_t = embed[t Vp/T : (t+1) Vp/T, :] */
    d = push_dst(m, &cap, "embed", H);
    if (v_real) add_part(d, find_src(m, -1, "embed"), v_lo, 0, v_real);
    d->rows = Vp / T;
    embed_index = (int64_t)m->n_dst - 1;

    for (l = 0; l < c->n_layers; ++l) {
#define D(suffix, cc) (snprintf(nm, sizeof nm, "layers.%u." suffix, l), push_dst(m, &cap, nm, (cc)))
#define S(suffix) (snprintf(sn, sizeof sn, "layers.%u." suffix, l), find_src(m, l, sn))
        d = D("in_norm", H);
        add_part(d, S("in_norm"), 0, 0, 1);
        /* qkv = [ q rows of rank t ; k rows of rank t ; v rows of rank t ] */
        d = D("qkv", H);
        add_part(d, S("q"), t * (nq / T) * hd, 0, (nq / T) * hd);
        add_part(d, S("k"), kv_row0, 0, kv_rows);
        add_part(d, S("v"), kv_row0, 0, kv_rows);
        if (c->qk_norm) {
            d = D("q_norm", hd);
            add_part(d, S("q_norm"), 0, 0, 1);
            d = D("k_norm", hd);
            add_part(d, S("k_norm"), 0, 0, 1);
        }
        /* o_t = o[:, t nq hd / T : (t+1) nq hd / T] */
        d = D("o", nq * hd / T);
        add_part(d, S("o"), 0, t * (nq * hd / T), H);
        d = D("post_norm", H);
        add_part(d, S("post_norm"), 0, 0, 1);
        if (c->n_experts == 0) {
            /* gate_up = [ gate rows of rank t ; up rows of rank t ] */
            d = D("gate_up", H);
            add_part(d, S("gate"), t * (F / T), 0, F / T);
            add_part(d, S("up"), t * (F / T), 0, F / T);
            /* down_t = down[:, t F/T : (t+1) F/T] */
            d = D("down", F / T);
            add_part(d, S("down"), 0, t * (F / T), H);
        } else {
            const uint64_t Fm = c->moe_ffn, Fs = Fm / MT; /* width kept per expert */
            d = D("router", H);
            add_part(d, S("router"), 0, 0, c->n_experts);
            /* w13[j] = [gate_e rows of this rank ; up_e rows of this rank], e = e0 + j, expert-major */
            d = D("w13", H);
            for (e = (uint32_t)e0; e < e0 + E_loc; ++e) {
                snprintf(sn, sizeof sn, "layers.%u.experts.%u.gate", l, e);
                add_part(d, find_src(m, l, sn), mt * Fs, 0, Fs);
                snprintf(sn, sizeof sn, "layers.%u.experts.%u.up", l, e);
                add_part(d, find_src(m, l, sn), mt * Fs, 0, Fs);
            }
            /* w2[j] = down_e columns of this rank */
            d = D("w2", Fs);
            for (e = (uint32_t)e0; e < e0 + E_loc; ++e) {
                snprintf(sn, sizeof sn, "layers.%u.experts.%u.down", l, e);
                add_part(d, find_src(m, l, sn), 0, mt * Fs, H);
            }
        }
#undef D
#undef S
    }
    d = push_dst(m, &cap, "final_norm", H);
    add_part(d, find_src(m, -1, "final_norm"), 0, 0, 1);
    d = push_dst(m, &cap, "lm_head", H);
    if (c->tied) {
        d->alias_of = embed_index;
        d->rows = m->dst[embed_index].rows;
    } else {
        if (v_real) add_part(d, find_src(m, -1, "lm_head"), v_lo, 0, v_real);
        d->rows = Vp / T;
    }
    /* arena offsets: tensors in order, each start aligned up to arena_align bytes */
    for (i = 0; i < m->n_dst; ++i) {
        d = &m->dst[i];
        if (d->alias_of >= 0) {
            d->arena_off = m->dst[d->alias_of].arena_off;
            continue;
        }
        off = align_up(off, m->arena_align);
        d->arena_off = off;
        off += d->rows * d->cols * m->elem_size;
    }
    m->arena_bytes = off;
}

/* Returns NULL when the shapes do not divide as the chosen options need. */
orc_model *orc_model_create_ex(const orc_spec *spec, uint64_t align, uint64_t world, uint64_t tp, uint64_t tp_rank,
                               uint64_t elem_size, uint64_t arena_align, const orc_opts *opt)
{
    orc_model *m;
    orc_opts o = {0, 0, 1, 1, 0};
    uint64_t Vp;
    if (opt) o = *opt;
    if (!spec || align == 0 || world == 0 || tp == 0 || tp_rank >= tp || arena_align == 0) return NULL;
    if (elem_size != 2 && elem_size != 4) return NULL;
    if (spec->n_q_heads % tp) return NULL;
    if (spec->n_kv_heads % tp && !(o.kv_replicate && tp > spec->n_kv_heads && tp % spec->n_kv_heads == 0)) return NULL;
    Vp = o.vocab_pad ? align_up(spec->vocab, o.vocab_pad) : spec->vocab;
    if (Vp % tp) return NULL;
    if (spec->n_experts == 0 && spec->ffn % tp) return NULL;
    if (o.moe_tp != 1 && o.moe_tp != tp) return NULL;
    if (spec->n_experts && o.moe_tp > 1 && spec->moe_ffn % tp) return NULL;
    if (o.moe_ep == 0) o.moe_ep = 1;
    if (spec->n_experts % o.moe_ep || o.moe_ep_rank >= o.moe_ep) return NULL;
    m = (orc_model *)calloc(1, sizeof *m);
    m->spec = *spec;
    m->opt = o;
    m->align = align;
    m->world = world;
    m->tp = tp;
    m->tp_rank = tp_rank;
    m->elem_size = elem_size;
    m->arena_align = arena_align;
    enumerate_src(m);
    build_dst(m);
    return m;
}

orc_model *orc_model_create(const orc_spec *spec, uint64_t align, uint64_t world, uint64_t tp, uint64_t tp_rank,
                            uint64_t elem_size, uint64_t arena_align)
{
    return orc_model_create_ex(spec, align, world, tp, tp_rank, elem_size, arena_align, NULL);
}

void orc_model_destroy(orc_model *m)
{
    uint64_t i;
    if (!m) return;
    for (i = 0; i < m->n_dst; ++i) free(m->dst[i].parts);
    free(m->dst);
    free(m->src);
    free(m->layer_first);
    free(m);
}

uint64_t orc_n_src(const orc_model *m) { return m->n_src; }
uint64_t orc_n_dst(const orc_model *m) { return m->n_dst; }
uint64_t orc_flat_elems(const orc_model *m) { return m->flat_elems; }
uint64_t orc_shard_elems(const orc_model *m) { return m->shard_elems; }
uint64_t orc_arena_bytes(const orc_model *m) { return m->arena_bytes; }

int orc_src_info(const orc_model *m, uint64_t i, char *name64, uint64_t *rows, uint64_t *cols, uint64_t *flat_off)
{
    if (i >= m->n_src) return -1;
    memcpy(name64, m->src[i].name, 64);
    *rows = m->src[i].rows;
    *cols = m->src[i].cols;
    *flat_off = m->src[i].flat_off;
    return 0;
}

int orc_dst_info(const orc_model *m, uint64_t i, char *name64, uint64_t *rows, uint64_t *cols, uint64_t *arena_off,
                 int64_t *alias_of)
{
    if (i >= m->n_dst) return -1;
    memcpy(name64, m->dst[i].name, 64);
    *rows = m->dst[i].rows;
    *cols = m->dst[i].cols;
    *arena_off = m->dst[i].arena_off;
    *alias_of = m->dst[i].alias_of;
    return 0;
}

/* ---- D4: element map ------------------------------------------------------
 * Flat index of the source element that rollout element (tensor i, row, col)
 * is a copy of; -1 for an alias tensor or an out-of-range coordinate.
 */
int64_t orc_map(const orc_model *m, uint64_t i, uint64_t row, uint64_t col)
{
    const orc_dst *d;
    uint64_t p;
    if (i >= m->n_dst) return -1;
    d = &m->dst[i];
    if (d->alias_of >= 0 || row >= d->rows || col >= d->cols) return -1;
    for (p = 0; p < d->n_parts; ++p) {
        const orc_part *q = &d->parts[p];
        if (row >= q->dst_row0 && row < q->dst_row0 + q->rows) {
            const orc_src *s = &m->src[q->src];
            uint64_t srow = q->src_row0 + (row - q->dst_row0);
            uint64_t scol = q->src_col0 + col;
            return (int64_t)(s->flat_off + srow * s->cols + scol);
        }
    }
    return -1;
}

/* Flat indices of rows [row0, row0 + nrows) of rollout tensor i, row-major into out. */
int orc_map_rows(const orc_model *m, uint64_t i, uint64_t row0, uint64_t nrows, int64_t *out)
{
    uint64_t r, c, cols;
    if (i >= m->n_dst) return -1;
    cols = m->dst[i].cols;
    for (r = 0; r < nrows; ++r)
        for (c = 0; c < cols; ++c) out[r * cols + c] = orc_map(m, i, row0 + r, c);
    return 0;
}

/* Is flat index f visible to this call?  gathered: the whole buffer; else only shard `rank`. */
static int visible(const orc_model *m, uint64_t f, int gathered, uint64_t rank, uint64_t *local)
{
    if (gathered) {
        *local = f;
        return 1;
    }
    if (f >= rank * m->shard_elems && f < (rank + 1) * m->shard_elems) {
        *local = f - rank * m->shard_elems;
        return 1;
    }
    return 0;
}

/* ---- forward: Training -> Rollout (D4 with D5) ----------------------------
 * src: fp32 words, the whole flat buffer (gathered) or shard `rank` alone.
 * arena: rollout buffers; only mapped, visible elements are written.
 * Restricting to one rollout tensor (only >= 0) is the same loop over a
 * subset, used to stream big models tensor by tensor.
 */
int orc_forward(const orc_model *m, const uint32_t *src, int gathered, uint64_t rank, uint8_t *arena, int64_t only)
{
    uint64_t i, p, r, c;
    for (i = 0; i < m->n_dst; ++i) {
        const orc_dst *d = &m->dst[i];
        if (only >= 0 && (uint64_t)only != i) continue;
        if (d->alias_of >= 0) continue;
        for (p = 0; p < d->n_parts; ++p) {
            const orc_part *q = &d->parts[p];
            const orc_src *s = &m->src[q->src];
            for (r = 0; r < q->rows; ++r) {
                for (c = 0; c < d->cols; ++c) {
                    uint64_t f = s->flat_off + (q->src_row0 + r) * s->cols + (q->src_col0 + c);
                    uint64_t j = (q->dst_row0 + r) * d->cols + c;
                    uint64_t local;
                    if (!visible(m, f, gathered, rank, &local)) continue;
                    if (m->elem_size == 2) {
                        uint16_t b = orc_cast_bf16(src[local]);
                        memcpy(arena + d->arena_off + j * 2, &b, 2);
                    } else {
                        memcpy(arena + d->arena_off + j * 4, &src[local], 4);
                    }
                }
            }
        }
    }
    return 0;
}

/* ---- inverse: Rollout -> Training ----------------------------------------
 * Every mapped, visible flat position receives the widened rollout element;
 * all other words of `flat` (padding, other TP ranks' slices, other shards)
 * are left as they were.
 */
int orc_inverse(const orc_model *m, const uint8_t *arena, int gathered, uint64_t rank, uint32_t *flat)
{
    uint64_t i, p, r, c;
    for (i = 0; i < m->n_dst; ++i) {
        const orc_dst *d = &m->dst[i];
        if (d->alias_of >= 0) continue;
        for (p = 0; p < d->n_parts; ++p) {
            const orc_part *q = &d->parts[p];
            const orc_src *s = &m->src[q->src];
            for (r = 0; r < q->rows; ++r) {
                for (c = 0; c < d->cols; ++c) {
                    uint64_t f = s->flat_off + (q->src_row0 + r) * s->cols + (q->src_col0 + c);
                    uint64_t j = (q->dst_row0 + r) * d->cols + c;
                    uint64_t local;
                    if (!visible(m, f, gathered, rank, &local)) continue;
                    if (m->elem_size == 2) {
                        uint16_t b;
                        memcpy(&b, arena + d->arena_off + j * 2, 2);
                        flat[local] = orc_widen_bf16(b);
                    } else {
                        memcpy(&flat[local], arena + d->arena_off + j * 4, 4);
                    }
                }
            }
        }
    }
    return 0;
}

/* ---- D6: bounded chunked staging (Sec. 3.3) -------------------------------
 * The state buffers form one logical byte stream X = buf_0 | buf_1 | ...;
 * chunk k is X[k C, min((k+1) C, B)).  Stage-out moves the stream through a
 * ring of `slots` host buffers of C bytes (slots * C <= budget) into the
 * sink, one byte at a time here.  Returns the number of chunks, or -1 when
 * the budget cannot hold two slots.  `first_chunk` resumes a transfer.
 */
static uint8_t stream_byte(const uint8_t *const *bufs, const uint64_t *bytes, uint64_t n_bufs, uint64_t pos)
{
    uint64_t b;
    for (b = 0; b < n_bufs; ++b) {
        if (pos < bytes[b]) return bufs[b][pos];
        pos -= bytes[b];
    }
    abort();
}

static void stream_put(uint8_t *const *bufs, const uint64_t *bytes, uint64_t n_bufs, uint64_t pos, uint8_t v)
{
    uint64_t b;
    for (b = 0; b < n_bufs; ++b) {
        if (pos < bytes[b]) {
            bufs[b][pos] = v;
            return;
        }
        pos -= bytes[b];
    }
    abort();
}

int64_t orc_stage_out(const uint8_t *const *bufs, const uint64_t *bytes, uint64_t n_bufs, uint64_t budget,
                      uint64_t chunk, uint64_t first_chunk, uint8_t *sink, uint64_t *chunk_sizes)
{
    uint64_t total = 0, b, k, n_chunks, slots, i;
    uint8_t *ring;
    if (chunk == 0) chunk = budget / 2 / 4096 * 4096;
    if (chunk == 0) return -1;
    slots = budget / chunk;
    if (slots < 2) return -1;
    for (b = 0; b < n_bufs; ++b) total += bytes[b];
    n_chunks = (total + chunk - 1) / chunk;
    ring = (uint8_t *)malloc(slots * chunk);
    for (k = first_chunk; k < n_chunks; ++k) {
        uint64_t lo = k * chunk, hi = lo + chunk < total ? lo + chunk : total;
        uint8_t *slot = ring + (k % slots) * chunk;
        for (i = lo; i < hi; ++i) slot[i - lo] = stream_byte(bufs, bytes, n_bufs, i); /* device -> ring slot */
        for (i = lo; i < hi; ++i) sink[i] = slot[i - lo];                             /* ring slot -> sink   */
        if (chunk_sizes) chunk_sizes[k] = hi - lo;
    }
    free(ring);
    return (int64_t)n_chunks;
}

/* Stage-in (Sec. 3.3: weights at the transition, optimizer state deferred): buffers are restored one
 * after the other in `order` (weights first), and each buffer on its own is cut into pieces of at most C
 * bytes, so a piece never holds bytes of two buffers and buffer order[0] is whole before the first byte
 * of order[1] moves.  Piece number i goes through ring slot i mod slots.  The walk is recorded:
 * piece_list receives (buffer, position inside the buffer, bytes) for every piece in the order taken,
 * completed[o] the buffer that became whole o-th.  Returns the number of pieces. */
int64_t orc_stage_in(uint8_t *const *bufs, const uint64_t *bytes, uint64_t n_bufs, const uint32_t *order,
                     uint64_t budget, uint64_t chunk, const uint8_t *source, uint32_t *completed,
                     uint64_t *piece_list)
{
    uint64_t b, o, slots, pieces = 0, i, n_completed = 0;
    uint8_t *ring;
    if (chunk == 0) chunk = budget / 2 / 4096 * 4096;
    if (chunk == 0) return -1;
    slots = budget / chunk;
    if (slots < 2) return -1;
    ring = (uint8_t *)malloc(slots * chunk);
    for (o = 0; o < n_bufs; ++o) {
        uint64_t base = 0, pos;
        b = order ? order[o] : o;
        for (i = 0; i < b; ++i) base += bytes[i];
        for (pos = 0; pos < bytes[b]; pos += chunk) {
            uint64_t n = bytes[b] - pos < chunk ? bytes[b] - pos : chunk;
            uint8_t *slot = ring + (pieces % slots) * chunk;
            for (i = 0; i < n; ++i) slot[i] = source[base + pos + i];          /* source -> ring slot */
            for (i = 0; i < n; ++i) stream_put(bufs, bytes, n_bufs, base + pos + i, slot[i]); /* -> device */
            if (piece_list) {
                piece_list[3 * pieces] = b;
                piece_list[3 * pieces + 1] = pos;
                piece_list[3 * pieces + 2] = n;
            }
            pieces++;
        }
        if (completed) completed[n_completed] = (uint32_t)b; /* every byte of b has now been put */
        n_completed++;
    }
    free(ring);
    return (int64_t)pieces;
}

/* ---- Re-sharding the training state across a changed world size (Sec. 3.3) -----------------
 * Old training ranks hold shards of a flat buffer of N elements cut for world W_old
 * (S_old = ceil(N / W_old), the last shard padded); the new topology cuts the same flat buffer for
 * W_new.  Staged through a host image of the flat buffer: old rank r writes its real elements to
 * image[r S_old ...], new rank q reads image[q S_new ...]; elements past N are padding and read as
 * zero.  Written here element by element (4-byte words).
 */
void orc_restage_out(const uint32_t *old_shard, uint64_t N, uint64_t W_old, uint64_t r, uint32_t *image)
{
    uint64_t S = (N + W_old - 1) / W_old, i;
    for (i = 0; i < S; ++i) {
        uint64_t f = r * S + i;
        if (f < N) image[f] = old_shard[i];
    }
}

void orc_restage_in(const uint32_t *image, uint64_t N, uint64_t W_new, uint64_t q, uint32_t *new_shard)
{
    uint64_t S = (N + W_new - 1) / W_new, i;
    for (i = 0; i < S; ++i) {
        uint64_t f = q * S + i;
        new_shard[i] = f < N ? image[f] : 0u;
    }
}

/* ---- D7: fp8 (e4m3) rollout weights with one fp32 scale per 128 x 128 block ----------------------
 * A reading for rollout engines that serve block-quantised weights (the paper is silent).  The linear
 * weights (qkv, o, gate_up, down, w13, w2) are quantised; embeddings, lm_head, router and norms stay
 * bf16.  The definition is the plain one of scaled quantisation: the stored code is the e4m3 rounding
 * of x / scale, where scale is the number a consumer multiplies the code by to get x back.  For a
 * quantised rollout tensor X[rows, cols]:
 *   block (bi, bj) = rows [128 bi, 128 bi + 128) x cols [128 bj, 128 bj + 128), clipped to the tensor;
 *   amax  = max |x| over the block, NaNs skipped (infinities count), starting from 0;
 *   scale = amax / 448 in fp32 (one division, round to nearest), then clamped to
 *           [2^-126, FLT_MAX]: the smallest normal fp32 for blocks whose amax / 448 would be zero or
 *           subnormal (the all-zero block among them), so that x / scale and code * scale stay finite
 *           and zeros stay zeros; the largest finite fp32 for a block holding an infinity;
 *   q     = e4m3( x / scale ): one fp32 division (round to nearest), then round to nearest even onto
 *           the e4m3 grid (3 mantissa bits, bias 7, subnormal step 2^-9), magnitudes above 448 saturate
 *           to 448 (code 0x7E), NaN becomes 0x7F.
 * Arena: payload rows*cols bytes at arena_off, then the scales [ceil(rows/128), ceil(cols/128)] fp32,
 * row-major, at the next multiple of arena_align.
 */
uint8_t orc_cast_e4m3(uint32_t u)
{
    uint32_t sign = (u >> 31) << 7, mag = u & 0x7FFFFFFFu;
    float a;
    double q, quantum;
    int e;
    if (mag > 0x7F800000u) return 0x7F;
    memcpy(&a, &mag, 4);
    if (a > 448.0f) return (uint8_t)(sign | 0x7E);
    if (a == 0.0f) return (uint8_t)sign;
    e = (int)floor(log2((double)a));        /* exact for powers of two in double; a is fp32 */
    if (ldexp(1.0, e) > (double)a) e--;     /* guard against log2 rounding up */
    if (ldexp(1.0, e + 1) <= (double)a) e++;
    quantum = e < -6 ? ldexp(1.0, -9) : ldexp(1.0, e - 3);
    q = nearbyint((double)a / quantum);     /* exact quotient; default rounding mode: ties to even */
    {
        double v = q * quantum;
        int ev, m;
        if (v == 0.0) return (uint8_t)sign;
        if (v < ldexp(1.0, -6)) return (uint8_t)(sign | (uint32_t)q); /* subnormal: mantissa 1..7 */
        ev = (int)floor(log2(v));
        if (ldexp(1.0, ev) > v) ev--;
        if (ldexp(1.0, ev + 1) <= v) ev++;
        m = (int)(v / ldexp(1.0, ev - 3)) - 8;
        return (uint8_t)(sign | (uint32_t)((ev + 7) << 3) | (uint32_t)m);
    }
}

/* exact value of an e4m3 code (NaN codes 0x7F / 0xFF decode as NaN) */
float orc_e4m3_value(uint8_t c)
{
    int e = (c >> 3) & 15, m = c & 7;
    double v;
    if ((c & 0x7F) == 0x7F) return NAN;
    v = e == 0 ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (float)((c & 0x80) ? -v : v);
}

static int is_quantised(const char *name)
{
    const char *leaf = strrchr(name, '.');
    leaf = leaf ? leaf + 1 : name;
    return !strcmp(leaf, "qkv") || !strcmp(leaf, "o") || !strcmp(leaf, "gate_up") || !strcmp(leaf, "down") ||
           !strcmp(leaf, "w13") || !strcmp(leaf, "w2");
}

/* Layout of the fp8 arena: for rollout tensor i, *quant tells whether it is quantised, *off where its
 * payload starts, *scale_off where its scales start (quantised only).  Returns the arena size. */
uint64_t orc_fp8_layout(const orc_model *m, uint64_t i, int *quant, uint64_t *off, uint64_t *scale_off)
{
    uint64_t k, pos = 0, my_off = 0, my_scale = 0;
    int my_q = 0;
    for (k = 0; k < m->n_dst; ++k) {
        const orc_dst *d = &m->dst[k];
        uint64_t o = 0, so = 0;
        int qz = is_quantised(d->name);
        if (d->alias_of < 0) {
            pos = align_up(pos, m->arena_align);
            o = pos;
            if (qz) {
                pos += d->rows * d->cols;
                pos = align_up(pos, m->arena_align);
                so = pos;
                pos += ((d->rows + 127) / 128) * ((d->cols + 127) / 128) * 4;
            } else {
                pos += d->rows * d->cols * 2;
            }
        }
        if (k == i) {
            my_q = qz;
            my_off = d->alias_of >= 0 ? 0 : o;
            my_scale = so;
        }
    }
    if (i < m->n_dst && m->dst[i].alias_of >= 0) {
        int q2;
        uint64_t o2, s2;
        orc_fp8_layout(m, (uint64_t)m->dst[i].alias_of, &q2, &o2, &s2);
        my_off = o2;
    }
    if (quant) *quant = my_q;
    if (off) *off = my_off;
    if (scale_off) *scale_off = my_scale;
    return pos;
}

/* Forward into an fp8 arena: the whole flat buffer must be visible (a block cannot be scaled from part
 * of its elements). */
int orc_forward_fp8(const orc_model *m, const uint32_t *src, uint8_t *arena, int64_t only)
{
    uint64_t i, p, r, c;
    for (i = 0; i < m->n_dst; ++i) {
        const orc_dst *d = &m->dst[i];
        int qz;
        uint64_t off, soff;
        if (only >= 0 && (uint64_t)only != i) continue;
        if (d->alias_of >= 0) continue;
        orc_fp8_layout(m, i, &qz, &off, &soff);
        if (!qz) { /* bf16, as in the base definition */
            for (p = 0; p < d->n_parts; ++p) {
                const orc_part *q = &d->parts[p];
                const orc_src *s = &m->src[q->src];
                for (r = 0; r < q->rows; ++r)
                    for (c = 0; c < d->cols; ++c) {
                        uint64_t f = s->flat_off + (q->src_row0 + r) * s->cols + (q->src_col0 + c);
                        uint16_t b = orc_cast_bf16(src[f]);
                        memcpy(arena + off + ((q->dst_row0 + r) * d->cols + c) * 2, &b, 2);
                    }
            }
            continue;
        }
        {
            /* gather the rollout tensor as fp32 words, then quantise block by block */
            uint32_t *x = (uint32_t *)malloc(d->rows * d->cols * 4);
            uint8_t *has = (uint8_t *)calloc(d->rows, 1);
            uint64_t bi, bj, nbr = (d->rows + 127) / 128, nbc = (d->cols + 127) / 128;
            for (p = 0; p < d->n_parts; ++p) {
                const orc_part *q = &d->parts[p];
                const orc_src *s = &m->src[q->src];
                for (r = 0; r < q->rows; ++r) {
                    has[q->dst_row0 + r] = 1;
                    for (c = 0; c < d->cols; ++c)
                        x[(q->dst_row0 + r) * d->cols + c] =
                            src[s->flat_off + (q->src_row0 + r) * s->cols + (q->src_col0 + c)];
                }
            }
            for (bi = 0; bi < nbr; ++bi)
                for (bj = 0; bj < nbc; ++bj) {
                    uint64_t r1 = bi * 128 + 128 < d->rows ? bi * 128 + 128 : d->rows;
                    uint64_t c1 = bj * 128 + 128 < d->cols ? bj * 128 + 128 : d->cols;
                    float amax = 0.0f, scale;
                    for (r = bi * 128; r < r1; ++r)
                        for (c = bj * 128; c < c1; ++c) {
                            uint32_t mag = x[r * d->cols + c] & 0x7FFFFFFFu;
                            float a;
                            if (!has[r] || mag > 0x7F800000u) continue;
                            memcpy(&a, &mag, 4);
                            if (a > amax) amax = a;
                        }
                    scale = amax / 448.0f;
                    if (scale < FLT_MIN) scale = FLT_MIN; /* 2^-126 */
                    if (scale > FLT_MAX) scale = FLT_MAX; /* amax was an infinity */
                    memcpy(arena + soff + (bi * nbc + bj) * 4, &scale, 4);
                    for (r = bi * 128; r < r1; ++r)
                        for (c = bj * 128; c < c1; ++c) {
                            float v, qv;
                            uint32_t qb;
                            if (!has[r]) continue;
                            memcpy(&v, &x[r * d->cols + c], 4);
                            qv = v / scale;
                            memcpy(&qb, &qv, 4);
                            arena[off + r * d->cols + c] = orc_cast_e4m3(qb);
                        }
                }
            free(x);
            free(has);
        }
    }
    return 0;
}

/* Inverse of D7: Rollout -> Training from an fp8 arena.  A bf16 rollout tensor is widened exactly, as in
 * the base definition.  An element of a quantised tensor becomes value(code) * scale of its block: the
 * exact e4m3 value, one fp32 multiplication (round to nearest); a NaN code, or a NaN product (a scale
 * that is itself NaN, or 0 * Inf), becomes the quiet NaN 0x7FC00000.  Positions no rollout element maps
 * to keep their words. */
int orc_inverse_fp8(const orc_model *m, const uint8_t *arena, uint32_t *flat, int64_t only)
{
    uint64_t i, p, r, c;
    for (i = 0; i < m->n_dst; ++i) {
        const orc_dst *d = &m->dst[i];
        int qz;
        uint64_t off, soff, nbc = (d->cols + 127) / 128;
        if (only >= 0 && (uint64_t)only != i) continue; /* the same loop over one rollout tensor */
        if (d->alias_of >= 0) continue;
        orc_fp8_layout(m, i, &qz, &off, &soff);
        for (p = 0; p < d->n_parts; ++p) {
            const orc_part *q = &d->parts[p];
            const orc_src *s = &m->src[q->src];
            for (r = 0; r < q->rows; ++r)
                for (c = 0; c < d->cols; ++c) {
                    uint64_t f = s->flat_off + (q->src_row0 + r) * s->cols + (q->src_col0 + c);
                    uint64_t row = q->dst_row0 + r;
                    if (!qz) {
                        uint16_t b;
                        memcpy(&b, arena + off + (row * d->cols + c) * 2, 2);
                        flat[f] = orc_widen_bf16(b);
                    } else {
                        float scale, y;
                        uint32_t bits;
                        memcpy(&scale, arena + soff + ((row / 128) * nbc + c / 128) * 4, 4);
                        y = orc_e4m3_value(arena[off + row * d->cols + c]) * scale;
                        memcpy(&bits, &y, 4);
                        if ((bits & 0x7FFFFFFFu) > 0x7F800000u) bits = 0x7FC00000u;
                        flat[f] = bits;
                    }
                }
        }
    }
    return 0;
}
