// C ABI entry points: argument validation, plan lifetime, reshard enqueue.
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstring>
#include <new>

#include "dr_internal.h"

namespace dr {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

namespace {

int validate(const dr_model_spec* s, const dr_src_layout* a, const dr_dst_layout* b, uint32_t tp, uint32_t rank)
{
    if (!s || !a || !b) {
        set_error("NULL spec or layout");
        return DR_ERR_INVALID;
    }
    if (s->struct_size != sizeof(dr_model_spec) || s->version != DR_VERSION || a->struct_size != sizeof(dr_src_layout) ||
        b->struct_size != sizeof(dr_dst_layout)) {
        set_error("struct_size / version mismatch");
        return DR_ERR_INVALID;
    }
    if (a->kind != DR_SRC_FSDP_FLAT || a->dtype != DR_F32 || b->kind != DR_DST_ROLLOUT_FUSED ||
        (b->dtype != DR_BF16 && b->dtype != DR_F32 && b->dtype != DR_FP8_E4M3_B128)) {
        set_error("unknown layout kind or dtype");
        return DR_ERR_UNSUPPORTED;
    }
    if (!s->hidden || !s->n_q_heads || !s->n_kv_heads || !s->head_dim || !s->vocab ||
        (s->n_experts == 0 ? !s->ffn : !s->moe_ffn)) {
        set_error("zero model dimension");
        return DR_ERR_INVALID;
    }
    if (!a->world || a->rank >= a->world || !a->align_elems || a->gathered > 1 || !tp || rank >= tp) {
        set_error("world/rank/tp/align out of range");
        return DR_ERR_INVALID;
    }
    uint32_t al = b->arena_align_bytes;
    if (al < 16 || (al & (al - 1))) {
        set_error("arena_align_bytes must be a power of two >= 16");
        return DR_ERR_INVALID;
    }
    if (b->dtype == DR_FP8_E4M3_B128 && !a->gathered && a->world > 1) {
        set_error("fp8 block scaling needs the whole flat buffer (gathered = 1)");
        return DR_ERR_UNSUPPORTED;
    }
    if (b->moe_tp != 1 && b->moe_tp != tp) {
        set_error("moe_tp must be 1 (experts unsliced) or tp");
        return DR_ERR_UNSUPPORTED;
    }
    const bool kv_ok = s->n_kv_heads % tp == 0 || (b->kv_replicate && tp > s->n_kv_heads && tp % s->n_kv_heads == 0);
    const uint64_t vp = b->vocab_pad ? ((uint64_t)s->vocab + b->vocab_pad - 1) / b->vocab_pad * b->vocab_pad : s->vocab;
    if (s->n_q_heads % tp || !kv_ok || vp % tp || (s->n_experts == 0 && s->ffn % tp) ||
        (s->n_experts && b->moe_tp > 1 && s->moe_ffn % tp)) {
        set_error("n_q_heads, n_kv_heads (or tp a multiple of it with kv_replicate), ffn and the padded vocabulary "
                  "must be divisible by tp");
        return DR_ERR_UNSUPPORTED;
    }
    const uint32_t ep = b->moe_ep ? b->moe_ep : 1;
    if (b->moe_ep_rank >= ep) {
        set_error("moe_ep_rank out of range");
        return DR_ERR_INVALID;
    }
    if (s->n_experts % ep) {
        set_error("moe_ep must divide n_experts");
        return DR_ERR_UNSUPPORTED;
    }
    return DR_OK;
}

int create(const dr_model_spec* s, const dr_src_layout* a, const dr_dst_layout* b, uint32_t tp, uint32_t rank,
           bool host_only, dr_plan** out)
{
    if (!out) {
        set_error("NULL out");
        return DR_ERR_INVALID;
    }
    *out = nullptr;
    int rc = validate(s, a, b, tp, rank);
    if (rc) return rc;
    dr_plan* p = new (std::nothrow) dr_plan();
    if (!p) return DR_ERR_NOMEM;
    p->spec = *s;
    p->src = *a;
    p->dst = *b;
    p->tp = tp;
    p->tp_rank = rank;
    p->elem_size = b->dtype == DR_F32 ? 4 : 2;
    p->fp8 = b->dtype == DR_FP8_E4M3_B128;
    p->host_only = host_only;
    try {
        rc = compile_plan(p);
    } catch (const std::bad_alloc&) {
        rc = DR_ERR_NOMEM;
    }
    if (rc == DR_OK && !host_only) {
        cudaError_t e = cudaGetDevice(&p->device);
        size_t bytes = p->dev_segs.size() * sizeof(DevSeg);
        if (e == cudaSuccess && bytes) e = cudaMalloc((void**)&p->d_segs, bytes);
        if (e == cudaSuccess && bytes) e = cudaMemcpy(p->d_segs, p->dev_segs.data(), bytes, cudaMemcpyHostToDevice);
        size_t hbytes = p->hints.size() * sizeof(uint32_t);
        if (e == cudaSuccess) e = cudaMalloc((void**)&p->d_hints, hbytes);
        if (e == cudaSuccess) e = cudaMemcpy(p->d_hints, p->hints.data(), hbytes, cudaMemcpyHostToDevice);
        auto upload = [&](void** dst, const void* src, size_t n) {
            if (e == cudaSuccess && n) e = cudaMalloc(dst, n);
            if (e == cudaSuccess && n) e = cudaMemcpy(*dst, src, n, cudaMemcpyHostToDevice);
        };
        if (p->fp8) {
            upload((void**)&p->d_qtensors, p->qtensors.data(), p->qtensors.size() * sizeof(QTensor));
            upload((void**)&p->d_qparts, p->qparts.data(), p->qparts.size() * sizeof(QPart));
            upload((void**)&p->d_qhints, p->qhints.data(), p->qhints.size() * sizeof(uint32_t));
        }
        if (e == cudaSuccess) p->grid = choose_grid(p->device, p->elem_size);
        if (e != cudaSuccess || p->grid <= 0) {
            set_error("plan upload: %s", cudaGetErrorString(e));
            rc = e == cudaErrorMemoryAllocation ? DR_ERR_NOMEM : DR_ERR_CUDA;
        } else {
            rc = ensure_bulk_smem(p->device);  // keeps its own error message
        }
    }
    if (rc) {
        dr_plan_destroy(p);
        return rc;
    }
    *out = p;
    return DR_OK;
}

int check_call(const dr_plan* p, const void* a, uint64_t a_bytes, uint64_t a_need, const void* b, uint64_t b_bytes,
               uint64_t b_need)
{
    if (!p || (!a && a_need) || (!b && b_need)) {
        set_error("NULL plan or buffer");
        return DR_ERR_INVALID;
    }
    if (p->host_only) {
        set_error("host-only plan cannot launch");
        return DR_ERR_STATE;
    }
    if (a_bytes < a_need || b_bytes < b_need) {
        set_error("buffer too small: have %llu / %llu bytes, need %llu / %llu", (unsigned long long)a_bytes,
                  (unsigned long long)b_bytes, (unsigned long long)a_need, (unsigned long long)b_need);
        return DR_ERR_SIZE;
    }
    if (((uintptr_t)a | (uintptr_t)b) & 15) {
        set_error("base pointers must be 16-byte aligned");
        return DR_ERR_ALIGN;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) {
        set_error("current device differs from the plan's device");
        return DR_ERR_STATE;
    }
    return DR_OK;
}

}  // namespace
}  // namespace dr

using namespace dr;

extern "C" {

int dr_plan_create(const dr_model_spec* spec, const dr_src_layout* src, const dr_dst_layout* dst, uint32_t tp,
                   uint32_t rank, dr_plan** out)
{
    return create(spec, src, dst, tp, rank, false, out);
}

int dr_plan_create_host(const dr_model_spec* spec, const dr_src_layout* src, const dr_dst_layout* dst, uint32_t tp,
                        uint32_t rank, dr_plan** out)
{
    return create(spec, src, dst, tp, rank, true, out);
}

int dr_plan_window_host(const dr_plan* plan, uint64_t src_elem_lo, uint64_t src_elem_hi, dr_plan** out)
{
    if (!plan || !out) {
        set_error("NULL argument");
        return DR_ERR_INVALID;
    }
    *out = nullptr;
    if (plan->fp8) {
        set_error("fp8 plans have no source windows");
        return DR_ERR_UNSUPPORTED;
    }
    if (src_elem_lo >= src_elem_hi || src_elem_hi > plan->info.src_bytes / 4) {
        set_error("window is empty or outside the source buffer");
        return DR_ERR_INVALID;
    }
    dr_plan* w = new (std::nothrow) dr_plan();
    if (!w) return DR_ERR_NOMEM;
    w->spec = plan->spec;
    w->src = plan->src;
    w->dst = plan->dst;
    w->tp = plan->tp;
    w->tp_rank = plan->tp_rank;
    w->elem_size = plan->elem_size;
    w->bulk_forward = plan->bulk_forward;
    w->host_only = true;
    int rc = DR_OK;
    try {
        w->tensors = plan->tensors;
        w->segs = window_segments(plan->segs, src_elem_lo, src_elem_hi, plan->elem_size);
        Tables tb;
        rc = build_tables(w->segs, &tb);
        if (rc == DR_OK) {
            w->dev_segs.swap(tb.segs);
            w->hints.swap(tb.hints);
            w->hint_shift = tb.hint_shift;
            w->info = plan->info;
            w->info.src_bytes = 4 * (src_elem_hi - src_elem_lo);
            w->info.n_segments = w->segs.size();
            w->info.bulk_forward = plan->info.bulk_forward;
            w->info.n_tiles = tb.n_tiles;
            w->info.elems_moved = tb.elems;
            w->info.bytes_moved_fwd = w->info.bytes_moved_inv = tb.elems * (4 + plan->elem_size);
        }
    } catch (const std::bad_alloc&) {
        rc = DR_ERR_NOMEM;
    }
    if (rc) {
        dr_plan_destroy(w);
        return rc;
    }
    *out = w;
    return DR_OK;
}

int dr_plan_query(const dr_plan* plan, dr_plan_info* out)
{
    if (!plan || !out) {
        set_error("NULL argument");
        return DR_ERR_INVALID;
    }
    *out = plan->info;
    return DR_OK;
}

int dr_plan_tensor(const dr_plan* plan, uint32_t i, dr_tensor_desc* out)
{
    if (!plan || !out || i >= plan->tensors.size()) {
        set_error("bad tensor index");
        return DR_ERR_INVALID;
    }
    const Tensor& t = plan->tensors[i];
    memset(out, 0, sizeof *out);
    snprintf(out->name, sizeof out->name, "%s", t.name.c_str());
    out->arena_off = t.arena_off;
    out->rows = t.rows;
    out->cols = t.cols;
    out->alias_of = t.alias_of;
    out->elem_size = t.es;
    out->quantised = t.quant ? 1 : 0;
    out->scale_off = t.scale_off;
    out->scale_rows = t.quant ? (t.rows + 127) / 128 : 0;
    out->scale_cols = t.quant ? (t.cols + 127) / 128 : 0;
    return DR_OK;
}

int dr_plan_segment(const dr_plan* plan, uint64_t i, dr_segment_desc* out)
{
    if (!plan || !out || i >= plan->segs.size()) {
        set_error("bad segment index");
        return DR_ERR_INVALID;
    }
    const HostSeg& g = plan->segs[i];
    out->dst_off = g.dst_off;
    out->src_off = g.src_off;
    out->rows = g.rows;
    out->row_len = g.row_len;
    out->src_row_stride = g.src_stride;
    out->dst_row_stride = g.dst_stride;
    out->vector_bytes = (g.flags & kSegVec32) ? 32 : (g.flags & kSegVec16) ? 16 : 0;
    out->tensor = g.tensor;
    return DR_OK;
}

int dr_reshard(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* dst_dev, uint64_t dst_bytes,
               void* cuda_stream)
{
    int rc = check_call(plan, src_dev, src_bytes, plan ? plan->info.src_bytes : 0, dst_dev, dst_bytes,
                        plan ? plan->info.dst_bytes : 0);
    if (rc) return rc;
    rc = launch_reshard(plan, false, src_dev, dst_dev, nullptr, cuda_stream);
    if (rc == DR_OK && plan->fp8) rc = launch_quant(plan, src_dev, dst_dev, cuda_stream);
    return rc;
}

int dr_plan_group(const dr_plan* plan, uint32_t g, dr_group_desc* out)
{
    if (!plan || !out || g >= plan->groups.size()) {
        set_error("bad group index");
        return DR_ERR_INVALID;
    }
    const Group& G = plan->groups[g];
    out->first_tensor = G.first_tensor;
    out->n_tensors = G.n_tensors;
    out->elems = G.elems + G.qelems;
    out->bytes_moved = G.elems * (4 + plan->elem_size) + G.qelems * 5 + (G.qblock_hi - G.qblock_lo) * 4;
    return DR_OK;
}

int dr_reshard_groups(const dr_plan* plan, uint32_t first, uint32_t count, const void* src_dev, uint64_t src_bytes,
                      void* dst_dev, uint64_t dst_bytes, void* cuda_stream)
{
    int rc = check_call(plan, src_dev, src_bytes, plan ? plan->info.src_bytes : 0, dst_dev, dst_bytes,
                        plan ? plan->info.dst_bytes : 0);
    if (rc) return rc;
    if (count == 0 || first >= plan->groups.size() || count > plan->groups.size() - first) {
        set_error("group range outside the plan's %zu groups", plan->groups.size());
        return DR_ERR_INVALID;
    }
    // groups own consecutive tile ranges: the union of the non-empty ones is one range
    uint64_t lo = ~0ull, hi = 0, qlo = ~0ull, qhi = 0;
    for (uint32_t g = first; g < first + count; ++g) {
        const Group& G = plan->groups[g];
        if (G.tile_hi > G.tile_lo) {
            lo = G.tile_lo < lo ? G.tile_lo : lo;
            hi = G.tile_hi > hi ? G.tile_hi : hi;
        }
        if (G.qblock_hi > G.qblock_lo) {  // fp8 plans: the groups' quantisation blocks, consecutive as well
            qlo = G.qblock_lo < qlo ? G.qblock_lo : qlo;
            qhi = G.qblock_hi > qhi ? G.qblock_hi : qhi;
        }
    }
    if (hi != 0) rc = launch_reshard(plan, false, src_dev, dst_dev, nullptr, cuda_stream, lo, hi);
    if (rc == DR_OK && qhi != 0) rc = launch_quant(plan, src_dev, dst_dev, cuda_stream, qlo, qhi);
    return rc;  // nothing launched when none of these groups lies in this shard
}

int dr_plan_ranges(const dr_plan* plan, uint64_t max_ranges, dr_range* out, uint64_t* n_ranges)
{
    if (!plan || !n_ranges || (max_ranges && !out)) {
        set_error("NULL argument");
        return DR_ERR_INVALID;
    }
    if (plan->fp8) {
        set_error("fp8 plans have no exchange ranges: a block is scaled from all of its elements");
        return DR_ERR_UNSUPPORTED;
    }
    try {
        std::vector<dr_range> v = plan_ranges(plan);
        *n_ranges = v.size();
        for (uint64_t i = 0; i < v.size() && i < max_ranges; ++i) out[i] = v[i];
    } catch (const std::bad_alloc&) {
        return DR_ERR_NOMEM;
    }
    return DR_OK;
}

int dr_reshard_push(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* const* dst_dev, uint32_t n_dst,
                    uint64_t dst_bytes, void* cuda_stream)
{
    if (!dst_dev || n_dst == 0 || n_dst > DR_MAX_PUSH_DST) {
        set_error("n_dst must be 1..%u and dst_dev non-NULL", DR_MAX_PUSH_DST);
        return DR_ERR_INVALID;
    }
    for (uint32_t i = 0; i < n_dst; ++i) {
        int rc = check_call(plan, src_dev, src_bytes, plan ? plan->info.src_bytes : 0, dst_dev[i], dst_bytes,
                            plan ? plan->info.dst_bytes : 0);
        if (rc) return rc;
    }
    if (plan->fp8) {
        set_error("fp8 plans cannot be pushed shard by shard");
        return DR_ERR_UNSUPPORTED;
    }
    return launch_push(plan, src_dev, dst_dev, n_dst, cuda_stream);
}

int dr_reshard_inverse(const dr_plan* plan, const void* rollout_dev, uint64_t rollout_bytes, void* flat_dev,
                       uint64_t flat_bytes, void* cuda_stream)
{
    int rc = check_call(plan, rollout_dev, rollout_bytes, plan ? plan->info.dst_bytes : 0, flat_dev, flat_bytes,
                        plan ? plan->info.src_bytes : 0);
    if (rc) return rc;
    rc = launch_reshard(plan, true, nullptr, flat_dev, rollout_dev, cuda_stream);
    if (rc == DR_OK && plan->fp8) rc = launch_dequant(plan, rollout_dev, flat_dev, cuda_stream);
    return rc;
}

int dr_shard_range(uint64_t flat_elems, uint32_t world, uint32_t rank, uint64_t* begin, uint64_t* end,
                   uint64_t* shard_elems)
{
    if (!world || rank >= world || !begin || !end) {
        set_error("bad world/rank or NULL output");
        return DR_ERR_INVALID;
    }
    const uint64_t S = (flat_elems + world - 1) / world;
    const uint64_t lo = (uint64_t)rank * S, hi = lo + S;
    *begin = lo < flat_elems ? lo : flat_elems;
    *end = hi < flat_elems ? hi : flat_elems;
    if (shard_elems) *shard_elems = S;
    return DR_OK;
}

int dr_plan_destroy(dr_plan* plan)
{
    if (!plan) return DR_OK;
    if (plan->stream) stream_destroy(plan->stream);
    if (plan->ring) ring_destroy(plan->ring);
    if (plan->d_segs) cudaFree(plan->d_segs);
    if (plan->d_hints) cudaFree(plan->d_hints);
    if (plan->d_qtensors) cudaFree(plan->d_qtensors);
    if (plan->d_qparts) cudaFree(plan->d_qparts);
    if (plan->d_qhints) cudaFree(plan->d_qhints);
    delete plan;
    return DR_OK;
}

int dr_diag_bulk_wait_failures(uint64_t* count)
{
    if (!count) {
        set_error("NULL argument");
        return DR_ERR_INVALID;
    }
    return bulk_wait_failures(count);
}

int dr_diag_bulk_starve(int on) { return bulk_starve(on); }

const char* dr_strerror(int status)
{
    switch (status) {
    case DR_OK: return "ok";
    case DR_ERR_INVALID: return "invalid argument";
    case DR_ERR_UNSUPPORTED: return "unsupported layout";
    case DR_ERR_SIZE: return "buffer too small";
    case DR_ERR_ALIGN: return "misaligned base pointer";
    case DR_ERR_NOMEM: return "out of memory";
    case DR_ERR_CUDA: return "CUDA error";
    case DR_ERR_BUDGET: return "staging budget cannot hold two chunk slots";
    case DR_ERR_SINK: return "chunk callback failed";
    case DR_ERR_TIMEOUT: return "wait timed out";
    case DR_ERR_STATE: return "call not valid in this state";
    default: return "unknown status";
    }
}

const char* dr_last_error(void) { return g_err; }

}  // extern "C"
