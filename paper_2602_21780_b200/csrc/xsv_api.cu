// Host layer of the xsv library: the cache object, its HBM layout and buffer
// rotation, the closed-form length schedule and the per-step launch sequence.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>
#include <cstdlib>
#include <vector>

#include "../../include/xsv.h"
#include "xsv_kernels.h"

static std::atomic<long long> g_launches{0};
void xsv_count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static thread_local cudaError_t g_last_cuda = cudaSuccess;

namespace {

// records the CUDA error behind an XSV_ERR_CUDA return (see xsv_last_cuda_error)
inline xsv_status cuda_fail(cudaError_t e) {
    g_last_cuda = e;
    cudaGetLastError();   // clear the runtime's sticky copy of a launch-configuration error
    return XSV_ERR_CUDA;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct BufSet {
    void* slab = nullptr;
    LayerView view{};
};

struct PendingEvent {
    int phase;
    cudaEvent_t a, b;
};

}  // namespace

struct xsv_cache {
    int device = 0;
    int layers = 0, H = 0, d = 0, bits = 0;
    long long L_max = 0;
    int n_special = 5, g = 16, G = 64;
    int F_max = 0;           // most tokens a frame may hold (0 until known: set_options, or the first frame's size)
    int dtype = -1;          // xsv_dtype of the first step
    long long max_cache_tokens = 0;
    long long cap = 0;       // capacity in tokens of each buffer set
    bool allocated = false;
    bool stepped = false;
    int attn_impl = XSV_ATTN_AUTO;

    std::vector<BufSet> bufs;          // layers + 1 (one spare for out-of-place compaction)
    std::vector<int> buf_of_layer;
    int spare = 0;
    std::vector<long long> len, frames;
    std::vector<long long> tokens_seen;   // per layer: tokens of all frames so far (the origin of the next frame's first token)
    std::vector<int> F_first;             // per layer: tokens of its first frame (T_first of Eq. 8), 0 before the first step

    // scratch shared by all layers (steps are ordered on one stream)
    float* qpart = nullptr;
    float* attn_ws = nullptr;   // parts of query tiles shared by several CTAs (tcgen05 attention)
    float* scores = nullptr;
    int* srcmap = nullptr;
    int* dscal = nullptr;    // [0] frozen key groups of the current pruning step
    int* status = nullptr;   // sticky device status word
    void* scratch_slab = nullptr;
    long long last_scores_n = 0;

    // staging for xsv_step_host: two slots of (Q, K, V, out), a copy-in and a copy-out stream
    void* stage = nullptr;
    size_t stage_bytes = 0;
    cudaStream_t cs_in = nullptr, cs_out = nullptr;
    cudaStream_t cs_sel = nullptr;                          // selection, then the keys' re-quantisation, beside the attention kernel
    cudaStream_t cs_val = nullptr;                          // the values, beside the keys
    cudaEvent_t ev_scored = nullptr, ev_selected = nullptr, ev_picked = nullptr, ev_values = nullptr;
    bool defer_join = false;                                // the caller's stream does not wait for the side streams at the end of a step
    bool select_outstanding = false;                        // a selection has been enqueued that the caller's stream has not waited for
    std::vector<cudaEvent_t> ev_keys_of, ev_vals_of;        // per layer: end of its side-stream work (deferred join)
    std::vector<char> side_pending;                         // per layer: the caller's stream has not yet waited for those
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    bool slot_used[2] = {false, false}, out_pending[2] = {false, false};
    bool slot_deferred[2] = {false, false};                 // the step that last read the slot left side-stream work outstanding
    int slot_layer[2] = {0, 0};                             // the layer whose step last read the slot
    bool defer_output = false;
    unsigned long long host_calls = 0;

    size_t bytes = 0;

    int profiling = 0;          // 0 off, 1 events around every phase, 2 around the attention phase only, 3 around every 7th one, 4 as 1 with every kernel on the caller's stream
    unsigned long long attn_calls = 0;
    std::vector<PendingEvent> pending;
    std::vector<cudaEvent_t> free_events;
    double prof_ms[XSV_PHASE_COUNT] = {0, 0, 0, 0};
    long long prof_launches[XSV_PHASE_COUNT] = {0, 0, 0, 0};
};

namespace {

size_t bufset_bytes(const xsv_cache* c, long long cap, size_t off[7]) {
    const int rowb = c->bits == 16 ? c->d * 2 : c->d * c->bits / 8;
    const long long capg = (cap + XSV_G - 1) / XSV_G;
    size_t o = 0;
    off[0] = o; o = align_up(o + (size_t)c->H * cap * rowb, 256);                 // kcodes
    off[1] = o; o = align_up(o + (size_t)c->H * cap * rowb, 256);                 // vcodes
    off[2] = o; if (c->bits < 16) o = align_up(o + (size_t)c->H * capg * 64 * 4, 256);   // kscale
    off[3] = o; if (c->bits < 16) o = align_up(o + (size_t)c->H * capg * 64 * 4, 256);   // kzero
    off[4] = o; if (c->bits < 16) o = align_up(o + (size_t)c->H * cap * 4, 256);  // vscale
    off[5] = o; if (c->bits < 16) o = align_up(o + (size_t)c->H * cap * 4, 256);  // vzero
    off[6] = o; o = align_up(o + (size_t)cap * 8, 256);                           // origin
    return o;
}

void release_device_memory(xsv_cache* c) {
    for (auto& b : c->bufs) if (b.slab) cudaFree(b.slab);
    c->bufs.clear();
    if (c->scratch_slab) cudaFree(c->scratch_slab);
    c->scratch_slab = nullptr;
}

// Streams and events of the cache: created once, with the device memory, so that no later step creates any.
cudaError_t create_streams_and_events(xsv_cache* c) {
    cudaError_t e;
    if ((e = cudaStreamCreateWithFlags(&c->cs_sel, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&c->cs_val, cudaStreamNonBlocking)) != cudaSuccess) return e;
    cudaEvent_t* single[4] = {&c->ev_scored, &c->ev_selected, &c->ev_picked, &c->ev_values};
    for (cudaEvent_t* ev : single)
        if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return e;
    c->ev_keys_of.assign(c->layers, nullptr);
    c->ev_vals_of.assign(c->layers, nullptr);
    c->side_pending.assign(c->layers, 0);
    for (int l = 0; l < c->layers; ++l) {
        if ((e = cudaEventCreateWithFlags(&c->ev_keys_of[l], cudaEventDisableTiming)) != cudaSuccess) return e;
        if ((e = cudaEventCreateWithFlags(&c->ev_vals_of[l], cudaEventDisableTiming)) != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// All device memory of the cache (and its streams and events).  Capacity: a bounded cache never holds more than
// max(L_max, first frame + current frame) tokens, and neither frame exceeds F_max.
xsv_status allocate(xsv_cache* c) {
    if (c->allocated) return XSV_OK;
    const long long F = c->F_max;
    long long cap;
    if (c->L_max > 0) cap = c->L_max > 2 * F ? c->L_max : 2 * F;
    else cap = c->max_cache_tokens > 0 ? c->max_cache_tokens : 16 * F;
    if (cap < F) cap = F;
    cap = (long long)align_up((size_t)cap, 128);   // whole attention tiles
    c->cap = cap;
    size_t off[7];
    const size_t per = bufset_bytes(c, cap, off);
    const int nb = c->layers + (c->L_max > 0 ? 1 : 0);
    c->bufs.assign(nb, BufSet{});
    size_t total = 0;
    for (int i = 0; i < nb; ++i) {
        void* p = nullptr;
        if (cudaMalloc(&p, per) != cudaSuccess) { cudaGetLastError(); release_device_memory(c); return XSV_ERR_OOM; }
        c->bufs[i].slab = p;
        if (cudaMemset(p, 0, per) != cudaSuccess) { release_device_memory(c); return XSV_ERR_CUDA; }
        BufSet& b = c->bufs[i];
        uint8_t* base = (uint8_t*)p;
        b.view.kcodes = base + off[0];
        b.view.vcodes = base + off[1];
        b.view.kscale = (float*)(base + off[2]);
        b.view.kzero = (float*)(base + off[3]);
        b.view.vscale = (float*)(base + off[4]);
        b.view.vzero = (float*)(base + off[5]);
        b.view.origin = (long long*)(base + off[6]);
        b.view.cap = cap;
        b.view.capg = (int)((cap + XSV_G - 1) / XSV_G);
        b.view.rowb = c->bits == 16 ? c->d * 2 : c->d * c->bits / 8;
        b.view.bits = c->bits;
        total += per;
    }
    c->buf_of_layer.resize(c->layers);
    for (int l = 0; l < c->layers; ++l) c->buf_of_layer[l] = l;
    c->spare = c->layers;   // valid only when nb == layers + 1
    // scratch: qpart | scores | srcmap | dscal | status | attention parts
    size_t so = 0;
    const size_t o_q = so; so = align_up(so + (size_t)c->H * XSV_QCHUNKS * 64 * 4, 256);
    const size_t o_s = so; so = align_up(so + (size_t)cap * 4, 256);
    const size_t o_m = so; so = align_up(so + (size_t)cap * 4, 256);
    const size_t o_d = so; so = align_up(so + 64, 256);
    const size_t o_t = so; so = align_up(so + 64, 256);
    const size_t o_w = so; so = align_up(so + xsv_attn_tc5_workspace_bytes(), 256);
    if (cudaMalloc(&c->scratch_slab, so) != cudaSuccess) { cudaGetLastError(); release_device_memory(c); return XSV_ERR_OOM; }
    if (cudaMemset(c->scratch_slab, 0, so) != cudaSuccess) { release_device_memory(c); return XSV_ERR_CUDA; }
    uint8_t* sb = (uint8_t*)c->scratch_slab;
    c->qpart = (float*)(sb + o_q);
    c->scores = (float*)(sb + o_s);
    c->srcmap = (int*)(sb + o_m);
    c->dscal = (int*)(sb + o_d);
    c->status = (int*)(sb + o_t);
    c->attn_ws = (float*)(sb + o_w);
    if (!c->cs_sel) {
        const cudaError_t e = create_streams_and_events(c);
        if (e != cudaSuccess) { release_device_memory(c); g_last_cuda = e; cudaGetLastError(); return XSV_ERR_CUDA; }
    }
    c->bytes = total + so;
    c->allocated = true;
    return XSV_OK;
}

cudaEvent_t get_event(xsv_cache* c) {
    if (!c->free_events.empty()) {
        cudaEvent_t e = c->free_events.back();
        c->free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

// The selection kernel is one block; XSV_NO_SIDE_SELECT keeps it on the caller's stream (for comparisons).
bool side_select_enabled() {
    static const bool on = (getenv("XSV_NO_SIDE_SELECT") == nullptr);
    return on;
}

// Host-side wait for the cache's own streams (after the caller's stream has been synchronised).
cudaError_t sync_side_streams(xsv_cache* c) {
    cudaError_t e = cudaSuccess;
    if (c->cs_sel) e = cudaStreamSynchronize(c->cs_sel);
    if (e == cudaSuccess && c->cs_val) e = cudaStreamSynchronize(c->cs_val);
    for (auto& p : c->side_pending) p = 0;
    c->select_outstanding = false;
    return e;
}

struct PhaseTimer {
    xsv_cache* c;
    cudaStream_t st;
    int phase;
    cudaEvent_t a = nullptr, b = nullptr;
    long long launches0;
    bool on;
    PhaseTimer(xsv_cache* c_, cudaStream_t st_, int phase_) : c(c_), st(st_), phase(phase_) {
        launches0 = g_launches.load(std::memory_order_relaxed);
        on = c->profiling == 1 || c->profiling == 4 || (c->profiling == 2 && phase == XSV_PHASE_ATTN) ||
             (c->profiling == 3 && phase == XSV_PHASE_ATTN && (c->attn_calls++ % 7ull) == 0ull);
        if (on) {
            a = get_event(c);
            b = get_event(c);
            cudaEventRecord(a, st);
        }
    }
    ~PhaseTimer() {
        if (on) {
            cudaEventRecord(b, st);
            c->pending.push_back({phase, a, b});
            c->prof_launches[phase] += g_launches.load(std::memory_order_relaxed) - launches0;
        }
    }
};

}  // namespace

extern "C" {

const char* xsv_strerror(xsv_status s) {
    switch (s) {
        case XSV_OK: return "ok";
        case XSV_ERR_ARG: return "invalid argument";
        case XSV_ERR_SHAPE: return "shape, dtype or alignment mismatch";
        case XSV_ERR_ORDER: return "call out of order";
        case XSV_ERR_OOM: return "out of memory";
        case XSV_ERR_CUDA: return "CUDA runtime error";
        case XSV_ERR_TIMEOUT: return "bounded device-side wait ran out";
        case XSV_ERR_RANGE: return "a 16-bit input beyond the supported range of +-65504";
        case XSV_ERR_CAPACITY: return "unbounded cache exceeded max_cache_tokens";
        case XSV_ERR_LIMIT: return "size exceeds the fixed maximum of this no-allocation entry point";
    }
    return "unknown status";
}

const char* xsv_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda); }

long long xsv_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

xsv_status xsv_cache_create(xsv_cache** out, int layers, int heads, int head_dim, long long budget_tokens, int bits) {
    if (!out) return XSV_ERR_ARG;
    *out = nullptr;
    if (layers <= 0 || layers > 4096 || heads <= 0 || heads > 1024) return XSV_ERR_ARG;
    if (head_dim != XSV_D) return XSV_ERR_ARG;
    if (!(bits == 2 || bits == 4 || bits == 8 || bits == 16)) return XSV_ERR_ARG;
    if (budget_tokens > (1LL << 30)) return XSV_ERR_ARG;
    xsv_cache* c = new (std::nothrow) xsv_cache();
    if (!c) return XSV_ERR_OOM;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; cudaGetLastError(); return XSV_ERR_CUDA; }
    c->layers = layers; c->H = heads; c->d = head_dim; c->bits = bits;
    c->L_max = budget_tokens > 0 ? budget_tokens : 0;
    c->len.assign(layers, 0);
    c->frames.assign(layers, 0);
    c->tokens_seen.assign(layers, 0);
    c->F_first.assign(layers, 0);
    *out = c;
    return XSV_OK;
}

xsv_status xsv_cache_set_options(xsv_cache* c, int n_special, int pool_group, int quant_group, int max_frame_tokens,
                                 long long max_cache_tokens) {
    if (!c) return XSV_ERR_ARG;
    if (c->stepped || c->allocated) return XSV_ERR_ORDER;
    if (pool_group == 0 || (quant_group >= 0 && quant_group != XSV_G)) return XSV_ERR_ARG;
    if (max_frame_tokens > (1 << 24) || max_cache_tokens > (1LL << 30)) return XSV_ERR_ARG;
    if (n_special >= 0) c->n_special = n_special;
    if (pool_group > 0) c->g = pool_group;
    if (max_cache_tokens >= 0) c->max_cache_tokens = max_cache_tokens;
    if (max_frame_tokens > 0) {
        if (c->n_special > max_frame_tokens) return XSV_ERR_ARG;
        c->F_max = max_frame_tokens;
        cudaSetDevice(c->device);
        const xsv_status st = allocate(c);
        if (st != XSV_OK) c->F_max = 0;
        return st;
    }
    return XSV_OK;
}

xsv_status xsv_cache_set_attn_impl(xsv_cache* c, xsv_attn_impl impl) {
    if (!c || impl < XSV_ATTN_AUTO || impl > XSV_ATTN_TC5) return XSV_ERR_ARG;
    c->attn_impl = impl;
    return XSV_OK;
}

}  // extern "C"

namespace {

// What one step of one cache comes to, worked out on the host before anything is launched.
struct StepPlan {
    xsv_cache* c;
    int layer;
    const void *Q, *K, *V;
    void* out;
    int dtype, F, H;
    long long T_c, T, t, origin0;
    bool prune, side_select, append_only;
    bool scores_on_side;      // the scores run on the cache's own stream too (several caches stepped together)
    int cur, T_first, n_mid, k;
};

// Argument, shape and order checks, allocation on the first step, and the step's quantities.  Launches nothing.
xsv_status plan_step(xsv_cache* c, int layer, const void* Q, const void* K, const void* V, int n_tokens, xsv_dtype dtype,
                     void* out, bool append_only, StepPlan& p) {
    if (!c || !Q || !K || !V || !out) return XSV_ERR_ARG;
    if (layer < 0 || layer >= c->layers || n_tokens <= 0) return XSV_ERR_ARG;
    if (dtype != XSV_F16 && dtype != XSV_BF16) return XSV_ERR_ARG;
    if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V) & 15) return XSV_ERR_SHAPE;
    if (!append_only && ((uintptr_t)out & 15)) return XSV_ERR_SHAPE;
    if (out == Q || out == K || out == V) return XSV_ERR_ARG;
    if (c->F_max != 0 && n_tokens > c->F_max) return XSV_ERR_SHAPE;   // frames may differ in size up to max_frame_tokens
    if (c->dtype >= 0 && (int)dtype != c->dtype) return XSV_ERR_SHAPE;
    if (c->n_special > n_tokens) return XSV_ERR_ARG;
    long long min_frames = c->frames[0];
    for (int l = 1; l < c->layers; ++l) min_frames = c->frames[l] < min_frames ? c->frames[l] : min_frames;
    if (c->frames[layer] > min_frames) return XSV_ERR_ORDER;   // this layer already took the current frame
    if (!c->allocated) {
        c->F_max = n_tokens;          // not told otherwise: no later frame is larger than the first
        cudaSetDevice(c->device);
        xsv_status s = allocate(c);
        if (s != XSV_OK) { c->F_max = 0; return s; }
    }
    p.c = c; p.layer = layer; p.Q = Q; p.K = K; p.V = V; p.out = out; p.dtype = (int)dtype; p.append_only = append_only;
    p.F = n_tokens; p.H = c->H;
    p.T_c = c->len[layer];
    p.T = p.T_c + p.F;
    p.t = c->frames[layer] + 1;
    p.prune = p.t >= 2 && c->L_max > 0 && p.T > c->L_max;
    if (!p.prune && p.T > c->cap) return XSV_ERR_CAPACITY;
    if (append_only && p.prune) return XSV_ERR_ORDER;      // a step that prunes needs the frame's queries (Eq. 3-7)
    p.cur = c->buf_of_layer[layer];
    // Eq. 8 with the sizes of the first and of the current frame as separate quantities:
    // k = max(0, L_max - T_first - T_current) of the middle segment's T_c - T_first tokens are kept.
    p.origin0 = c->tokens_seen[layer];
    p.T_first = p.t == 1 ? p.F : c->F_first[layer];
    p.n_mid = (int)(p.T_c - p.T_first);
    const long long kk = c->L_max - p.T_first - p.F;
    p.k = (int)(kk > 0 ? kk : 0);
    // The scores (Eq. 3-7) need the frame's queries and the cached keys only, so they come first; the selection
    // (Eq. 8), one block that is bound by latency, then runs on a stream of its own: it takes the first multiprocessor
    // that an attention CTA leaves (the CTAs' finishing times are spread over some tens of microseconds) and what
    // follows it takes the next ones.  (Keeping one multiprocessor free of attention CTAs for that stream from the
    // start gives 0.7 % more frames per second and 3 % less throughput of the attention kernel; not done.)
    p.side_select = p.prune && side_select_enabled() && c->profiling != 4 && c->attn_impl != XSV_ATTN_MMA && c->attn_ws != nullptr;
    return XSV_OK;
}

// Everything of the step that comes before the attention kernel on the caller's stream: the waits for earlier
// side-stream work, the scores, and (on the cache's own streams) the selection and the re-quantisation.
xsv_status launch_before_attention(const StepPlan& p, cudaStream_t st) {
    xsv_cache* c = p.c;
    const int layer = p.layer, F = p.F, H = p.H, T_first = p.T_first, k = p.k;
    const LayerView& lv = c->bufs[p.cur].view;
    cudaError_t e;
    c->dtype = p.dtype;
    c->stepped = true;
    // Deferred join: side-stream work of earlier steps may still be running.  This layer's own must have ended before
    // its cache is read, and the last selection before the score buffer is rewritten.
    if (!c->side_pending.empty() && c->side_pending[layer]) {
        if ((e = cudaStreamWaitEvent(st, c->ev_keys_of[layer], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(st, c->ev_vals_of[layer], 0)) != cudaSuccess) return cuda_fail(e);
        c->side_pending[layer] = 0;
    }
    if (c->select_outstanding) {
        if ((e = cudaStreamWaitEvent(st, c->ev_picked, 0)) != cudaSuccess) return cuda_fail(e);
        c->select_outstanding = false;
    }
    if (!p.prune) return XSV_OK;
    const bool side_scores = p.side_select && p.scores_on_side;
    if (side_scores) {
        // Several caches stepped together: each cache's scores run on its own stream, side by side with the other
        // caches', from the point the caller's stream has reached (the inputs are ready there).
        if (c->defer_join && (e = cudaStreamWaitEvent(c->cs_sel, c->ev_values, 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventRecord(c->ev_scored, st)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(c->cs_sel, c->ev_scored, 0)) != cudaSuccess) return cuda_fail(e);
    }
    {   // ---- Eq. 3-7
        cudaStream_t sc_st = side_scores ? c->cs_sel : st;
        PhaseTimer pt(c, sc_st, XSV_PHASE_SCORE);
        e = xsv_launch_qtilde(p.Q, p.dtype, H, F, c->n_special, c->g, c->qpart, sc_st);
        if (e != cudaSuccess) return cuda_fail(e);
        const int n_pooled = c->n_special + (F - c->n_special + c->g - 1) / c->g;
        const float qnorm = 1.0f / ((float)H * (float)n_pooled);
        if (c->bits == 16) e = xsv_launch_score_raw(lv, p.dtype, H, T_first, (int)p.T_c, c->qpart, qnorm, c->scores, sc_st);
        else e = xsv_launch_score(lv, H, T_first, (int)p.T_c, c->qpart, qnorm, c->scores, sc_st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    cudaStream_t sel_st = st;
    if (p.side_select) {
        if (!side_scores) {
            // the new selection overwrites the kept-position map that the values of the previous step may still read
            if (c->defer_join && (e = cudaStreamWaitEvent(c->cs_sel, c->ev_values, 0)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventRecord(c->ev_scored, st)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamWaitEvent(c->cs_sel, c->ev_scored, 0)) != cudaSuccess) return cuda_fail(e);
        }
        sel_st = c->cs_sel;
    }
    {   // ---- Eq. 8
        PhaseTimer pt(c, sel_st, XSV_PHASE_SELECT);
        e = xsv_launch_select(c->scores, p.n_mid, k, T_first, (int)p.T_c, c->srcmap, c->dscal, sel_st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (p.side_select) {
        // Eq. 9-11 need the selection only, not the attention output: they follow it into the spare buffer -- the keys
        // on its stream, the values (two short kernels: kept rows move verbatim, the frame's rows are quantised)
        // on a third one, so that neither waits for the other -- on the multiprocessors that the attention CTAs
        // leave one by one, and beside the merge kernel.  The caller's stream waits for both afterwards, so the step
        // ends when all of it has.
        if (c->bits < 16) {
            const LayerView& dv = c->bufs[c->spare].view;
            if ((e = cudaEventRecord(c->ev_picked, c->cs_sel)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamWaitEvent(c->cs_val, c->ev_picked, 0)) != cudaSuccess) return cuda_fail(e);
            {
                PhaseTimer pt(c, c->cs_val, XSV_PHASE_QUANT);
                e = xsv_launch_values(lv, dv, p.V, p.dtype, H, F, T_first + k, T_first, c->srcmap, p.origin0, c->status, c->cs_val);
                if (e != cudaSuccess) return cuda_fail(e);
            }
            if ((e = cudaEventRecord(c->ev_values, c->cs_val)) != cudaSuccess) return cuda_fail(e);
            PhaseTimer pt(c, sel_st, XSV_PHASE_QUANT);
            e = xsv_launch_compress(lv, dv, p.K, p.V, p.dtype, H, F, T_first + k, T_first + k + F, T_first, c->srcmap,
                                    c->dscal, 0, p.origin0, false, c->status, sel_st);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        if ((e = cudaEventRecord(c->ev_selected, c->cs_sel)) != cudaSuccess) return cuda_fail(e);
    }
    return XSV_OK;
}

// ---- Eq. 2 / Eq. 12: attention of one cache's frame over [cache ; frame]
xsv_status launch_attention(const StepPlan& p, cudaStream_t st) {
    xsv_cache* c = p.c;
    const LayerView& lv = c->bufs[p.cur].view;
    cudaError_t e;
    bool tc5 = false;
    {
        PhaseTimer pt(c, st, XSV_PHASE_ATTN);      // the attention kernel proper; the merge of shared tiles follows
        e = cudaErrorNotSupported;
        if (c->attn_impl != XSV_ATTN_MMA)
            e = xsv_launch_attn_tc5(lv, (int)p.T_c, p.Q, p.K, p.V, p.out, p.dtype, p.H, p.F, c->attn_ws, c->status, 0, st);
        tc5 = (e == cudaSuccess);
        if (e == cudaErrorNotSupported) {
            if (c->attn_impl == XSV_ATTN_TC5) return XSV_ERR_ARG;
            e = xsv_launch_attn_mma(lv, (int)p.T_c, p.Q, p.K, p.V, p.out, p.dtype, p.H, p.F, st);
        }
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (tc5) {
        e = xsv_launch_attn_tc5_merge(lv, (int)p.T_c, p.Q, p.K, p.V, p.out, p.dtype, p.H, p.F, c->attn_ws, c->status, 0, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return XSV_OK;
}

// What follows the attention: the join with the cache's own streams (or its deferral), the cache update of a
// step that does not prune, and the bookkeeping.
xsv_status launch_after_attention(const StepPlan& p, cudaStream_t st) {
    xsv_cache* c = p.c;
    const int layer = p.layer, F = p.F, H = p.H, T_first = p.T_first, k = p.k;
    const LayerView& lv = c->bufs[p.cur].view;
    cudaError_t e = cudaSuccess;
    const bool deferred = p.side_select && c->defer_join && c->bits < 16;
    if (deferred) {
        // the caller's stream goes on; it waits for this layer's side-stream work when the layer is stepped again
        // (or in xsv_cache_join)
        if ((e = cudaEventRecord(c->ev_keys_of[layer], c->cs_sel)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventRecord(c->ev_vals_of[layer], c->cs_val)) != cudaSuccess) return cuda_fail(e);
        c->side_pending[layer] = 1;
        c->select_outstanding = true;
    } else {
        if (p.side_select && (e = cudaStreamWaitEvent(st, c->ev_selected, 0)) != cudaSuccess) return cuda_fail(e);
        if (p.side_select && c->bits < 16 && (e = cudaStreamWaitEvent(st, c->ev_values, 0)) != cudaSuccess) return cuda_fail(e);
    }
    if (p.prune) {
        const int n_old_new = T_first + k;
        const int T_new = n_old_new + F;
        const LayerView& dv = c->bufs[c->spare].view;
        {   // ---- Eq. 9-11 on the new order [first ; kept ; current], written to the spare buffer
            PhaseTimer pt(c, st, XSV_PHASE_QUANT);
            if (c->bits == 16) {
                e = xsv_launch_raw_update(lv, dv, p.K, p.V, H, F, n_old_new, T_first, c->srcmap, p.origin0, st);
            } else {
                if (!p.side_select)
                    e = xsv_launch_compress(lv, dv, p.K, p.V, p.dtype, H, F, n_old_new, T_new, T_first, c->srcmap, c->dscal, 0,
                                            p.origin0, true, c->status, st);
            }
            if (e != cudaSuccess) return cuda_fail(e);
        }
        c->buf_of_layer[layer] = c->spare;
        c->spare = p.cur;
        c->len[layer] = T_new;
        c->last_scores_n = p.n_mid;
    } else {
        // append in place: cached tokens keep their slots; the partial tail key
        // group (if any) is rebuilt together with the fresh tokens
        PhaseTimer pt(c, st, XSV_PHASE_QUANT);
        if (c->bits == 16) {
            e = xsv_launch_raw_update(lv, lv, p.K, p.V, H, F, (int)p.T_c, F, nullptr, p.origin0, st);
        } else {
            e = xsv_launch_compress(lv, lv, p.K, p.V, p.dtype, H, F, (int)p.T_c, (int)p.T, F, nullptr, nullptr,
                                    (int)(p.T_c / XSV_G), p.origin0, true, c->status, st);
        }
        if (e != cudaSuccess) return cuda_fail(e);
        c->len[layer] = p.T;
        c->last_scores_n = 0;
    }
    c->frames[layer] = p.t;
    c->tokens_seen[layer] = p.origin0 + F;
    if (p.t == 1) c->F_first[layer] = F;
    return XSV_OK;
}

xsv_status step_impl(xsv_cache* c, int layer, const void* Q, const void* K, const void* V, int n_tokens,
                     xsv_dtype dtype, void* out, void* stream, bool append_only) {
    StepPlan p{};
    xsv_status s = plan_step(c, layer, Q, K, V, n_tokens, dtype, out, append_only, p);
    if (s != XSV_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if ((s = launch_before_attention(p, st)) != XSV_OK) return s;
    if (!append_only && (s = launch_attention(p, st)) != XSV_OK) return s;
    return launch_after_attention(p, st);
}

}  // namespace

extern "C" {

xsv_status xsv_step(xsv_cache* c, int layer, const void* Q, const void* K, const void* V, int n_tokens,
                    xsv_dtype dtype, void* out, void* stream) {
    return step_impl(c, layer, Q, K, V, n_tokens, dtype, out, stream, false);
}

xsv_status xsv_cache_append(xsv_cache* c, int layer, const void* K, const void* V, int n_tokens, xsv_dtype dtype,
                            void* stream) {
    // Q and out are not touched on this path; K stands in for them in the argument checks
    return step_impl(c, layer, K, K, V, n_tokens, dtype, c, stream, true);
}

xsv_status xsv_step_batch(xsv_cache* const* caches, int n, int layer, const void* const* Q, const void* const* K,
                          const void* const* V, const int* n_tokens, xsv_dtype dtype, void* const* out, void* stream) {
    if (!caches || !Q || !K || !V || !n_tokens || !out || n <= 0 || n > XSV_MAX_BATCH) return XSV_ERR_ARG;
    StepPlan plans[XSV_MAX_BATCH];
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j < i; ++j)
            if (caches[i] == caches[j]) return XSV_ERR_ARG;
        const xsv_status s = plan_step(caches[i], layer, Q[i], K[i], V[i], n_tokens[i], dtype, out[i], false, plans[i]);
        if (s != XSV_OK) return s;                      // nothing has been launched: every cache is unchanged
        const xsv_cache* a = caches[0];
        const xsv_cache* b = caches[i];
        if (b->device != a->device || b->H != a->H || b->bits != a->bits) return XSV_ERR_SHAPE;
        if (b->attn_impl == XSV_ATTN_MMA || !b->attn_ws) return XSV_ERR_ARG;
        plans[i].scores_on_side = n > 1;
    }
    cudaStream_t st = (cudaStream_t)stream;
    xsv_status s;
    for (int i = 0; i < n; ++i)
        if ((s = launch_before_attention(plans[i], st)) != XSV_OK) return s;
    {   // one attention launch and one merge launch for all streams
        LayerView lvs[XSV_MAX_BATCH];
        int T_cs[XSV_MAX_BATCH], Fs[XSV_MAX_BATCH];
        const void *Qs[XSV_MAX_BATCH], *Ks[XSV_MAX_BATCH], *Vs[XSV_MAX_BATCH];
        void* outs[XSV_MAX_BATCH];
        int* statuses[XSV_MAX_BATCH];
        for (int i = 0; i < n; ++i) {
            lvs[i] = caches[i]->bufs[plans[i].cur].view;
            T_cs[i] = (int)plans[i].T_c; Fs[i] = plans[i].F;
            Qs[i] = Q[i]; Ks[i] = K[i]; Vs[i] = V[i]; outs[i] = out[i];
            statuses[i] = caches[i]->status;
        }
        PhaseTimer pt(caches[0], st, XSV_PHASE_ATTN);
        cudaError_t e = xsv_launch_attn_tc5_batch(n, lvs, T_cs, Qs, Ks, Vs, outs, (int)dtype, caches[0]->H, Fs,
                                                  caches[0]->attn_ws, statuses, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    for (int i = 0; i < n; ++i)
        if ((s = launch_after_attention(plans[i], st)) != XSV_OK) return s;
    return XSV_OK;
}

xsv_status xsv_cache_set_deferred_join(xsv_cache* c, int on) {
    if (!c) return XSV_ERR_ARG;
    c->defer_join = on != 0;
    return XSV_OK;
}

xsv_status xsv_cache_join(xsv_cache* c, void* stream) {
    if (!c) return XSV_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    for (size_t l = 0; l < c->side_pending.size(); ++l) {
        if (!c->side_pending[l]) continue;
        if ((e = cudaStreamWaitEvent(st, c->ev_keys_of[l], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(st, c->ev_vals_of[l], 0)) != cudaSuccess) return cuda_fail(e);
        c->side_pending[l] = 0;
    }
    if (c->select_outstanding) {
        if ((e = cudaStreamWaitEvent(st, c->ev_picked, 0)) != cudaSuccess) return cuda_fail(e);
        c->select_outstanding = false;
    }
    return XSV_OK;
}

xsv_status xsv_step_host(xsv_cache* c, int layer, const void* Qh, const void* Kh, const void* Vh, int n_tokens,
                         xsv_dtype dtype, void* out_h, void* stream) {
    if (!c || !Qh || !Kh || !Vh || !out_h || n_tokens <= 0) return XSV_ERR_ARG;
    if (c->F_max != 0 && n_tokens > c->F_max) return XSV_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaSuccess;
    if (!c->stage) {
        // First call: the staging slots (sized for the largest frame), two copy streams and their events.  This is the
        // only call of the host path that allocates; make it before the frame loop.
        const int F_stage = c->F_max != 0 ? c->F_max : n_tokens;
        const size_t nb_max = (size_t)c->H * F_stage * c->d * 2;
        cudaSetDevice(c->device);
        if (cudaMalloc(&c->stage, 8 * nb_max) != cudaSuccess) { cudaGetLastError(); c->stage = nullptr; return XSV_ERR_OOM; }
        c->stage_bytes = 8 * nb_max;
        c->bytes += c->stage_bytes;
        if ((e = cudaStreamCreateWithFlags(&c->cs_in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamCreateWithFlags(&c->cs_out, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        for (int i = 0; i < 2; ++i) {
            if ((e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        }
    }
    const size_t nb = (size_t)c->H * n_tokens * c->d * 2;          // this frame's bytes per tensor
    const size_t slot_bytes = c->stage_bytes / 2, part = slot_bytes / 4;
    if (nb > part) return XSV_ERR_SHAPE;
    // Two staging slots alternate.  The inputs of this call are copied on a stream of their own, as soon as the
    // step that last used the slot has finished, so the copy overlaps the previous call's kernels.
    const int slot = (int)(c->host_calls & 1ull);
    uint8_t* s = (uint8_t*)c->stage + (size_t)slot * slot_bytes;
    if (c->slot_used[slot] && (e = cudaStreamWaitEvent(c->cs_in, c->ev_done[slot], 0)) != cudaSuccess) return cuda_fail(e);
    if (c->slot_used[slot] && c->slot_deferred[slot]) {
        // Deferred join: the side-stream kernels of the step that read this slot may still be reading the staged K and
        // V.  Their events are waited for whatever the caller's stream has joined since (a join makes only that stream
        // wait, not this copy stream).
        if ((e = cudaStreamWaitEvent(c->cs_in, c->ev_keys_of[c->slot_layer[slot]], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(c->cs_in, c->ev_vals_of[c->slot_layer[slot]], 0)) != cudaSuccess) return cuda_fail(e);
    }
    if ((e = cudaMemcpyAsync(s, Qh, nb, cudaMemcpyHostToDevice, c->cs_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(s + part, Kh, nb, cudaMemcpyHostToDevice, c->cs_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(s + 2 * part, Vh, nb, cudaMemcpyHostToDevice, c->cs_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaEventRecord(c->ev_in[slot], c->cs_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(st, c->ev_in[slot], 0)) != cudaSuccess) return cuda_fail(e);
    if (c->out_pending[slot]) {   // the slot's previous result must have left before the step overwrites it
        if ((e = cudaStreamWaitEvent(st, c->ev_out[slot], 0)) != cudaSuccess) return cuda_fail(e);
        c->out_pending[slot] = false;
    }
    xsv_status r = xsv_step(c, layer, s, s + part, s + 2 * part, n_tokens, dtype, s + 3 * part, stream);
    if (r != XSV_OK) return r;
    ++c->host_calls;
    c->slot_used[slot] = true;
    c->slot_layer[slot] = layer;
    c->slot_deferred[slot] = !c->side_pending.empty() && c->side_pending[layer] != 0;
    if ((e = cudaEventRecord(c->ev_done[slot], st)) != cudaSuccess) return cuda_fail(e);
    if (!c->defer_output) {
        if ((e = cudaMemcpyAsync(out_h, s + 3 * part, nb, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e);
    } else {
        if ((e = cudaStreamWaitEvent(c->cs_out, c->ev_done[slot], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaMemcpyAsync(out_h, s + 3 * part, nb, cudaMemcpyDeviceToHost, c->cs_out)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventRecord(c->ev_out[slot], c->cs_out)) != cudaSuccess) return cuda_fail(e);
        c->out_pending[slot] = true;
    }
    return XSV_OK;
}

xsv_status xsv_cache_set_host_pipelining(xsv_cache* c, int defer_output) {
    if (!c) return XSV_ERR_ARG;
    if (c->out_pending[0] || c->out_pending[1]) return XSV_ERR_ORDER;   // flush first
    c->defer_output = defer_output != 0;
    return XSV_OK;
}

xsv_status xsv_cache_host_flush(xsv_cache* c, void* stream) {
    if (!c) return XSV_ERR_ARG;
    for (int i = 0; i < 2; ++i) {
        if (!c->out_pending[i]) continue;
        const cudaError_t e = cudaStreamWaitEvent((cudaStream_t)stream, c->ev_out[i], 0);
        if (e != cudaSuccess) return cuda_fail(e);
        c->out_pending[i] = false;
    }
    return XSV_OK;
}

xsv_status xsv_importance_scores(const void* Q, const void* keys, int heads, int n_tokens, long long n_keys,
                                 xsv_dtype dtype, int n_special, int pool_group, float* scores, void* stream) {
    if (!Q || !keys || !scores || heads <= 0 || n_tokens <= 0 || n_keys <= 0 || n_keys > (1LL << 30)) return XSV_ERR_ARG;
    if (dtype != XSV_F16 && dtype != XSV_BF16) return XSV_ERR_ARG;
    if (n_special < 0 || n_special > n_tokens || pool_group <= 0) return XSV_ERR_ARG;
    if (((uintptr_t)Q | (uintptr_t)keys) & 15) return XSV_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    float* qpart = nullptr;
    if (cudaMallocAsync((void**)&qpart, (size_t)heads * XSV_QCHUNKS * 64 * sizeof(float), st) != cudaSuccess) {
        cudaGetLastError();
        return XSV_ERR_OOM;
    }
    LayerView lv{};
    lv.kcodes = (uint8_t*)const_cast<void*>(keys);
    lv.cap = n_keys;
    lv.rowb = XSV_D * 2;
    lv.bits = 16;
    const int n_pooled = n_special + (n_tokens - n_special + pool_group - 1) / pool_group;
    const float qnorm = 1.0f / ((float)heads * (float)n_pooled);
    cudaError_t e = xsv_launch_qtilde(Q, (int)dtype, heads, n_tokens, n_special, pool_group, qpart, st);
    if (e == cudaSuccess) e = xsv_launch_score_raw(lv, (int)dtype, heads, 0, (int)n_keys, qpart, qnorm, scores, st);
    cudaFreeAsync(qpart, st);
    return e == cudaSuccess ? XSV_OK : cuda_fail(e);
}

int xsv_plan_batch_groups(int n, const int* cache_tokens, const int* frame_tokens, int heads, int multiprocessors) {
    if (!cache_tokens || !frame_tokens || heads < 1) return -1;
    for (int i = 0; i < n && i < XSV_MAX_BATCH; ++i)
        if (cache_tokens[i] < 0 || frame_tokens[i] < 1) return -1;
    return xsv_attn_batch_group_size(n, cache_tokens, frame_tokens, heads, multiprocessors);
}

int xsv_selftest_device_table(void) {
    // host-only: the per-device slots are independent, survive other slots' updates, and ignore devices
    // beyond the table (which then are configured on every launch instead of once)
    XsvPerDeviceInt t;
    for (int d = 0; d < XSV_MAX_DEVICES; ++d) if (t.get(d) != 0) return 1;
    t.set(0, 5);
    if (t.get(0) != 5 || t.get(1) != 0) return 2;
    t.set(1, 9);
    t.set(XSV_MAX_DEVICES - 1, 7);
    if (t.get(0) != 5 || t.get(1) != 9 || t.get(XSV_MAX_DEVICES - 1) != 7 || t.get(2) != 0) return 3;
    t.set(XSV_MAX_DEVICES, 11);
    t.set(-1, 13);
    if (t.get(XSV_MAX_DEVICES) != 0 || t.get(-1) != 0 || t.get(0) != 5 || t.get(XSV_MAX_DEVICES - 1) != 7) return 4;
    return 0;
}

xsv_status xsv_selftest_bounded_wait(void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    int* d = nullptr;
    if (cudaMalloc((void**)&d, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return XSV_ERR_OOM; }
    int w = 0;
    cudaError_t e = cudaMemsetAsync(d, 0, sizeof(int), st);
    if (e == cudaSuccess) e = xsv_launch_wait_selftest(d, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&w, d, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(d);
    if (e != cudaSuccess) return cuda_fail(e);
    return (w & XSV_DEV_TIMEOUT) ? XSV_ERR_TIMEOUT : XSV_OK;
}

size_t xsv_cache_bytes(const xsv_cache* c) { return c ? c->bytes : 0; }

size_t xsv_cache_layer_kv_bytes(const xsv_cache* c, int layer) {
    if (!c || layer < 0 || layer >= c->layers) return 0;
    const size_t T = (size_t)c->len[layer], H = c->H, d = c->d;
    if (c->bits == 16) return 2 * H * T * d * 2;
    const size_t groups = (T + XSV_G - 1) / XSV_G;
    return 2 * H * T * d * c->bits / 8 + H * groups * d * 8 + H * T * 8;
}

void xsv_cache_destroy(xsv_cache* c) {
    if (!c) return;
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    for (auto& b : c->bufs) if (b.slab) cudaFree(b.slab);
    if (c->scratch_slab) cudaFree(c->scratch_slab);
    if (c->stage) cudaFree(c->stage);
    for (int i = 0; i < 2; ++i) {
        if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
        if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
        if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
    }
    for (cudaEvent_t ev : c->ev_keys_of) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : c->ev_vals_of) if (ev) cudaEventDestroy(ev);
    if (c->cs_sel) cudaStreamDestroy(c->cs_sel);
    if (c->cs_val) cudaStreamDestroy(c->cs_val);
    if (c->ev_picked) cudaEventDestroy(c->ev_picked);
    if (c->ev_values) cudaEventDestroy(c->ev_values);
    if (c->ev_scored) cudaEventDestroy(c->ev_scored);
    if (c->ev_selected) cudaEventDestroy(c->ev_selected);
    if (c->cs_in) cudaStreamDestroy(c->cs_in);
    if (c->cs_out) cudaStreamDestroy(c->cs_out);
    for (auto& p : c->pending) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
    for (auto e : c->free_events) cudaEventDestroy(e);
    delete c;
}

long long xsv_cache_len(const xsv_cache* c, int layer) {
    if (!c || layer < 0 || layer >= c->layers) return -1;
    return c->len[layer];
}

long long xsv_cache_frames(const xsv_cache* c, int layer) {
    if (!c || layer < 0 || layer >= c->layers) return -1;
    return c->frames[layer];
}

xsv_status xsv_cache_export_layer(xsv_cache* c, int layer, unsigned char* k_codes, float* k_scale, float* k_zero,
                                  unsigned char* v_codes, float* v_scale, float* v_zero, long long* origin,
                                  unsigned short* k_raw, unsigned short* v_raw, void* stream) {
    if (!c || layer < 0 || layer >= c->layers) return XSV_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaStreamSynchronize(st) != cudaSuccess || sync_side_streams(c) != cudaSuccess) return XSV_ERR_CUDA;
    const long long T = c->len[layer];
    if (T == 0 || !c->allocated) return XSV_OK;
    const LayerView& lv = c->bufs[c->buf_of_layer[layer]].view;
    const int H = c->H, d = c->d, rowb = lv.rowb, bits = c->bits;
    const long long groups = (T + XSV_G - 1) / XSV_G;
    std::vector<uint8_t> tmp((size_t)T * rowb);
    for (int pass = 0; pass < 2; ++pass) {
        const uint8_t* dev = pass == 0 ? lv.kcodes : lv.vcodes;
        unsigned char* codes = pass == 0 ? k_codes : v_codes;
        unsigned short* raw = pass == 0 ? k_raw : v_raw;
        if ((bits < 16 && !codes) || (bits == 16 && !raw)) continue;
        for (int h = 0; h < H; ++h) {
            if (cudaMemcpy(tmp.data(), dev + (size_t)h * lv.cap * rowb, (size_t)T * rowb, cudaMemcpyDeviceToHost) != cudaSuccess)
                return XSV_ERR_CUDA;
            if (bits == 16) {
                memcpy(raw + (size_t)h * T * d, tmp.data(), (size_t)T * rowb);
            } else {
                const unsigned mask = (1u << bits) - 1u;
                for (long long p = 0; p < T; ++p)
                    for (int ch = 0; ch < d; ++ch) {
                        const int bit = ch * bits;
                        codes[((size_t)h * T + p) * d + ch] = (tmp[(size_t)p * rowb + bit / 8] >> (bit % 8)) & mask;
                    }
            }
        }
    }
    if (bits < 16) {
        for (int h = 0; h < H; ++h) {
            if (k_scale && cudaMemcpy(k_scale + (size_t)h * groups * 64, lv.kscale + (size_t)h * lv.capg * 64, (size_t)groups * 64 * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
            if (k_zero && cudaMemcpy(k_zero + (size_t)h * groups * 64, lv.kzero + (size_t)h * lv.capg * 64, (size_t)groups * 64 * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
            if (v_scale && cudaMemcpy(v_scale + (size_t)h * T, lv.vscale + (size_t)h * lv.cap, (size_t)T * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
            if (v_zero && cudaMemcpy(v_zero + (size_t)h * T, lv.vzero + (size_t)h * lv.cap, (size_t)T * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
        }
    }
    if (origin && cudaMemcpy(origin, lv.origin, (size_t)T * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
    return XSV_OK;
}

xsv_status xsv_cache_import_layer(xsv_cache* c, int layer, long long n_cached, long long frames_done, int frame_tokens,
                                  xsv_dtype dtype, const unsigned char* k_codes, const float* k_scale, const float* k_zero,
                                  const unsigned char* v_codes, const float* v_scale, const float* v_zero,
                                  const long long* origin, const unsigned short* k_raw, const unsigned short* v_raw,
                                  void* stream) {
    if (!c || layer < 0 || layer >= c->layers || n_cached < 0 || frames_done < 0 || frame_tokens <= 0 || !origin) return XSV_ERR_ARG;
    if (dtype != XSV_F16 && dtype != XSV_BF16) return XSV_ERR_ARG;
    if (c->bits == 16 ? (!k_raw || !v_raw) : (!k_codes || !k_scale || !k_zero || !v_codes || !v_scale || !v_zero)) return XSV_ERR_ARG;
    if (c->F_max != 0 && frame_tokens > c->F_max) return XSV_ERR_SHAPE;
    if (c->dtype >= 0 && (int)dtype != c->dtype) return XSV_ERR_SHAPE;
    if (c->n_special > frame_tokens) return XSV_ERR_ARG;
    if (n_cached > 0 && n_cached < frame_tokens) return XSV_ERR_ARG;      // the first frame is always in the cache
    if (c->bits < 16) {
        // every code is checked before anything is written, so that an error leaves the cache unchanged
        const unsigned mask = (1u << c->bits) - 1u;
        const size_t n = (size_t)c->H * (size_t)n_cached * c->d;
        for (size_t i = 0; i < n; ++i)
            if (k_codes[i] > mask || v_codes[i] > mask) return XSV_ERR_ARG;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (!c->allocated) {
        c->F_max = frame_tokens;
        cudaSetDevice(c->device);
        const xsv_status s = allocate(c);
        if (s != XSV_OK) { c->F_max = 0; return s; }
    }
    if (n_cached > c->cap) return XSV_ERR_CAPACITY;
    if (cudaStreamSynchronize(st) != cudaSuccess || sync_side_streams(c) != cudaSuccess) return XSV_ERR_CUDA;
    const LayerView& lv = c->bufs[c->buf_of_layer[layer]].view;
    const int H = c->H, d = c->d, rowb = lv.rowb, bits = c->bits;
    const long long T = n_cached, groups = (T + XSV_G - 1) / XSV_G;
    cudaError_t e = cudaSuccess;
    if (T > 0) {
        std::vector<uint8_t> tmp((size_t)T * rowb);
        for (int pass = 0; pass < 2 && e == cudaSuccess; ++pass) {
            uint8_t* dev = pass == 0 ? lv.kcodes : lv.vcodes;
            const unsigned char* codes = pass == 0 ? k_codes : v_codes;
            const unsigned short* raw = pass == 0 ? k_raw : v_raw;
            for (int h = 0; h < H && e == cudaSuccess; ++h) {
                if (bits == 16) {
                    memcpy(tmp.data(), raw + (size_t)h * T * d, (size_t)T * rowb);
                } else {
                    memset(tmp.data(), 0, tmp.size());
                    const unsigned mask = (1u << bits) - 1u;
                    for (long long p = 0; p < T; ++p)
                        for (int ch = 0; ch < d; ++ch) {
                            const unsigned code = codes[((size_t)h * T + p) * d + ch] & mask;   // validated above
                            const int bit = ch * bits;
                            tmp[(size_t)p * rowb + bit / 8] |= (uint8_t)(code << (bit % 8));
                        }
                }
                e = cudaMemcpy(dev + (size_t)h * lv.cap * rowb, tmp.data(), (size_t)T * rowb, cudaMemcpyHostToDevice);
            }
        }
        if (bits < 16) {
            for (int h = 0; h < H && e == cudaSuccess; ++h) {
                e = cudaMemcpy(lv.kscale + (size_t)h * lv.capg * 64, k_scale + (size_t)h * groups * 64, (size_t)groups * 64 * 4, cudaMemcpyHostToDevice);
                if (e == cudaSuccess) e = cudaMemcpy(lv.kzero + (size_t)h * lv.capg * 64, k_zero + (size_t)h * groups * 64, (size_t)groups * 64 * 4, cudaMemcpyHostToDevice);
                if (e == cudaSuccess) e = cudaMemcpy(lv.vscale + (size_t)h * lv.cap, v_scale + (size_t)h * T, (size_t)T * 4, cudaMemcpyHostToDevice);
                if (e == cudaSuccess) e = cudaMemcpy(lv.vzero + (size_t)h * lv.cap, v_zero + (size_t)h * T, (size_t)T * 4, cudaMemcpyHostToDevice);
            }
        }
        if (e == cudaSuccess) e = cudaMemcpy(lv.origin, origin, (size_t)T * 8, cudaMemcpyHostToDevice);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    c->len[layer] = T;
    c->frames[layer] = frames_done;
    c->F_first[layer] = frames_done > 0 ? frame_tokens : 0;
    c->tokens_seen[layer] = T > 0 ? origin[T - 1] + 1 : 0;      // the last token of the last frame is always kept
    c->dtype = (int)dtype;
    c->stepped = true;
    return XSV_OK;
}

xsv_status xsv_last_scores(xsv_cache* c, float* scores_host, long long cap, long long* n, void* stream) {
    if (!c || !n) return XSV_ERR_ARG;
    *n = c->last_scores_n;
    if (c->last_scores_n == 0) return XSV_OK;
    if (!scores_host || cap < c->last_scores_n) return XSV_ERR_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess || sync_side_streams(c) != cudaSuccess) return XSV_ERR_CUDA;
    if (cudaMemcpy(scores_host, c->scores, (size_t)c->last_scores_n * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
    return XSV_OK;
}

xsv_status xsv_cache_status(xsv_cache* c, void* stream) {
    if (!c) return XSV_ERR_ARG;
    if (!c->allocated) return XSV_OK;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess || sync_side_streams(c) != cudaSuccess) return XSV_ERR_CUDA;
    int w = 0;
    if (cudaMemcpy(&w, c->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return XSV_ERR_CUDA;
    if (w & XSV_DEV_TIMEOUT) return XSV_ERR_TIMEOUT;
    if (w & XSV_DEV_RANGE) return XSV_ERR_RANGE;
    return XSV_OK;
}

int xsv_cache_status_word(xsv_cache* c, void* stream) {
    if (!c) return -1;
    if (!c->allocated) return 0;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess || sync_side_streams(c) != cudaSuccess) return -1;
    int w = 0;
    if (cudaMemcpy(&w, c->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    return w;
}

xsv_status xsv_cache_set_profiling(xsv_cache* c, int on) {
    if (!c) return XSV_ERR_ARG;
    if (on < 0 || on > 4) return XSV_ERR_ARG;
    if (on && c->free_events.empty() && c->pending.empty()) {
        // a pool of timing events, so that the steps that follow create none
        cudaSetDevice(c->device);
        for (int i = 0; i < 64 + 16 * c->layers; ++i) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); break; }
            c->free_events.push_back(e);
        }
    }
    c->profiling = on;
    return XSV_OK;
}

xsv_status xsv_cache_profile_read(xsv_cache* c, double ms[XSV_PHASE_COUNT], long long launches[XSV_PHASE_COUNT], int reset) {
    if (!c) return XSV_ERR_ARG;
    for (auto& p : c->pending) {
        if (cudaEventSynchronize(p.b) != cudaSuccess) return XSV_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, p.a, p.b) != cudaSuccess) return XSV_ERR_CUDA;
        c->prof_ms[p.phase] += t;
        c->free_events.push_back(p.a);
        c->free_events.push_back(p.b);
    }
    c->pending.clear();
    for (int i = 0; i < XSV_PHASE_COUNT; ++i) {
        if (ms) ms[i] = c->prof_ms[i];
        if (launches) launches[i] = c->prof_launches[i];
        if (reset) { c->prof_ms[i] = 0; c->prof_launches[i] = 0; }
    }
    return XSV_OK;
}

}  // extern "C"
