// Host side of the C ABI declared in include/kvs.h: the layer -> slot indirection
// table, slot lengths, capacity and state checks, byte accounting, and the launches.
#include "../../include/kvs.h"

#include "kvs_kernels.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

namespace {

constexpr size_t kAlign = 256;
constexpr int kRowStrideQuantum = 128;
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

// ---------------------------------------------------------------------------------------
// Scratch of kvs_decode_attention_static: attention without any caller- or library-allocated
// scratch memory.
//
// The split-K partial results and the device status word of that one entry point live in a
// fixed array that is part of the loaded library image.  Every GPU that loads the library
// carries these kStaticScratchBytes until the process exits, and every call, from every
// context, uses the same bytes.
// ---------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = 2u << 20;  // 2 MiB
constexpr size_t kStaticStatusBytes = 256;        // first 256 bytes: device status word
// then the per-unit hand-over flags, at a fixed place and of a fixed size, so that no call's partial results
// (which follow) ever lie where another call, of another size, keeps its flags: they are zero when the library
// is loaded and every launch leaves them zero
constexpr size_t kStaticFlagBytes = 32768;        // 8192 (sequence, kv-head) units
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

// In host code `g_static_scratch` is only a handle for the symbol, not an address the GPU can
// use, so the device address is looked up once per device, with that device current, as part of
// the per-device set-up that kvs_bind_memory runs (see init_device_once).  The look-up is also
// what makes the driver load this file's module and reserve the array on that GPU, so it happens
// where allocating is still allowed and no stream is being captured; the entry point itself then
// only reads the cached address.
cudaError_t g_static_err[64];
unsigned char* g_static_ptr[64];

cudaError_t resolve_static_scratch(int device) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    g_static_err[device] = e;
    g_static_ptr[device] = e == cudaSuccess ? static_cast<unsigned char*>(p) : nullptr;
    return e;
}

}  // namespace

struct kvs_ctx {
    kvs_config cfg;
    int G = 1;
    int elem = 2;
    int row_bytes = 0;
    int row_stride = 0;        // rows between units of a plane
    size_t plane_bytes = 0;
    float scale = 0.f;

    std::vector<int32_t> share_map, root, slot_of_layer;
    int n_slots = 0;
    std::vector<int32_t> slot_len;
    int cur_batch = 0;         // batch the cached rows were appended for (0 = none yet)

    // Ragged slots: after kvs_evict the units of a slot differ in length; the lengths then live in
    // a device array (one per slot, in the workspace) with a host mirror.
    std::vector<char> ragged;                       // per slot
    std::vector<std::vector<int32_t>> unit_len_host;  // per slot, [max_batch * Hkv]

    bool bound = false;
    char* pool = nullptr;
    char* ws = nullptr;
    int sm_count = 148;
    long long l2_bytes = 64ll << 20;

    // workspace carve-up (byte offsets)
    size_t off_status = 0, off_part_o = 0, off_part_ml = 0, off_stage_q = 0, off_stage_k = 0, off_stage_v = 0,
           off_stage_out = 0, off_unit_len = 0, off_counts = 0, off_search = 0, off_replay = 0, off_flags = 0, ws_bytes = 0,
           search_bytes = 0;

    alignas(64) unsigned char tensor_map[128];  // TMA view of the pool (bf16 storage only), 64-row boxes
    alignas(64) unsigned char tensor_map_tail[128];   // the same view with 16-row boxes (partly filled tiles)
    bool have_tensor_map = false;

    // Launch bookkeeping for early-start (programmatic) launches.  Every kernel of this context
    // gets a sequence number.  A split-K kernel lets its successor start only after its own
    // wait, so when any later kernel runs, everything before the latest split-K kernel is
    // complete; appends newer than that may still be in flight.
    uint64_t seq = 0;
    uint64_t last_splitk_seq = 0;
    std::vector<uint64_t> app_seq_latest, app_seq_prev;   // per slot, 0 = none
    std::vector<int32_t> app_start_latest;                // first row the latest append wrote

    // kvs_step_host: second stream and events that overlap the host copies with the layers
    static constexpr int kChunks = 8;
    bool copy_ready = false;
    cudaStream_t copy_stream = nullptr, out_stream = nullptr;
    cudaEvent_t ev_in[kChunks] = {}, ev_done[kChunks] = {}, ev_start = nullptr;
    // kvs_layer_distances: a second stream on which the pair sums of one slab run beside the averaging of the next

    int opt_max_ctas = 0;
    int opt_kernel = 0;
    int opt_pdl = 1;
    int opt_host_chunks = 4;
    // tracing build: where the next attention launch stamps its timeline (kvs_trace_begin / kvs_trace_end)
    unsigned long long* trace_buf = nullptr;
    int trace_capacity = 0, trace_launch = 0;
    int opt_wait_us = 2000000;   // limit of the waits inside the split-K kernels, microseconds
    long long stall_tile = -1;   // kvs_selftest_stalled_copy: tile whose copies the next attention launch withholds
    int opt_finish = 1;   // units of at most two pieces are finished by the split-K kernel itself (no combine launch)
    int opt_replay = 0;   // launches carry the device-side growth counter (for CUDA-graph replay)
    // The split-K kernels read the growth counter before their wait.  That is safe because the
    // first launch after anything wrote the counter never starts early (full dependency): it and
    // everything after it then begin with the write complete.
    bool counter_written = false;
    kvs::DecodePlan last_plan{};
    kvs_stats_t stats{};
};

namespace {

void resolve_map(kvs_ctx* c) {
    const int L = c->cfg.n_layers;
    c->root.assign(L, 0);
    c->slot_of_layer.assign(L, -1);
    int n = 0;
    for (int l = 0; l < L; ++l) {
        if (c->share_map[l] == l) {
            c->root[l] = l;
            c->slot_of_layer[l] = n++;
        } else {
            // sources precede targets, so the source is already resolved
            c->root[l] = c->root[c->share_map[l]];
            c->slot_of_layer[l] = c->slot_of_layer[c->root[l]];
        }
    }
    c->n_slots = n;
    c->slot_len.assign(n, 0);
    c->cur_batch = 0;
    c->app_seq_latest.assign(n, 0);
    c->app_seq_prev.assign(n, 0);
    c->app_start_latest.assign(n, 0);
    c->ragged.assign(n, 0);
    c->unit_len_host.assign(n, std::vector<int32_t>());
}

// Whether the next launch may start early; consumes the "counter was just written" mark.
bool take_early_start(kvs_ctx* c) {
    const bool early = c->opt_pdl != 0 && !c->counter_written;
    c->counter_written = false;
    return early;
}

const int* replay_counter(const kvs_ctx* c) {
    return c->opt_replay ? reinterpret_cast<const int*>(c->ws + c->off_replay) : nullptr;
}

int* unit_len_dev(const kvs_ctx* c, int slot) {
    return reinterpret_cast<int*>(c->ws + c->off_unit_len) + (size_t)slot * c->cfg.max_batch * c->cfg.n_kv_heads;
}

// Rows of `slot` that no kernel possibly still in flight writes (see kvs_ctx::seq).
int safe_rows_of(const kvs_ctx* c, int slot) {
    const uint64_t complete_upto = c->last_splitk_seq ? c->last_splitk_seq - 1 : 0;
    if (c->app_seq_latest[slot] <= complete_upto) return c->slot_len[slot];
    if (c->app_seq_prev[slot] <= complete_upto) return c->app_start_latest[slot];
    return 0;
}

void layout_workspace(kvs_ctx* c) {
    const kvs_config& f = c->cfg;
    const size_t units = (size_t)f.max_batch * f.n_kv_heads;
    const size_t pieces = units + kvs::kMaxCtas;
    size_t off = 0;
    c->off_status = off;
    off += kAlign;
    c->off_part_o = off;
    off = align_up(off + pieces * c->G * f.head_dim * sizeof(float), kAlign);
    c->off_part_ml = off;
    off = align_up(off + pieces * c->G * 2 * sizeof(float), kAlign);
    const size_t L = f.n_layers;
    c->off_stage_q = off;
    off = align_up(off + L * f.max_batch * f.n_q_heads * f.head_dim * c->elem, kAlign);
    c->off_stage_k = off;
    off = align_up(off + L * f.max_batch * f.n_kv_heads * f.head_dim * c->elem, kAlign);
    c->off_stage_v = off;
    off = align_up(off + L * f.max_batch * f.n_kv_heads * f.head_dim * c->elem, kAlign);
    c->off_stage_out = off;
    off = align_up(off + L * f.max_batch * f.n_q_heads * f.head_dim * sizeof(float), kAlign);
    c->off_unit_len = off;      // per slot (at most one per layer): int32 [max_batch * Hkv]
    off = align_up(off + L * units * sizeof(int32_t), kAlign);
    c->off_counts = off;        // staging for the kept-row counts of one kvs_evict call
    off = align_up(off + units * sizeof(int32_t), kAlign);
    c->off_replay = off;        // one int: rows every slot has grown by since a recorded launch
    off += kAlign;
    c->off_flags = off;         // one int per unit: "second piece written" (zero between launches)
    off = align_up(off + units * sizeof(int32_t), kAlign);
    c->off_search = off;        // per-block partial sums of the strategy-search reductions
    {
        // at most one slot per layer, at most max_seq rows: enough for every strategy and length
        const size_t need = std::max(kvs::distance_scratch_bytes(f.n_layers <= kvs::kMaxLayersSearch ? f.n_layers : 4,
                                                                 2LL * f.n_kv_heads * f.max_seq * f.head_dim),
                                     (size_t)kvs::kCosineMaxBlocks * 3 * sizeof(double));
        c->search_bytes = need;
        off = align_up(off + need, kAlign);
    }
    c->ws_bytes = off;
}

std::once_flag g_init_flag[64];
cudaError_t g_init_err[64];

cudaError_t init_device_once(int device) {
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    std::call_once(g_init_flag[device], [device]() {
        g_init_err[device] = kvs::init_kernels();
        if (g_init_err[device] == cudaSuccess) g_init_err[device] = kvs::init_mma_kernels();
        if (g_init_err[device] == cudaSuccess) g_init_err[device] = kvs::init_prefill_kernels();
        if (g_init_err[device] == cudaSuccess) g_init_err[device] = resolve_static_scratch(device);
    });
    return g_init_err[device];
}

// RAII: make ctx's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard() {
        if (ok && prev != target) cudaSetDevice(prev);
    }
    int target = -1;
};

kvs_status check_append(kvs_ctx* c, int layer, const void* k, const void* v, int batch, int n_new, bool* sharing) {
    if (!c) return KVS_ERR_INVALID_ARG;
    if (!c->bound) return KVS_ERR_STATE;
    if (layer < 0 || layer >= c->cfg.n_layers) return KVS_ERR_INVALID_ARG;
    if (batch < 1 || batch > c->cfg.max_batch || n_new < 1) return KVS_ERR_INVALID_ARG;
    *sharing = c->share_map[layer] != layer;
    if (*sharing) return KVS_OK;
    if (!k || !v) return KVS_ERR_INVALID_ARG;
    if (((uintptr_t)k % 16) != 0 || ((uintptr_t)v % 16) != 0) return KVS_ERR_INVALID_ARG;   // 16-byte vector loads
    if (c->cur_batch != 0 && batch != c->cur_batch) return KVS_ERR_INVALID_ARG;
    const int slot = c->slot_of_layer[layer];
    if ((long long)c->slot_len[slot] + n_new > c->cfg.max_seq) return KVS_ERR_CAPACITY;
    return KVS_OK;
}

kvs_status check_attention(kvs_ctx* c, int layer, const void* q, const void* out, int batch) {
    if (!c) return KVS_ERR_INVALID_ARG;
    if (!c->bound) return KVS_ERR_STATE;
    if (layer < 0 || layer >= c->cfg.n_layers || !q || !out) return KVS_ERR_INVALID_ARG;
    if (((uintptr_t)q % 16) != 0 || ((uintptr_t)out % 4) != 0) return KVS_ERR_INVALID_ARG;   // q is fetched by bulk copies
    if (batch < 1 || batch > c->cfg.max_batch) return KVS_ERR_INVALID_ARG;
    const int slot = c->slot_of_layer[layer];
    if (c->slot_len[slot] == 0) return KVS_ERR_STATE;
    if (batch > c->cur_batch) return KVS_ERR_INVALID_ARG;
    return KVS_OK;
}

kvs_status do_append(kvs_ctx* c, int layer, const void* k, const void* v, int batch, int n_new, cudaStream_t st) {
    const int slot = c->slot_of_layer[layer];
    char* kp = c->pool + (size_t)(2 * slot) * c->plane_bytes;
    char* vp = kp + c->plane_bytes;
    const bool rag = c->ragged[slot] != 0;
    if (kvs::launch_append(k, v, kp, vp, batch, n_new, c->cfg.n_kv_heads, c->row_bytes, c->row_stride,
                           c->slot_len[slot], rag ? unit_len_dev(c, slot) : nullptr, replay_counter(c), c->cfg.max_seq,
                           reinterpret_cast<int*>(c->ws + c->off_status), (long long)c->plane_bytes, take_early_start(c),
                           st) != cudaSuccess)
        return KVS_ERR_CUDA;
    if (rag) {
        const int units = batch * c->cfg.n_kv_heads;
        if (kvs::launch_add_len(unit_len_dev(c, slot), n_new, units, c->opt_pdl != 0, st) != cudaSuccess)
            return KVS_ERR_CUDA;
        for (int u = 0; u < units; ++u) c->unit_len_host[slot][u] += n_new;
        c->seq += 1;
    }
    c->seq += 1;
    c->app_seq_prev[slot] = c->app_seq_latest[slot];
    c->app_seq_latest[slot] = c->seq;
    c->app_start_latest[slot] = c->slot_len[slot];
    c->slot_len[slot] += n_new;
    c->cur_batch = batch;
    c->stats.append_launches += 1;
    c->stats.kv_bytes_appended += 2ull * batch * c->cfg.n_kv_heads * n_new * c->row_bytes;
    return KVS_OK;
}

// Where one attention call keeps its split-K partial results and reports device-side trouble.
struct AttentionScratch {
    float* part_o;
    float* part_ml;
    int* flags;          // [units] ints, zero between launches
    int* status;
    bool programmatic;   // early-start launches (only when the call follows this context's own kernels)
    bool tracked;        // the call is part of the context's one ordered chain of launches (see kvs_ctx::seq)
};

// Which kernel serves the context's shape and how the call is cut into work.  bf16 groups of three
// or more q-heads per kv-head are a real (if thin) contraction and go to the tensor cores.
bool choose_plan(const kvs_ctx* c, int units, int n, kvs::DecodePlan* plan) {
    const bool use_mma = c->have_tensor_map && (c->opt_kernel == 2 || (c->opt_kernel == 0 && c->G >= 3));
    if (use_mma)
        kvs::plan_decode_mma(units, n, c->cfg.head_dim, c->sm_count, c->opt_max_ctas, plan);
    else
        kvs::plan_decode_scalar(units, n, c->G, c->cfg.head_dim, c->cfg.dtype, c->sm_count, c->opt_max_ctas, plan);
    return use_mma;
}

// Split-K kernel + combine kernel of one layer, with the given plan and scratch.
// With k_new / v_new the split-K kernel also appends that one row per unit (the slot's length must
// already count it).
kvs_status run_attention(kvs_ctx* c, int slot, const void* q, float* out, int batch, const kvs::DecodePlan& plan,
                         bool use_mma, const AttentionScratch& scratch, cudaStream_t st, const void* k_new = nullptr,
                         const void* v_new = nullptr) {
    kvs::DecodeArgs a;
    a.q = q;
    a.kplane = c->pool + (size_t)(2 * slot) * c->plane_bytes;
    a.vplane = c->pool + (size_t)(2 * slot + 1) * c->plane_bytes;
    a.part_o = scratch.part_o;
    a.part_ml = scratch.part_ml;
    a.out = out;
    a.status = scratch.status;
    a.n = c->slot_len[slot];
    a.row_stride = c->row_stride;
    a.capacity = c->cfg.max_seq;
    a.units = batch * c->cfg.n_kv_heads;
    a.G = c->G;
    a.D = c->cfg.head_dim;
    a.dtype = c->cfg.dtype;
    a.scale_log2 = c->scale * 1.4426950408889634f;
    a.programmatic = scratch.programmatic;
    a.safe_rows = scratch.programmatic ? safe_rows_of(c, slot) : 0;
    a.unit_len = c->ragged[slot] ? unit_len_dev(c, slot) : nullptr;
    a.n_extra = replay_counter(c);
    a.k_new = k_new;
    a.v_new = v_new;
    if (k_new) a.safe_rows = std::min(a.safe_rows, a.n - 1);   // the new row is fetched after the kernel has stored it
    a.plane_bytes = (long long)c->plane_bytes;
    a.wait_ns = 1000ull * (unsigned long long)c->opt_wait_us;
    a.trace = nullptr;
    if (c->trace_buf && c->trace_launch < c->trace_capacity)
        a.trace = c->trace_buf + (size_t)(c->trace_launch++) * kvs::kTraceLaunchWords;
    a.stall_tile = c->stall_tile >= 0 ? std::min<long long>(c->stall_tile, plan.T - 1) : -1;
    c->stall_tile = -1;
    a.finish_in_kernel = c->opt_finish != 0 && kvs::can_finish_in_kernel(plan, a.units);
    a.flags = scratch.flags;
    if (scratch.tracked) {
        c->seq += a.finish_in_kernel ? 1 : 2;     // split-K kernel, then (unless it finishes the units itself) combine
        c->last_splitk_seq = a.finish_in_kernel ? c->seq : c->seq - 1;
    }
    if (use_mma) {
        const long long plane_rows = (long long)c->cfg.max_batch * c->cfg.n_kv_heads * c->row_stride;
        if (kvs::launch_decode_mma(a, plan, c->tensor_map, c->tensor_map_tail, plane_rows * (2 * slot),
                                   plane_rows * (2 * slot + 1), st) != cudaSuccess)
            return KVS_ERR_CUDA;
    } else {
        if (kvs::launch_decode_scalar(a, plan, st) != cudaSuccess) return KVS_ERR_CUDA;
    }
    if (!a.finish_in_kernel) {
        if (kvs::launch_combine(a, plan, st) != cudaSuccess) return KVS_ERR_CUDA;
        c->stats.combine_launches += 1;
    }
    c->last_plan = plan;
    c->stats.attention_launches += 1;
    if (c->ragged[slot]) {
        unsigned long long rows = 0;
        for (int u = 0; u < a.units; ++u) rows += c->unit_len_host[slot][u];
        c->stats.kv_bytes_read += 2ull * rows * c->row_bytes;
    } else {
        c->stats.kv_bytes_read += 2ull * a.units * a.n * c->row_bytes;
    }
    return KVS_OK;
}

// One decode step of a computing layer with the append riding in the split-K kernel (the caller
// has checked the arguments; the slot is not ragged).
kvs_status do_fused_step(kvs_ctx* c, int layer, const void* q, const void* k, const void* v, float* out, int batch,
                         cudaStream_t st) {
    const int slot = c->slot_of_layer[layer];
    const int old_len = c->slot_len[slot];
    kvs::DecodePlan plan;
    const bool use_mma = choose_plan(c, batch * c->cfg.n_kv_heads, old_len + 1, &plan);
    const AttentionScratch scratch = {reinterpret_cast<float*>(c->ws + c->off_part_o),
                                      reinterpret_cast<float*>(c->ws + c->off_part_ml),
                                      reinterpret_cast<int*>(c->ws + c->off_flags),
                                      reinterpret_cast<int*>(c->ws + c->off_status), take_early_start(c), true};
    // run_attention works out which rows are stable from the appends before this one
    c->slot_len[slot] = old_len + 1;
    const kvs_status s = run_attention(c, slot, q, out, batch, plan, use_mma, scratch, st, k, v);
    if (s != KVS_OK) {
        c->slot_len[slot] = old_len;
        return s;
    }
    c->app_seq_prev[slot] = c->app_seq_latest[slot];
    c->app_seq_latest[slot] = c->last_splitk_seq;   // the kernel that appended is the split-K kernel itself
    c->app_start_latest[slot] = old_len;
    c->cur_batch = batch;
    c->stats.fused_appends += 1;
    c->stats.kv_bytes_appended += 2ull * batch * c->cfg.n_kv_heads * c->row_bytes;
    return KVS_OK;
}

kvs_status do_attention(kvs_ctx* c, int layer, const void* q, float* out, int batch, cudaStream_t st) {
    const int slot = c->slot_of_layer[layer];
    kvs::DecodePlan plan;
    const bool use_mma = choose_plan(c, batch * c->cfg.n_kv_heads, c->slot_len[slot], &plan);
    const AttentionScratch scratch = {reinterpret_cast<float*>(c->ws + c->off_part_o),
                                      reinterpret_cast<float*>(c->ws + c->off_part_ml),
                                      reinterpret_cast<int*>(c->ws + c->off_flags),
                                      reinterpret_cast<int*>(c->ws + c->off_status), take_early_start(c), true};
    return run_attention(c, slot, q, out, batch, plan, use_mma, scratch, st);
}

}  // namespace

extern "C" {

kvs_status kvs_create(const kvs_config* cfg, kvs_ctx** out) {
    if (!cfg || !out) return KVS_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_layers < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->max_batch < 1 || cfg->max_seq < 1)
        return KVS_ERR_INVALID_ARG;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0) return KVS_ERR_INVALID_ARG;
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    const bool pow2_group = (G == 1 || G == 2 || G == 4 || G == 8);
    if (G > 8) return KVS_ERR_INVALID_ARG;
    // groups of 3, 5, 6 or 7 q-heads exist only on the tensor-core kernel, which is bf16-only
    if (!pow2_group && cfg->dtype != KVS_BF16) return KVS_ERR_INVALID_ARG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return KVS_ERR_INVALID_ARG;
    if (cfg->dtype != KVS_BF16 && cfg->dtype != KVS_F32) return KVS_ERR_INVALID_ARG;
    if (cfg->device < 0 || cfg->device >= 64) return KVS_ERR_INVALID_ARG;
    if (!(cfg->softmax_scale >= 0.f) || std::isinf(cfg->softmax_scale)) return KVS_ERR_INVALID_ARG;
    if (cfg->max_seq > (1 << 30) - kRowStrideQuantum) return KVS_ERR_INVALID_ARG;
    kvs_ctx* c = new (std::nothrow) kvs_ctx();
    if (!c) return KVS_ERR_OOM;
    c->cfg = *cfg;
    c->G = G;
    c->elem = cfg->dtype == KVS_BF16 ? 2 : 4;
    c->row_bytes = cfg->head_dim * c->elem;
    c->row_stride = (cfg->max_seq + kRowStrideQuantum - 1) / kRowStrideQuantum * kRowStrideQuantum;
    c->plane_bytes = (size_t)cfg->max_batch * cfg->n_kv_heads * c->row_stride * c->row_bytes;
    c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    c->share_map.resize(cfg->n_layers);
    for (int l = 0; l < cfg->n_layers; ++l) c->share_map[l] = l;
    resolve_map(c);
    layout_workspace(c);
    *out = c;
    return KVS_OK;
}

kvs_status kvs_destroy(kvs_ctx* ctx) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (ctx->copy_ready) {
        DeviceGuard guard(ctx->cfg.device);
        if (guard.ok) {
            for (int i = 0; i < kvs_ctx::kChunks; ++i) {
                cudaEventDestroy(ctx->ev_in[i]);
                cudaEventDestroy(ctx->ev_done[i]);
            }
            cudaEventDestroy(ctx->ev_start);
            cudaStreamDestroy(ctx->copy_stream);
            cudaStreamDestroy(ctx->out_stream);
        }
    }
    delete ctx;
    return KVS_OK;
}

kvs_status kvs_set_share_map(kvs_ctx* ctx, const int32_t* share_map) {
    if (!ctx || !share_map) return KVS_ERR_INVALID_ARG;
    for (int s = 0; s < ctx->n_slots; ++s)
        if (ctx->slot_len[s] != 0) return KVS_ERR_STATE;
    const int L = ctx->cfg.n_layers;
    for (int l = 0; l < L; ++l)
        if (share_map[l] < 0 || share_map[l] > l) return KVS_ERR_BAD_SHARE_MAP;
    const int old_slots = ctx->n_slots;
    for (int l = 0; l < L; ++l) ctx->share_map[l] = share_map[l];
    resolve_map(ctx);
    // A pool bound for fewer slots than the new strategy needs can no longer be used.
    if (ctx->bound && ctx->n_slots > old_slots) {
        ctx->bound = false;
        ctx->pool = nullptr;
        ctx->ws = nullptr;
    }
    return KVS_OK;
}

kvs_status kvs_required_bytes(const kvs_ctx* ctx, size_t* pool_bytes, size_t* workspace_bytes) {
    if (!ctx || !pool_bytes || !workspace_bytes) return KVS_ERR_INVALID_ARG;
    *pool_bytes = (size_t)ctx->n_slots * 2 * ctx->plane_bytes;
    *workspace_bytes = ctx->ws_bytes;
    return KVS_OK;
}

kvs_status kvs_bind_memory(kvs_ctx* ctx, void* pool, size_t pool_bytes, void* workspace, size_t workspace_bytes) {
    if (!ctx || !pool || !workspace) return KVS_ERR_INVALID_ARG;
    if (((uintptr_t)pool % kAlign) != 0 || ((uintptr_t)workspace % kAlign) != 0) return KVS_ERR_INVALID_ARG;
    const size_t need_pool = (size_t)ctx->n_slots * 2 * ctx->plane_bytes;
    if (pool_bytes < need_pool || workspace_bytes < ctx->ws_bytes) return KVS_ERR_OOM;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (init_device_once(ctx->cfg.device) != cudaSuccess) return KVS_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->cfg.device) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaMemsetAsync(pool, 0, need_pool, 0) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaMemsetAsync(workspace, 0, ctx->ws_bytes, 0) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(0) != cudaSuccess) return KVS_ERR_CUDA;
    ctx->have_tensor_map = false;
    if (ctx->cfg.dtype == KVS_BF16) {
        const long long total_rows = (long long)(need_pool / ctx->row_bytes);
        if (total_rows >= (1ll << 31)) return KVS_ERR_INVALID_ARG;
        if (kvs::make_pool_tensor_map(ctx->tensor_map, pool, total_rows, ctx->cfg.head_dim, false) != cudaSuccess ||
            kvs::make_pool_tensor_map(ctx->tensor_map_tail, pool, total_rows, ctx->cfg.head_dim, true) != cudaSuccess)
            return KVS_ERR_CUDA;
        ctx->have_tensor_map = true;
    }
    ctx->sm_count = sms;
    {
        int l2 = 0;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, ctx->cfg.device) == cudaSuccess && l2 > 0) ctx->l2_bytes = l2;
    }
    ctx->pool = static_cast<char*>(pool);
    ctx->ws = static_cast<char*>(workspace);
    ctx->bound = true;
    for (auto& x : ctx->slot_len) x = 0;
    for (auto& x : ctx->ragged) x = 0;
    ctx->cur_batch = 0;
    // the device was idle a moment ago: nothing of this context is in flight
    for (auto& x : ctx->app_seq_latest) x = 0;
    for (auto& x : ctx->app_seq_prev) x = 0;
    ctx->last_splitk_seq = 0;
    return KVS_OK;
}

kvs_status kvs_reset(kvs_ctx* ctx) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    for (auto& x : ctx->ragged) x = 0;
    for (auto& x : ctx->slot_len) x = 0;
    ctx->cur_batch = 0;
    return KVS_OK;
}

kvs_status kvs_truncate(kvs_ctx* ctx, int32_t n_tokens) {
    if (!ctx || n_tokens < 0) return KVS_ERR_INVALID_ARG;
    // a slot rows were evicted from has per-unit lengths on the device as well: refused, not half-updated
    for (int s = 0; s < ctx->n_slots; ++s)
        if (ctx->slot_len[s] > n_tokens && ctx->ragged[s]) return KVS_ERR_STATE;
    for (int s = 0; s < ctx->n_slots; ++s) {
        if (ctx->slot_len[s] <= n_tokens) continue;
        ctx->slot_len[s] = n_tokens;
        // Rows from n_tokens on will be written again.  Kernels of earlier calls may still be reading
        // them, but every writer stores only after its wait for its predecessor; and what a later
        // launch may fetch before its own wait must lie below the old and the new writes alike.
        ctx->app_start_latest[s] = std::min(ctx->app_start_latest[s], n_tokens);
    }
    if (n_tokens == 0) ctx->cur_batch = 0;
    return KVS_OK;
}

kvs_status kvs_append(kvs_ctx* ctx, int32_t layer, const void* k, const void* v, int32_t batch, int32_t n_new,
                      void* stream) {
    bool sharing = false;
    kvs_status s = check_append(ctx, layer, k, v, batch, n_new, &sharing);
    if (s != KVS_OK) return s;
    if (sharing) {
        ctx->stats.append_skipped += 1;
        return KVS_OK;
    }
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    return do_append(ctx, layer, k, v, batch, n_new, static_cast<cudaStream_t>(stream));
}

kvs_status kvs_decode_attention(kvs_ctx* ctx, int32_t layer, const void* q, float* out, int32_t batch, void* stream) {
    kvs_status s = check_attention(ctx, layer, q, out, batch);
    if (s != KVS_OK) return s;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    return do_attention(ctx, layer, q, out, batch, static_cast<cudaStream_t>(stream));
}

kvs_status kvs_decode_step(kvs_ctx* ctx, int32_t layer, const void* q, const void* k, const void* v, float* out,
                           int32_t batch, void* stream) {
    bool sharing = false;
    kvs_status s = check_append(ctx, layer, k, v, batch, 1, &sharing);
    if (s != KVS_OK) return s;
    if (!q || !out) return KVS_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (sharing) {
        s = check_attention(ctx, layer, q, out, batch);
        if (s != KVS_OK) return s;
        DeviceGuard guard(ctx->cfg.device);
        if (!guard.ok) return KVS_ERR_CUDA;
        ctx->stats.append_skipped += 1;
        return do_attention(ctx, layer, q, out, batch, st);
    }
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    const int slot = ctx->slot_of_layer[layer];
    if (((uintptr_t)q % 16) != 0 || ((uintptr_t)out % 4) != 0) return KVS_ERR_INVALID_ARG;
    if (!ctx->ragged[slot]) return do_fused_step(ctx, layer, q, k, v, out, batch, st);
    s = do_append(ctx, layer, k, v, batch, 1, st);
    if (s != KVS_OK) return s;
    return do_attention(ctx, layer, q, out, batch, st);
}

kvs_status kvs_prefill_attention(kvs_ctx* ctx, int32_t layer, const void* q, float* out, int32_t batch, int32_t n_q,
                                 void* stream) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    if (layer < 0 || layer >= ctx->cfg.n_layers || !q || !out) return KVS_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch || n_q < 1) return KVS_ERR_INVALID_ARG;
    if (ctx->cfg.dtype == KVS_BF16 && !ctx->have_tensor_map) return KVS_ERR_STATE;
    if (((uintptr_t)q % 16) != 0 || ((uintptr_t)out % 16) != 0) return KVS_ERR_INVALID_ARG;
    const int slot = ctx->slot_of_layer[layer];
    const int n = ctx->slot_len[slot];
    if (n == 0 || ctx->ragged[slot]) return KVS_ERR_STATE;   // positions are undefined once rows were evicted
    if (batch > ctx->cur_batch || n_q > n) return KVS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (ctx->cfg.dtype == KVS_F32) {
        // fp32 storage: the plain fp32 kernel (a plain launch, like the tensor-core one)
        const char* kp = ctx->pool + (size_t)(2 * slot) * ctx->plane_bytes;
        if (kvs::launch_prefill_f32(q, out, kp, kp + ctx->plane_bytes, batch, n_q, ctx->cfg.n_q_heads, ctx->G,
                                    ctx->cfg.head_dim, n, ctx->row_stride, ctx->scale * 1.4426950408889634f,
                                    static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return KVS_ERR_CUDA;
        ctx->seq += 1;
        ctx->last_splitk_seq = ctx->seq;
        ctx->stats.prefill_launches += 1;
        ctx->counter_written = false;
        return KVS_OK;
    }
    const long long plane_rows = (long long)ctx->cfg.max_batch * ctx->cfg.n_kv_heads * ctx->row_stride;
    // the prefill kernel's work counter lives in the status block, 64 bytes after the status word
    if (kvs::launch_prefill(q, out, reinterpret_cast<int*>(ctx->ws + ctx->off_status),
                            reinterpret_cast<int*>(ctx->ws + ctx->off_status + 64), ctx->tensor_map, batch, n_q,
                            ctx->cfg.n_q_heads, ctx->G, ctx->cfg.head_dim, n, ctx->row_stride, plane_rows * (2 * slot),
                            plane_rows * (2 * slot + 1), plane_rows, ctx->scale * 1.4426950408889634f, ctx->sm_count, ctx->l2_bytes,
                            static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KVS_ERR_CUDA;
    // a plain launch: it starts only after everything before it on the stream has finished
    ctx->seq += 1;
    ctx->last_splitk_seq = ctx->seq;
    ctx->stats.prefill_launches += 1;
    ctx->counter_written = false;   // a plain launch: full dependency on everything before it
    ctx->stats.kv_bytes_read += 0;  // prefill is compute-bound; its K/V reads are not counted as decode traffic
    return KVS_OK;
}

kvs_status kvs_evict(kvs_ctx* ctx, int32_t layer, const int32_t* keep, const int32_t* n_keep, int32_t keep_stride,
                     int32_t batch, void* stream) {
    if (!ctx || !keep || !n_keep) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    if (layer < 0 || layer >= ctx->cfg.n_layers || keep_stride < 1) return KVS_ERR_INVALID_ARG;
    if (ctx->share_map[layer] != layer) return KVS_ERR_INVALID_ARG;   // a sharing layer has no cache of its own
    const int slot = ctx->slot_of_layer[layer];
    if (ctx->slot_len[slot] == 0) return KVS_ERR_STATE;
    if (batch < 1 || batch != ctx->cur_batch) return KVS_ERR_INVALID_ARG;
    const int units = batch * ctx->cfg.n_kv_heads;
    int longest = 0;
    for (int u = 0; u < units; ++u) {
        const int have = ctx->ragged[slot] ? ctx->unit_len_host[slot][u] : ctx->slot_len[slot];
        if (n_keep[u] < 1 || n_keep[u] > have || n_keep[u] > keep_stride) return KVS_ERR_INVALID_ARG;
        longest = n_keep[u] > longest ? n_keep[u] : longest;
    }
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* counts = reinterpret_cast<int*>(ctx->ws + ctx->off_counts);
    int* lens = unit_len_dev(ctx, slot);
    if (cudaMemcpyAsync(counts, n_keep, sizeof(int32_t) * units, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KVS_ERR_CUDA;
    char* kp = ctx->pool + (size_t)(2 * slot) * ctx->plane_bytes;
    const bool pdl = ctx->opt_pdl != 0;
    if (kvs::launch_evict(kp, kp + ctx->plane_bytes, keep, counts, ctx->ragged[slot] ? lens : nullptr,
                          ctx->slot_len[slot], units, keep_stride, ctx->row_bytes, ctx->row_stride,
                          reinterpret_cast<int*>(ctx->ws + ctx->off_status), false, st) != cudaSuccess ||
        kvs::launch_set_len(lens, counts, units, pdl, st) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->unit_len_host[slot].assign((size_t)ctx->cfg.max_batch * ctx->cfg.n_kv_heads, 0);
    for (int u = 0; u < units; ++u) ctx->unit_len_host[slot][u] = n_keep[u];
    ctx->ragged[slot] = 1;
    ctx->slot_len[slot] = longest;
    // every row of the slot may just have moved: nothing of it may be fetched early
    ctx->seq += 2;
    ctx->app_seq_prev[slot] = ctx->seq;
    ctx->app_seq_latest[slot] = ctx->seq;
    ctx->app_start_latest[slot] = 0;
    ctx->stats.evict_launches += 1;
    ctx->counter_written = false;   // a plain launch: full dependency on everything before it
    return KVS_OK;
}

kvs_status kvs_unit_len(const kvs_ctx* ctx, int32_t layer, int32_t b, int32_t h, int32_t* len) {
    if (!ctx || !len || layer < 0 || layer >= ctx->cfg.n_layers) return KVS_ERR_INVALID_ARG;
    if (b < 0 || b >= ctx->cfg.max_batch || h < 0 || h >= ctx->cfg.n_kv_heads) return KVS_ERR_INVALID_ARG;
    const int slot = ctx->slot_of_layer[layer];
    *len = ctx->ragged[slot] ? ctx->unit_len_host[slot][(size_t)b * ctx->cfg.n_kv_heads + h]
                             : (b < ctx->cur_batch ? ctx->slot_len[slot] : 0);
    return KVS_OK;
}

kvs_status kvs_layer_distances(kvs_ctx* ctx, int32_t batch, float* dist, void* stream) {
    if (!ctx || !dist) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    if (ctx->cfg.n_layers > kvs::kMaxLayersSearch) return KVS_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cur_batch) return ctx->cur_batch == 0 ? KVS_ERR_STATE : KVS_ERR_INVALID_ARG;
    const int n = ctx->slot_len[0];
    if (n == 0) return KVS_ERR_STATE;
    for (int s = 0; s < ctx->n_slots; ++s)
        if (ctx->slot_len[s] != n || ctx->ragged[s]) return KVS_ERR_STATE;   // equally long, un-evicted caches only
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    {
        // not recorded into graphs: the launch pattern (programmatic dependents between plain launches) is
        // only exercised on a live stream
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cap) != cudaSuccess) return KVS_ERR_CUDA;
        if (cap != cudaStreamCaptureStatusNone) return KVS_ERR_STATE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int launches = 0;
    if (kvs::launch_layer_distances(ctx->pool, (long long)ctx->plane_bytes, ctx->slot_of_layer.data(), ctx->cfg.n_layers,
                                    ctx->n_slots, batch, ctx->cfg.n_kv_heads, n, ctx->row_stride, ctx->cfg.head_dim,
                                    ctx->cfg.dtype, reinterpret_cast<float*>(ctx->ws + ctx->off_search), ctx->search_bytes,
                                    dist, ctx->sm_count, &launches, st) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->seq += launches;
    ctx->last_splitk_seq = ctx->seq;     // the first and the last launches are plain: everything before them has finished
    ctx->stats.search_launches += launches;
    ctx->counter_written = false;   // a plain launch: full dependency on everything before it
    return KVS_OK;
}

kvs_status kvs_mean_cosine(kvs_ctx* ctx, const void* a, const void* b, int32_t n_samples, int64_t dim, float* out,
                           void* stream) {
    if (!ctx || !a || !b || !out) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    if (n_samples < 1 || dim < 2 || (dim & 1) != 0) return KVS_ERR_INVALID_ARG;
    if (((uintptr_t)a % 8) != 0 || ((uintptr_t)b % 8) != 0) return KVS_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (kvs::launch_mean_cosine(a, b, n_samples, dim, ctx->cfg.dtype, reinterpret_cast<double*>(ctx->ws + ctx->off_search),
                                out, ctx->sm_count, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->seq += 2;
    ctx->last_splitk_seq = ctx->seq;
    ctx->stats.search_launches += 2;
    ctx->counter_written = false;   // a plain launch: full dependency on everything before it
    return KVS_OK;
}

kvs_status kvs_replay_advance(kvs_ctx* ctx, void* stream) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound || !ctx->opt_replay) return KVS_ERR_STATE;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    // Outside stream capture the host lengths already advance with every call, so there is nothing
    // to count: the same step function can be run eagerly and recorded.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cap) != cudaSuccess) return KVS_ERR_CUDA;
    if (cap != cudaStreamCaptureStatusActive) return KVS_OK;
    if (kvs::launch_replay_advance(reinterpret_cast<int*>(ctx->ws + ctx->off_replay), ctx->opt_pdl != 0,
                                   static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->seq += 1;
    ctx->counter_written = true;
    return KVS_OK;
}

kvs_status kvs_replay_commit(kvs_ctx* ctx, int32_t times_run, void* stream) {
    if (!ctx || times_run < 1) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound || !ctx->opt_replay) return KVS_ERR_STATE;
    const int extra = times_run - 1;     // the recording itself was already counted once
    for (int s = 0; s < ctx->n_slots; ++s)
        if (ctx->slot_len[s] > 0 && (long long)ctx->slot_len[s] + extra > ctx->cfg.max_seq) return KVS_ERR_CAPACITY;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (cudaMemsetAsync(ctx->ws + ctx->off_replay, 0, sizeof(int), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->counter_written = true;
    for (int s = 0; s < ctx->n_slots; ++s) {
        if (ctx->slot_len[s] == 0) continue;
        ctx->slot_len[s] += extra;
        if (ctx->ragged[s])
            for (int u = 0; u < ctx->cur_batch * ctx->cfg.n_kv_heads; ++u) ctx->unit_len_host[s][u] += extra;
    }
    return KVS_OK;
}

kvs_status kvs_step_host(kvs_ctx* ctx, const void* q_host, const void* k_host, const void* v_host, float* out_host,
                         int32_t batch, void* stream, uint64_t* h2d_bytes, uint64_t* d2h_bytes) {
    if (!ctx || !q_host || !k_host || !v_host || !out_host) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    const kvs_config& f = ctx->cfg;
    if (batch < 1 || batch > f.max_batch) return KVS_ERR_INVALID_ARG;
    if (ctx->cur_batch != 0 && batch != ctx->cur_batch) return KVS_ERR_INVALID_ARG;
    // every own-cache slot grows by one token; check all capacities before any work
    for (int sl = 0; sl < ctx->n_slots; ++sl)
        if (ctx->slot_len[sl] + 1 > f.max_seq) return KVS_ERR_CAPACITY;
    DeviceGuard guard(f.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t q_layer = (size_t)batch * f.n_q_heads * f.head_dim * ctx->elem;
    const size_t kv_layer = (size_t)batch * f.n_kv_heads * f.head_dim * ctx->elem;
    const size_t out_layer = (size_t)batch * f.n_q_heads * f.head_dim * sizeof(float);
    char* dq = ctx->ws + ctx->off_stage_q;
    char* dk = ctx->ws + ctx->off_stage_k;
    char* dv = ctx->ws + ctx->off_stage_v;
    char* dout = ctx->ws + ctx->off_stage_out;
    uint64_t h2d = 0;
    // The layers are cut into chunks; one extra stream copies chunk c+1's inputs in and another copies
    // chunk c-1's outputs out while chunk c computes, so only the first input copy and the last
    // output copy are exposed.  Chunk c+1's copies are queued before chunk c's kernels so that the
    // host never stands between the device and its next piece of work.
    if (!ctx->copy_ready) {
        if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->out_stream, cudaStreamNonBlocking) != cudaSuccess)
            return KVS_ERR_CUDA;
        for (int i = 0; i < kvs_ctx::kChunks; ++i)
            if (cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming) != cudaSuccess)
                return KVS_ERR_CUDA;
        if (cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming) != cudaSuccess) return KVS_ERR_CUDA;
        ctx->copy_ready = true;
    }
    cudaStream_t cs = ctx->copy_stream, os = ctx->out_stream;
    const int L = f.n_layers;
    const int chunks = L < ctx->opt_host_chunks ? L : ctx->opt_host_chunks;
    // the copy streams start after whatever the caller already queued on `st`
    if (cudaEventRecord(ctx->ev_start, st) != cudaSuccess || cudaStreamWaitEvent(cs, ctx->ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(os, ctx->ev_start, 0) != cudaSuccess)
        return KVS_ERR_CUDA;
    // Chunk c covers layers [edge(c), edge(c+1)).  With three or more chunks the first and the last are
    // a single layer, so that the input copy nothing can hide and the output copy nothing can hide
    // are as small as they can be; the layers between are cut evenly.
    auto edge = [&](int c) -> int {
        if (chunks < 3 || L < chunks + 2) return (int)((long long)c * L / chunks);
        if (c == 0) return 0;
        if (c == chunks) return L;
        return 1 + (int)((long long)(c - 1) * (L - 2) / (chunks - 2));
    };
    auto copy_in = [&](int c) -> bool {
        const int l0 = edge(c), l1 = edge(c + 1);
        if (cudaMemcpyAsync(dq + q_layer * l0, (const char*)q_host + q_layer * l0, q_layer * (l1 - l0),
                            cudaMemcpyHostToDevice, cs) != cudaSuccess)
            return false;
        h2d += q_layer * (l1 - l0);
        // K/V of own-cache layers only; consecutive own-cache layers go in one copy
        for (int l = l0; l < l1;) {
            if (ctx->share_map[l] != l) { ++l; continue; }
            int e = l;
            while (e + 1 < l1 && ctx->share_map[e + 1] == e + 1) ++e;
            const size_t off = kv_layer * l, len = kv_layer * (e - l + 1);
            if (cudaMemcpyAsync(dk + off, (const char*)k_host + off, len, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
                cudaMemcpyAsync(dv + off, (const char*)v_host + off, len, cudaMemcpyHostToDevice, cs) != cudaSuccess)
                return false;
            h2d += 2 * len;
            l = e + 1;
        }
        return cudaEventRecord(ctx->ev_in[c], cs) == cudaSuccess;
    };
    if (!copy_in(0)) return KVS_ERR_CUDA;
    for (int c = 0; c < chunks; ++c) {
        const int l0 = edge(c), l1 = edge(c + 1);
        if (c + 1 < chunks && !copy_in(c + 1)) return KVS_ERR_CUDA;
        if (cudaStreamWaitEvent(st, ctx->ev_in[c], 0) != cudaSuccess) return KVS_ERR_CUDA;
        for (int l = l0; l < l1; ++l) {
            float* o = reinterpret_cast<float*>(dout + out_layer * l);
            kvs_status s;
            if (ctx->share_map[l] == l && !ctx->ragged[ctx->slot_of_layer[l]]) {
                // the append rides in the split-K kernel (the staging rows are 16-byte aligned)
                s = do_fused_step(ctx, l, dq + q_layer * l, dk + kv_layer * l, dv + kv_layer * l, o, batch, st);
            } else {
                if (ctx->share_map[l] == l) {
                    s = do_append(ctx, l, dk + kv_layer * l, dv + kv_layer * l, batch, 1, st);
                    if (s != KVS_OK) return s;
                } else {
                    ctx->stats.append_skipped += 1;
                }
                s = do_attention(ctx, l, dq + q_layer * l, o, batch, st);
            }
            if (s != KVS_OK) return s;
        }
        if (cudaEventRecord(ctx->ev_done[c], st) != cudaSuccess || cudaStreamWaitEvent(os, ctx->ev_done[c], 0) != cudaSuccess)
            return KVS_ERR_CUDA;
        if (cudaMemcpyAsync((char*)out_host + out_layer * l0, dout + out_layer * l0, out_layer * (l1 - l0),
                            cudaMemcpyDeviceToHost, os) != cudaSuccess)
            return KVS_ERR_CUDA;
    }
    if (cudaStreamSynchronize(os) != cudaSuccess || cudaStreamSynchronize(cs) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return KVS_ERR_CUDA;
    if (h2d_bytes) *h2d_bytes = h2d;
    if (d2h_bytes) *d2h_bytes = out_layer * f.n_layers;
    return KVS_OK;
}

kvs_status kvs_num_slots(const kvs_ctx* ctx, int32_t* n_slots) {
    if (!ctx || !n_slots) return KVS_ERR_INVALID_ARG;
    *n_slots = ctx->n_slots;
    return KVS_OK;
}

kvs_status kvs_slot_of_layer(const kvs_ctx* ctx, int32_t layer, int32_t* slot) {
    if (!ctx || !slot || layer < 0 || layer >= ctx->cfg.n_layers) return KVS_ERR_INVALID_ARG;
    *slot = ctx->slot_of_layer[layer];
    return KVS_OK;
}

kvs_status kvs_seq_len(const kvs_ctx* ctx, int32_t layer, int32_t* len) {
    if (!ctx || !len || layer < 0 || layer >= ctx->cfg.n_layers) return KVS_ERR_INVALID_ARG;
    *len = ctx->slot_len[ctx->slot_of_layer[layer]];
    return KVS_OK;
}

kvs_status kvs_row_stride(const kvs_ctx* ctx, int32_t* rows) {
    if (!ctx || !rows) return KVS_ERR_INVALID_ARG;
    *rows = ctx->row_stride;
    return KVS_OK;
}

kvs_status kvs_plane_offset(const kvs_ctx* ctx, int32_t slot, int32_t kv, size_t* offset) {
    if (!ctx || !offset || slot < 0 || slot >= ctx->n_slots || (kv != 0 && kv != 1)) return KVS_ERR_INVALID_ARG;
    *offset = (size_t)(2 * slot + kv) * ctx->plane_bytes;
    return KVS_OK;
}

kvs_status kvs_stats(const kvs_ctx* ctx, kvs_stats_t* stats) {
    if (!ctx || !stats) return KVS_ERR_INVALID_ARG;
    *stats = ctx->stats;
    return KVS_OK;
}

kvs_status kvs_last_device_status(kvs_ctx* ctx, int32_t* device_status) {
    if (!ctx || !device_status) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, ctx->ws + ctx->off_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return KVS_ERR_CUDA;
    *device_status = v;
    return KVS_OK;
}

kvs_status kvs_clear_device_status(kvs_ctx* ctx, void* stream) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // a launch that gave up may have left hand-over flags raised: they go back to zero with the status word
    if (cudaMemsetAsync(ctx->ws + ctx->off_status, 0, sizeof(int), st) != cudaSuccess ||
        cudaMemsetAsync(ctx->ws + ctx->off_flags, 0, sizeof(int32_t) * ctx->cfg.max_batch * ctx->cfg.n_kv_heads, st) !=
            cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->counter_written = true;   // the next launch takes a full dependency: it starts with the clears done
    return KVS_OK;
}

kvs_status kvs_selftest_stalled_copy(kvs_ctx* ctx, int32_t layer, const void* q, float* out, int32_t batch, void* stream) {
    kvs_status s = check_attention(ctx, layer, q, out, batch);
    if (s != KVS_OK) return s;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    const int slot = ctx->slot_of_layer[layer];
    kvs::DecodePlan plan;
    choose_plan(ctx, batch * ctx->cfg.n_kv_heads, ctx->slot_len[slot], &plan);
    ctx->stall_tile = plan.T / 2;          // a tile in the middle of the line
    ctx->counter_written = true;           // a plain launch, and so is whatever follows it
    s = do_attention(ctx, layer, q, out, batch, static_cast<cudaStream_t>(stream));
    ctx->stall_tile = -1;
    ctx->counter_written = true;
    return s;
}

kvs_status kvs_selftest_wait_timeout(kvs_ctx* ctx, uint32_t limit_us, uint64_t* waited_ns, void* stream) {
    if (!ctx || limit_us < 1 || limit_us > 1000000u) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound) return KVS_ERR_STATE;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the measured wait goes to a spare word of the status block (128 bytes after the status word)
    unsigned long long* waited_dev = reinterpret_cast<unsigned long long*>(ctx->ws + ctx->off_status + 128);
    if (kvs::launch_wait_timeout_selftest(reinterpret_cast<int*>(ctx->ws + ctx->off_status), 1000ull * limit_us, waited_dev,
                                          st) != cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->seq += 1;
    ctx->last_splitk_seq = ctx->seq;   // a plain launch: everything before it has finished when it runs
    ctx->counter_written = false;
    unsigned long long w = 0;
    if (cudaMemcpyAsync(&w, waited_dev, sizeof(w), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return KVS_ERR_CUDA;
    if (waited_ns) *waited_ns = w;
    return KVS_OK;
}

kvs_status kvs_trace_begin(kvs_ctx* ctx, void* buffer, size_t bytes) {
    if (!ctx || !buffer || ((uintptr_t)buffer % 8) != 0) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound || !kvs::is_tracing_build()) return KVS_ERR_STATE;
    const size_t per_launch = (size_t)kvs::kTraceLaunchWords * sizeof(unsigned long long);
    if (bytes < per_launch) return KVS_ERR_INVALID_ARG;
    ctx->trace_buf = static_cast<unsigned long long*>(buffer);
    ctx->trace_capacity = (int)std::min<size_t>(bytes / per_launch, 1 << 20);
    ctx->trace_launch = 0;
    return KVS_OK;
}

kvs_status kvs_trace_end(kvs_ctx* ctx, int32_t* launches_recorded) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (launches_recorded) *launches_recorded = ctx->trace_launch;
    ctx->trace_buf = nullptr;
    ctx->trace_capacity = ctx->trace_launch = 0;
    return KVS_OK;
}

kvs_status kvs_selftest_bounds(kvs_ctx* ctx, void* stream) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    if (!ctx->bound || !kvs::is_bounds_checking_build()) return KVS_ERR_STATE;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (kvs::launch_bounds_selftest(reinterpret_cast<int*>(ctx->ws + ctx->off_status), static_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
        return KVS_ERR_CUDA;
    ctx->seq += 1;
    ctx->last_splitk_seq = ctx->seq;   // a plain launch: everything before it has finished when it runs
    ctx->counter_written = false;
    return KVS_OK;
}

kvs_status kvs_set_option(kvs_ctx* ctx, int32_t option, int32_t value) {
    if (!ctx) return KVS_ERR_INVALID_ARG;
    switch (option) {
        case KVS_OPT_MAX_CTAS:
            if (value < 0 || value > kvs::kMaxCtas) return KVS_ERR_INVALID_ARG;
            ctx->opt_max_ctas = value;
            return KVS_OK;
        case KVS_OPT_EARLY_START:
            if (value != 0 && value != 1) return KVS_ERR_INVALID_ARG;
            ctx->opt_pdl = value;
            return KVS_OK;
        case KVS_OPT_REPLAY:
            if (value != 0 && value != 1) return KVS_ERR_INVALID_ARG;
            ctx->opt_replay = value;
            return KVS_OK;
        case KVS_OPT_HOST_CHUNKS:
            if (value < 1 || value > kvs_ctx::kChunks) return KVS_ERR_INVALID_ARG;
            ctx->opt_host_chunks = value;
            return KVS_OK;
        case KVS_OPT_WAIT_LIMIT_US:
            if (value < 100 || value > 10000000) return KVS_ERR_INVALID_ARG;
            ctx->opt_wait_us = value;
            return KVS_OK;
        case KVS_OPT_FINISH_IN_KERNEL:
            if (value != 0 && value != 1) return KVS_ERR_INVALID_ARG;
            ctx->opt_finish = value;
            return KVS_OK;
        case KVS_OPT_KERNEL:
            if (value < 0 || value > 2) return KVS_ERR_INVALID_ARG;
            if (value == 2 && ctx->cfg.dtype != KVS_BF16) return KVS_ERR_INVALID_ARG;  // tensor-core path is bf16 only
            if (value == 1 && ctx->G != 1 && ctx->G != 2 && ctx->G != 4 && ctx->G != 8)
                return KVS_ERR_INVALID_ARG;                                          // scalar path: groups of 1, 2, 4, 8
            ctx->opt_kernel = value;
            return KVS_OK;
        default:
            return KVS_ERR_INVALID_ARG;
    }
}

kvs_status kvs_last_launch(const kvs_ctx* ctx, int32_t* ctas, int32_t* tile_rows, int32_t* kernel) {
    if (!ctx || !ctas || !tile_rows || !kernel) return KVS_ERR_INVALID_ARG;
    *ctas = ctx->last_plan.NC;
    *tile_rows = ctx->last_plan.tile_rows;
    *kernel = ctx->last_plan.kernel;
    return KVS_OK;
}

const char* kvs_status_string(kvs_status s) {
    switch (s) {
        case KVS_OK: return "ok";
        case KVS_ERR_INVALID_ARG: return "invalid argument";
        case KVS_ERR_BAD_SHARE_MAP: return "bad share map";
        case KVS_ERR_STATE: return "call made in the wrong state";
        case KVS_ERR_CAPACITY: return "slot capacity exceeded";
        case KVS_ERR_OOM: return "bound buffer too small";
        case KVS_ERR_CUDA: return "CUDA call failed";
        case KVS_ERR_TIMEOUT: return "device-side wait timed out";
        case KVS_ERR_SCRATCH_LIMIT: return "call needs more scratch than the built-in scratch array holds";
        case KVS_ERR_BOUNDS: return "a bounds-checking build found an offset outside its buffer";
    }
    return "unknown status";
}

kvs_status kvs_read_roof(const void* src, size_t bytes, uint64_t* checksum, int32_t device, void* stream) {
    if (!src || !checksum || bytes == 0 || bytes % 32768 != 0 || device < 0 || device >= 64) return KVS_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return KVS_ERR_CUDA;
    if (init_device_once(device) != cudaSuccess) return KVS_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return KVS_ERR_CUDA;
    if (kvs::launch_read_roof(src, bytes, reinterpret_cast<unsigned long long*>(checksum), sms,
                              static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KVS_ERR_CUDA;
    return KVS_OK;
}

kvs_status kvs_decode_attention_static(kvs_ctx* ctx, int32_t layer, const void* q, float* out, int32_t batch,
                                       void* stream, int32_t* device_status) {
    kvs_status s = check_attention(ctx, layer, q, out, batch);
    if (s != KVS_OK) return s;
    if (((uintptr_t)device_status % 4) != 0) return KVS_ERR_INVALID_ARG;   // the kernels update it atomically
    kvs_ctx* c = ctx;
    const int slot = c->slot_of_layer[layer];
    const int units = batch * c->cfg.n_kv_heads;
    const int D = c->cfg.head_dim;
    kvs::DecodePlan plan;
    const bool use_mma = choose_plan(c, units, c->slot_len[slot], &plan);
    // one partial (o[D], m, l) per (piece, q-head); pieces are indexed unit + block
    const size_t pieces = (size_t)units + plan.NC;
    const size_t part_o_bytes = align_up(pieces * c->G * D * sizeof(float), kAlign);
    const size_t part_ml_bytes = align_up(pieces * c->G * 2 * sizeof(float), kAlign);
    const size_t flag_bytes = kStaticFlagBytes;
    if ((size_t)units * sizeof(int32_t) > kStaticFlagBytes ||
        kStaticStatusBytes + part_o_bytes + part_ml_bytes + flag_bytes > kStaticScratchBytes)
        return KVS_ERR_SCRATCH_LIMIT;

    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return KVS_ERR_CUDA;
    // the address was looked up when the context's memory was bound (per-device set-up): no
    // runtime query here
    unsigned char* base = g_static_ptr[c->cfg.device];
    if (g_static_err[c->cfg.device] != cudaSuccess || base == nullptr) return KVS_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status_word = device_status ? device_status : reinterpret_cast<int*>(base);
    // the array keeps whatever the previous call left; only the status word must start at zero
    if (cudaMemsetAsync(status_word, 0, sizeof(int), st) != cudaSuccess) return KVS_ERR_CUDA;
    // Plain launches: the kernels start after everything before them on `stream`.  The call may be
    // on another stream than the context's other calls, so it stays out of the bookkeeping that
    // decides what those calls may fetch early (untracked), and it leaves the "growth counter was
    // just written" mark for the next call of the chain.
    // layout: status word, flags (fixed size), partial outputs, partial (max, sum) pairs
    const AttentionScratch scratch = {reinterpret_cast<float*>(base + kStaticStatusBytes + flag_bytes),
                                      reinterpret_cast<float*>(base + kStaticStatusBytes + flag_bytes + part_o_bytes),
                                      reinterpret_cast<int*>(base + kStaticStatusBytes), status_word, false, false};
    return run_attention(c, slot, q, out, batch, plan, use_mma, scratch, st);
}

}  // extern "C"
