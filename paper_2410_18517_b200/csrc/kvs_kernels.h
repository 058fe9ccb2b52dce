// Internal launcher interface between the host API and the sm_100a kernels.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace kvs {

// How one decode-attention call is cut into work.  A *unit* is one
// (sequence, kv-head) pair, i.e. n contiguous K rows and n contiguous V rows.
// Units are cut into tiles of tile_rows rows; all tiles of all units form one
// line of T tiles which is divided evenly among NC persistent thread blocks.
// Each (thread block, unit) overlap is a *piece* and yields one partial result,
// stored at index unit + block.
struct DecodePlan {
    int tile_rows;   // rows per tile
    int tpu;         // tiles per unit = ceil(n / tile_rows)
    long long T;     // total tiles = units * tpu
    int NC;          // thread blocks launched
    int kernel;      // 1 = scalar, 2 = tensor-core
};

struct DecodeArgs {
    const void* q;        // [B][Hq][D] storage type
    const void* kplane;   // plane of the slot read: [B][Hkv][row_stride][D]
    const void* vplane;
    float* part_o;        // [units + NC][G][D]
    float* part_ml;       // [units + NC][G][2]  (max in log2 domain, sum)
    float* out;           // [B][Hq][D]
    int* status;          // device status word
    int n;                // rows cached per unit
    int row_stride;       // rows between units of a plane
    int capacity;         // rows a unit can hold (max_seq): lengths that grew on the device are cut off there
    int units;            // B * Hkv
    int G;                // q-heads per kv-head
    int D;
    int dtype;            // 0 bf16, 1 f32
    float scale_log2;     // softmax scale * log2(e)
    const int* unit_len;  // device, [units]: rows cached per unit when units differ (else nullptr and n holds)
    const int* n_extra;   // device int: rows grown since the launch was recorded (graph replay), or nullptr
    int safe_rows;        // rows per unit that no kernel possibly still in flight is writing
    bool programmatic;    // launch with programmatic stream serialization (early start, explicit wait)
    const void* k_new;    // [B][1][Hkv][D] rows the launch also appends (n already counts them), or nullptr
    const void* v_new;
    // No unit has more than two pieces (at least as many units as blocks): the split-K kernel merges
    // the two itself and writes `out`; no combine launch.  flags: [units] ints, zero between launches.
    bool finish_in_kernel;
    int* flags;
    long long plane_bytes;   // size of one plane: what a bounds-checking build checks tile offsets against
    unsigned long long wait_ns;   // limit of every wait inside the split-K kernels
    long long stall_tile;    // self-test only: the K/V copies of this tile of the line are withheld (-1: none)
    unsigned long long* trace;    // tracing build only: this launch's [kTraceBlocks][kTraceSlots] words, or nullptr
};

// Whether a launch of this plan over `units` units can finish inside the split-K kernel.
inline bool can_finish_in_kernel(const DecodePlan& plan, int units) { return units >= plan.NC; }

// Largest number of thread blocks any plan may use (sizes the partial buffers).
constexpr int kMaxCtas = 1024;

// Fill `plan` for the scalar kernel on a device with `sm_count` SMs.
// max_ctas <= 0 means automatic.  Host-only arithmetic (no CUDA call).
void plan_decode_scalar(int units, int n, int G, int D, int dtype, int sm_count, int max_ctas, DecodePlan* plan);

// Same for the tensor-core kernel (bf16 storage only).
void plan_decode_mma(int units, int n, int D, int sm_count, int max_ctas, DecodePlan* plan);

// One-time per-process kernel attribute set-up for the current device.
cudaError_t init_kernels();
cudaError_t init_mma_kernels();

// Encode the TMA tensor map of a bf16 pool seen as [total_rows][D]; `storage` is 128 bytes,
// 64-byte aligned, host memory.  tail = false: 64-row boxes (whole tiles); true: 16-row boxes (the
// partly filled last tile of a unit).
cudaError_t make_pool_tensor_map(void* storage, void* pool, long long total_rows, int D, bool tail);

// krow0 / vrow0: first row of the K / V plane in the pool-wide row numbering.
cudaError_t launch_decode_mma(const DecodeArgs& a, const DecodePlan& plan, const void* tensor_map,
                              const void* tensor_map_tail, long long krow0, long long vrow0, cudaStream_t stream);

// Tensor-core prefill attention (bf16, head size D = 64 or 128): q [B][T][Hq][D], out fp32 of the same shape.
cudaError_t init_prefill_kernels();
// `sched`: a device int for the kernel's work counter (zeroed on `stream` by the launch).
cudaError_t launch_prefill(const void* q, float* out, int* status, int* sched, const void* pool_tensor_map, int B, int T,
                           int Hq, int G, int D, int n, int row_stride, long long krow0, long long vrow0,
                           long long plane_rows, float scale_log2, int sm_count, long long l2_bytes, cudaStream_t stream);

// The same causal prefill attention for fp32 storage (plain fp32 kernel; see kvs_prefill_f32.cu).
cudaError_t launch_prefill_f32(const void* q, float* out, const void* kplane, const void* vplane, int B, int T, int Hq,
                               int G, int D, int n, int row_stride, float scale_log2, cudaStream_t stream);

// Strategy-search reductions (see kvs_search.cu).
constexpr int kMaxLayersSearch = 80;     // bound of the layer -> slot table handed to the finishing kernel
constexpr int kSearchMaxBlocks = 640;    // sizes the per-block partial buffers
constexpr int kCosineMaxBlocks = 4096;   // the same for the cosine reduction (three doubles per block)
// The sample means of a slab of positions go through scratch memory between the two passes; a slab is
// sized so that they stay in L2 (a fraction of its 126 MB).
constexpr long long kMeanSlabBytes = 48ll << 20;
// Scratch the distance reduction needs for `n_slots` cache slots of `positions` = 2 * Hkv * n * D elements.
size_t distance_scratch_bytes(int n_slots, long long positions);
// *launches receives the number of kernels launched (two per slab and two to finish), all on `stream`: the
// distance pass of a slab runs beside the mean pass of the next, which is launched behind it as a programmatic
// dependent.
cudaError_t launch_layer_distances(const void* pool, long long plane_bytes, const int* slot_of_layer, int L, int n_slots,
                                   int B, int Hkv, int n, int row_stride, int D, int dtype, float* scratch,
                                   size_t scratch_bytes, float* dist, int sm_count, int* launches, cudaStream_t stream);
cudaError_t launch_mean_cosine(const void* a, const void* b, int S, long long dim, int dtype, double* partial,
                               float* out, int sm_count, cudaStream_t stream);

cudaError_t launch_append(const void* k, const void* v, void* kplane, void* vplane, int B, int n_new, int Hkv,
                          int row_bytes, int row_stride, int len0, const int* unit_len, const int* n_extra, int capacity, int* status,
                          long long plane_bytes, bool programmatic, cudaStream_t stream);
cudaError_t launch_replay_advance(int* n_extra, bool programmatic, cudaStream_t stream);

// Ragged slots (rows evicted by an outside intra-layer method).
//   launch_evict:   per unit u, rows keep[u*keep_stride + j], j < counts[u], move to rows 0..counts[u]-1
//                   (K and V planes); old lengths are old_len[u] or, if old_len is nullptr, old_uniform
//   launch_set_len: unit_len[u] = counts[u];  launch_add_len: unit_len[u] += delta
cudaError_t launch_evict(void* kplane, void* vplane, const int* keep, const int* counts, const int* old_len,
                         int old_uniform, int units, int keep_stride, int row_bytes, int row_stride, int* status,
                         bool programmatic, cudaStream_t stream);
cudaError_t launch_set_len(int* unit_len, const int* counts, int units, bool programmatic, cudaStream_t stream);
cudaError_t launch_add_len(int* unit_len, int delta, int units, bool programmatic, cudaStream_t stream);
cudaError_t launch_decode_scalar(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream);
cudaError_t launch_combine(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream);
// One thread waits, with the given limit, on a barrier nothing arrives at; *status receives the
// time-out code and *waited_ns (device, may be null) how long the wait lasted.
cudaError_t launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, unsigned long long* waited_ns,
                                         cudaStream_t stream);
// Whether this library was compiled with -DKVS_TRACE (kernels stamp their timeline into DecodeArgs::trace).
bool is_tracing_build();
// Words one attention call (split-K kernel + combine kernel) occupies in a trace buffer: 160 rows of 32 words
// (rows 0..147: the split-K kernel's blocks; rows 150 / 151: the first / last block of the combine kernel).
constexpr int kTraceLaunchWords = 160 * 32;
// Whether this library was compiled with -DKVS_DEBUG_BOUNDS, and a launch that makes its offset check
// record one violation (KVS_ERR_BOUNDS in *status) without touching memory.
bool is_bounds_checking_build();
cudaError_t launch_bounds_selftest(int* status, cudaStream_t stream);
cudaError_t launch_read_roof(const void* src, size_t bytes, unsigned long long* checksum, int sm_count,
                             cudaStream_t stream);

}  // namespace kvs
