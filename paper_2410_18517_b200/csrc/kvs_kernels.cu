// sm_100a kernels of the shared-KV decode path:
//   kv_append_kernel      new-token K/V rows -> slot planes (16-byte vectors)
//   decode_splitk_scalar  persistent split-K attention, bulk-copy ring, fp32 FMA
//   decode_combine_kernel merges the pieces of every (sequence, kv-head) unit
//   read_roof_kernel      the same ring with no arithmetic (bandwidth ceiling)
#include "kvs_device.cuh"
#include "kvs_kernels.h"

#include <algorithm>

namespace kvs {

// --------------------------------------------------------------------------------------
// K1: append.  k/v: [B][n_new][Hkv][row] -> plane [B][Hkv][row_stride][row], rows len0...
// One thread moves 16 bytes.  blockIdx.y = 0 copies K, 1 copies V.
// --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) kv_append_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v,
                                                        uint4* __restrict__ kplane, uint4* __restrict__ vplane,
                                                        long long total_vecs, int n_new, int Hkv, int row_vecs,
                                                        int row_stride, int len0, const int* __restrict__ unit_len,
                                                        const int* __restrict__ n_extra, int capacity, int* status,
                                                        long long plane_vecs) {
    pdl_launch_dependents();
    pdl_wait();
    if (n_extra) len0 += *n_extra;   // replayed launch: the slot has grown since the launch was recorded
    if (!unit_len && len0 + n_new > capacity) {   // can only happen in a replay that outran the capacity
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicExch(status, 4);
        return;
    }
    const uint4* __restrict__ src = blockIdx.y == 0 ? k : v;
    uint4* __restrict__ dst = blockIdx.y == 0 ? kplane : vplane;
    // where vector idx of the source goes in the plane (-1: nowhere)
    auto target = [&](long long idx) -> long long {
        const int c = (int)(idx % row_vecs);
        long long r = idx / row_vecs;
        const int h = (int)(r % Hkv);
        r /= Hkv;
        const int t = (int)(r % n_new);
        const long long b = r / n_new;
        const int first = unit_len ? unit_len[b * Hkv + h] : len0;   // ragged slots append per unit
        if (first + t >= capacity) {   // only a replay that outran the capacity gets here
            if (c == 0) atomicExch(status, 4);
            return -1;
        }
        const long long drow = (b * Hkv + h) * (long long)row_stride + first + t;
        if (!KVS_BOUNDS_OK(drow * row_vecs + c, 1, plane_vecs, status)) return -1;
        return drow * row_vecs + c;
    };
    // four vectors per thread and turn, all four loads issued before the first store (a prompt's worth of
    // rows is a plain copy at memory speed; one token's worth fits in the first turn of a few blocks)
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    for (; idx < total_vecs; idx += 4 * stride) {
        uint4 x[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (idx + i * stride < total_vecs) x[i] = __ldcs(src + idx + i * stride);      // read once
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (idx + i * stride >= total_vecs) break;
            const long long d = target(idx + i * stride);
            if (d >= 0) dst[d] = x[i];
        }
    }
}

cudaError_t launch_append(const void* k, const void* v, void* kplane, void* vplane, int B, int n_new, int Hkv,
                          int row_bytes, int row_stride, int len0, const int* unit_len, const int* n_extra, int capacity, int* status,
                          long long plane_bytes, bool programmatic, cudaStream_t stream) {
    const int row_vecs = row_bytes / 16;
    const long long total = (long long)B * n_new * Hkv * row_vecs;
    const long long blocks = std::min<long long>((total + 255) / 256, 148 * 16);
    dim3 grid((unsigned)blocks, 2);
    return launch_kernel(kv_append_kernel, grid, dim3(256), 0, stream, programmatic, (const uint4*)k, (const uint4*)v,
                         (uint4*)kplane, (uint4*)vplane, total, n_new, Hkv, row_vecs, row_stride, len0, unit_len, n_extra, capacity,
                         status, plane_bytes / 16);
}

// --------------------------------------------------------------------------------------
// Eviction: keep only the listed rows of every unit, moved to the front in order.  One block
// per (unit, K or V plane); rows go through shared memory 64 at a time, and because the list
// is strictly ascending (keep[j] >= j) a later chunk never reads a row an earlier chunk wrote.
// A list that is not ascending or points past the unit's length sets the status word to 1
// (invalid argument) and the offending entry is treated as "keep the row already there".
// --------------------------------------------------------------------------------------
constexpr int kEvictChunk = 64;

__global__ void __launch_bounds__(256) kv_evict_kernel(uint4* __restrict__ kplane, uint4* __restrict__ vplane,
                                                       const int* __restrict__ keep, const int* __restrict__ counts,
                                                       const int* __restrict__ old_len, int old_uniform, int keep_stride,
                                                       int row_vecs, int row_stride, int* status) {
    __shared__ uint4 buf[kEvictChunk * 32];   // 64 rows of up to 512 bytes
    pdl_launch_dependents();
    pdl_wait();
    const int u = blockIdx.x;
    uint4* base = (blockIdx.y == 0 ? kplane : vplane) + (long long)u * row_stride * row_vecs;
    const int cnt = counts[u];
    const int old = old_len ? old_len[u] : old_uniform;
    const int* list = keep + (long long)u * keep_stride;
    for (int c0 = 0; c0 < cnt; c0 += kEvictChunk) {
        const int rows = min(kEvictChunk, cnt - c0);
        for (int idx = threadIdx.x; idx < rows * row_vecs; idx += blockDim.x) {
            const int j = idx / row_vecs, v = idx - j * row_vecs;
            int src = list[c0 + j];
            const bool bad = src >= old || src < c0 + j || (c0 + j > 0 && list[c0 + j - 1] >= src);
            if (bad) {
                if (v == 0) atomicExch(status, 1);
                src = c0 + j;
            }
            if (!KVS_BOUNDS_OK(src, 1, row_stride, status)) src = 0;
            buf[idx] = base[(long long)src * row_vecs + v];
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < rows * row_vecs; idx += blockDim.x)
            if (KVS_BOUNDS_OK((long long)c0 * row_vecs + idx, 1, (long long)row_stride * row_vecs, status))
                base[(long long)c0 * row_vecs + idx] = buf[idx];
        __syncthreads();
    }
}

__global__ void set_len_kernel(int* __restrict__ unit_len, const int* __restrict__ counts, int units) {
    pdl_launch_dependents();
    pdl_wait();
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < units) unit_len[u] = counts[u];
}

__global__ void add_len_kernel(int* __restrict__ unit_len, int delta, int units) {
    pdl_launch_dependents();
    pdl_wait();
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < units) unit_len[u] += delta;
}

cudaError_t launch_evict(void* kplane, void* vplane, const int* keep, const int* counts, const int* old_len,
                         int old_uniform, int units, int keep_stride, int row_bytes, int row_stride, int* status,
                         bool programmatic, cudaStream_t stream) {
    return launch_kernel(kv_evict_kernel, dim3(units, 2), dim3(256), 0, stream, programmatic, (uint4*)kplane,
                         (uint4*)vplane, keep, counts, old_len, old_uniform, keep_stride, row_bytes / 16, row_stride,
                         status);
}

cudaError_t launch_set_len(int* unit_len, const int* counts, int units, bool programmatic, cudaStream_t stream) {
    return launch_kernel(set_len_kernel, dim3((units + 127) / 128), dim3(128), 0, stream, programmatic, unit_len, counts,
                         units);
}

__global__ void replay_advance_kernel(int* n_extra) {
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) *n_extra += 1;
}

cudaError_t launch_replay_advance(int* n_extra, bool programmatic, cudaStream_t stream) {
    return launch_kernel(replay_advance_kernel, dim3(1), dim3(32), 0, stream, programmatic, n_extra);
}

cudaError_t launch_add_len(int* unit_len, int delta, int units, bool programmatic, cudaStream_t stream) {
    return launch_kernel(add_len_kernel, dim3((units + 127) / 128), dim3(128), 0, stream, programmatic, unit_len, delta,
                         units);
}

// --------------------------------------------------------------------------------------
// Work decomposition shared by the split-K kernel and the combine kernel.
// Thread block c owns tiles [c*T/NC, (c+1)*T/NC) of the line of T tiles.
// --------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ long long first_tile_of_cta(long long c, long long T, int NC) {
    return (c * T) / NC;
}
// The thread block that owns tile gt (inverse of the above).
__host__ __device__ __forceinline__ int cta_of_tile(long long gt, long long T, int NC) {
    return (int)(((gt + 1) * NC + T - 1) / T - 1);
}

// --------------------------------------------------------------------------------------
// K2a: scalar split-K decode attention.
//
// Shapes: T = storage type, D = head size, G = q-heads per kv-head.
// A token row is RB = D*sizeof(T) bytes and is read by LPR = RB/16 lanes, 16 bytes
// each, so a warp reads 32/LPR consecutive rows (512 contiguous bytes) per shared-memory
// load: conflict-free without any swizzle.  A tile is 16 KiB of K and 16 KiB of V rows,
// fetched by two 1-D bulk copies that complete on the stage's mbarrier.  Warp 8 is the
// producer (one elected lane issues copies); warps 0..7 consume.
//
// Every group of LPR lanes keeps its own online-softmax state (running max, sum and
// un-normalised output chunk) over the rows it is dealt, so no block-wide
// synchronisation happens per tile; groups are merged once per piece.
// --------------------------------------------------------------------------------------
#ifndef KVS_CONSUMER_WARPS
#define KVS_CONSUMER_WARPS 8
#endif
constexpr int kConsumerWarps = KVS_CONSUMER_WARPS;
constexpr int kConsumerThreads = kConsumerWarps * 32;
// Tile size, ring depth and blocks per SM of the scalar kernel for groups of 1 or 2 q-heads
// (compile-time; the defaults are the measured best on B200).
#ifndef KVS_TILE_BYTES
#define KVS_TILE_BYTES 32768
#endif
#ifndef KVS_STAGES
#define KVS_STAGES 3
#endif
#ifndef KVS_BLOCKS_PER_SM
#define KVS_BLOCKS_PER_SM 1
#endif
constexpr int kTileBytes = KVS_TILE_BYTES;  // per K tile and per V tile
// One geometry serves every launch size.  (A second one for multi-gigabyte launches, 5 stages of 16 KiB tiles,
// was 3 % ahead when it was introduced and 5-9 % behind the default by the time the kernel finished its units
// itself: 13B shape, same box, builds alternating, 16.56 against 15.09 ms per step at 1.5-1.7 GHz, 15.55 against
// 14.86 at 1.84 GHz.  Sixteen consumer warps instead of eight repair that geometry (15.83 / 14.86) but add
// nothing to this one: 15.10 against 15.09 ms on the 13B shape, 2.566 against 2.548 on the 7B shape.)
template <typename T, int D, int G>
struct ScalarShape {
    static constexpr int TILE = kTileBytes;
    static constexpr int RB = D * (int)sizeof(T);
    static constexpr int LPR = RB / 16;
    static constexpr int EPL = 16 / (int)sizeof(T);
    static constexpr int WARPS = kConsumerWarps;          // consumer warps
    static constexpr int CTHREADS = WARPS * 32;           // consumer threads
    static constexpr int THREADS = CTHREADS + 64;         // + the producer warp and the hand-over warp
    static constexpr int GPW = 32 / LPR;                  // lane groups per warp
    static constexpr int NG = WARPS * GPW;                // lane groups per block
    static constexpr int TN = TILE / RB;                  // rows per tile
    static constexpr int R = TN / NG;                     // rows per group per tile
    static constexpr int STAGES = (G <= 2) ? KVS_STAGES : (6 * 16384) / kTileBytes;
    static constexpr int MIN_BLOCKS = (G <= 2) ? KVS_BLOCKS_PER_SM : 1;
    static constexpr int QBYTES = G * RB;
    static constexpr int STAGE_BYTES = 2 * TILE + QBYTES;
    static constexpr int SCRATCH_FLOATS = NG * (D + 2);
    // groups of more than four q-heads keep the piece's queries in shared memory instead of registers
    static constexpr int QKEEP_BYTES = G > 4 ? QBYTES : 0;
    static constexpr int HANDOVER_FLOATS = G * (D + 2);   // another block's piece of a cut unit: [q-head][D + 2]
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SCRATCH_FLOATS * 4 + (2 * STAGES + 2) * 8 + 16 + QKEEP_BYTES +
                                      HANDOVER_FLOATS * 4;
    static_assert(R >= 1 && R <= LPR && (R & (R - 1)) == 0, "rows per group must be a power of two <= lanes per row");
    static_assert(TN % NG == 0, "tile rows must divide evenly among lane groups");
};

template <int N>
struct Log2 {
    static constexpr int value = 1 + Log2<N / 2>::value;
};
template <>
struct Log2<1> {
    static constexpr int value = 0;
};

// Sum NV per-lane partial sums over a group of lanes by recursive halving: after the
// call, the lane whose index within the group has top bits i holds the full sum of
// value i.  OFF is the current xor distance (starts at lanes-per-group / 2).
template <int NV, int OFF>
__device__ __forceinline__ float reduce_transpose(float (&v)[NV], int lig) {
    if constexpr (NV == 1) {
        float x = v[0];
#pragma unroll
        for (int o = OFF; o >= 1; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        return x;
    } else {
        constexpr int H = NV / 2;
        const bool upper = (lig & OFF) != 0;
        float w[H];
#pragma unroll
        for (int k = 0; k < H; ++k) {
            const float send = upper ? v[k] : v[k + H];
            const float keep = upper ? v[k + H] : v[k];
            w[k] = keep + __shfl_xor_sync(0xffffffffu, send, OFF);
        }
        return reduce_transpose<H, OFF / 2>(w, lig);
    }
}

struct ScalarKernelArgs {
    const char* q;
    const char* kplane;
    const char* vplane;
    float* part_o;
    float* part_ml;
    int* status;
    int n;
    int row_stride;
    int tpu;
    long long T;
    float scale_log2;
    int safe_rows;  // rows of every unit that no kernel possibly still running writes
    const int* unit_len;  // per-unit row counts of a ragged slot, or nullptr (then n holds for all)
    const int* n_extra;   // graph replay: rows every slot has grown by since the launch was recorded, or nullptr
    int units;
    int cap;              // rows a unit can hold: lengths that grew on the device are cut off there
    const char* k_new;    // the step's new rows, appended by this kernel (n counts them), or nullptr
    const char* v_new;
    // Finishing inside this kernel (no combine launch): set when no unit has more than two pieces.
    float* out;           // [units][G][D] final results, or nullptr: every piece goes to part_o / part_ml
    int* flags;           // [units], all zero between launches: 1 = the unit's second piece is in part_o / part_ml
    long long plane_bytes;  // size of one plane (what a bounds-checking build checks tile offsets against)
    unsigned long long wait_ns;   // limit of every wait inside the kernel
    long long stall_tile;         // self-test only: the K/V copies of this tile are withheld (-1: none)
    unsigned long long* trace;    // tracing build: this launch's rows of time stamps, or nullptr
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(ScalarShape<T, D, G>::THREADS, ScalarShape<T, D, G>::MIN_BLOCKS)
    decode_splitk_scalar(const ScalarKernelArgs a_in) {
    using S = ScalarShape<T, D, G>;
    ScalarKernelArgs a = a_in;
    unsigned long long* tr = a.trace ? a.trace + (size_t)blockIdx.x * kTraceSlots : nullptr;
    if (threadIdx.x == 0) {
        KVS_TRACE_STAMP(tr, kTrEntry);
        KVS_TRACE_VALUE(tr, kTrSm, sm_id());
    }
    bool over = false;    // a replayed launch with an append that would pass the capacity
    if (a.n_extra != nullptr) {
        // A replayed launch: the lengths recorded with it have grown on the device since.  The
        // counter is stable here without a wait: the host gives the first launch after every write
        // of the counter a full dependency, so that write is complete before any reader starts.
        over = a.n + *a.n_extra > a.cap;
        a.n = min(a.n + *a.n_extra, a.cap);   // a replay that outran the capacity appended nothing more
        a.tpu = (a.n + S::TN - 1) / S::TN;
        a.T = (long long)a.units * a.tpu;
    }
    constexpr int kTile = S::TILE;
    constexpr int RB = S::RB, LPR = S::LPR, EPL = S::EPL, NG = S::NG, TN = S::TN, R = S::R, STAGES = S::STAGES;
    constexpr int SH = Log2<LPR>::value - Log2<R>::value;  // lane-in-group >> SH = row index held after the reduction
    // q-heads taken together over a staged tile (bf16 lanes hold eight elements per head, fp32 lanes four)
    constexpr int GP = G > 4 ? (sizeof(T) == 2 ? 2 : 4) : G;

    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* stage_base = smem;
    float* scratch = reinterpret_cast<float*>(smem + STAGES * S::STAGE_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(scratch + S::SCRATCH_FLOATS);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* tail_bar = empty_bar + STAGES;         // every consumer thread has written this block's second-piece partial
    uint64_t* head_bar = tail_bar + 1;               // the next block's second-piece partial is in handover[]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(head_bar + 1);
    uint4* q_keep = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(head_bar + 1) + 16);   // G > 4 only
    float* handover = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(q_keep) + S::QKEEP_BYTES);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int NC = gridDim.x;
    const long long t0 = first_tile_of_cta(blockIdx.x, a.T, NC);
    const long long t1 = first_tile_of_cta(blockIdx.x + 1, a.T, NC);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], S::WARPS);
        }
        mbar_init(tail_bar, S::CTHREADS);
        mbar_init(head_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // second word: bounds the producer's drain after a give-up
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == S::WARPS) {
        // ------------------------------ producer ------------------------------
        // Lane 0 issues the copies; the whole warp stores the step's new rows when the launch
        // carries an append.
        {
            // Issue the copies of tile `gt` into stage `st`.  kv / qpart select which of the
            // stage's copies are issued now; the barrier is armed with the stage's full byte
            // count by whichever call comes first (arm = true).
            auto issue = [&](long long gt, int st, bool arm, bool kv, bool qpart) {
                const long long u = gt / a.tpu;
                const int ti = (int)(gt - u * a.tpu);
                const int row0 = ti * TN;
                const int n_u = a.unit_len ? min(a.unit_len[u], a.cap) : a.n;
                const int rows = max(0, min(TN, n_u - row0));     // a ragged unit may end before this tile
                const uint32_t bytes = (uint32_t)rows * RB;
                const bool with_q = (gt == t0) || (ti == 0);
                unsigned char* sb = stage_base + st * S::STAGE_BYTES;
                if (arm) {
                    const uint32_t total = 2 * bytes + (with_q ? S::QBYTES : 0);
                    if (total) mbar_arrive_expect_tx(&full_bar[st], total);
                    else mbar_arrive(&full_bar[st]);
                }
                if (kv && bytes && gt != a.stall_tile) {
                    long long off = (u * a.row_stride + row0) * (long long)RB;
                    if (!KVS_BOUNDS_OK(off, bytes, a.plane_bytes, a.status) || !KVS_BOUNDS_OK(u, 1, a.units, a.status)) off = 0;
                    bulk_g2s(sb, a.kplane + off, bytes, &full_bar[st]);
                    bulk_g2s(sb + kTile, a.vplane + off, bytes, &full_bar[st]);
                }
                if (qpart && with_q)
                    bulk_g2s(sb + 2 * kTile, a.q + (KVS_BOUNDS_OK(u, 1, a.units, a.status) ? u : 0) * (long long)S::QBYTES,
                             S::QBYTES, &full_bar[st]);
            };
            // Before the preceding kernel in the stream is known to have finished, only K/V
            // tiles made entirely of rows that no kernel still in flight can be writing are
            // fetched (rows below safe_rows); q and everything else come after the wait.
            int npre = 0;
            if (lane == 0) {
                for (; npre < STAGES && t0 + npre < t1; ++npre) {
                    const long long gt = t0 + npre;
                    const int ti = (int)(gt % a.tpu);
                    if ((long long)(ti + 1) * TN > a.safe_rows) break;
                    issue(gt, npre, true, true, false);
                }
            }
            if (lane == 0) KVS_TRACE_STAMP(tr, kTrProducerPre);
            pdl_wait();
            if (lane == 0) KVS_TRACE_STAMP(tr, kTrProducerGo);
            pdl_launch_dependents();
            // first the queries of the tiles already fetched (the consumers wait for nothing else), then the new rows
            if (lane == 0)
                for (int j = 0; j < npre; ++j) issue(t0 + j, j, false, false, true);
            if (a.k_new != nullptr) {
                if (!over)
                    store_new_rows<RB>(lane, t0, t1, a.tpu, a.n, a.row_stride, a.k_new, a.v_new, const_cast<char*>(a.kplane),
                                       const_cast<char*>(a.vplane), a.plane_bytes, a.units, a.status);
                else if (lane == 0 && blockIdx.x == 0)
                    atomicExch(a.status, 4);
            }
            if (lane != 0) return;
            int it = npre;
            bool ok = true;
            for (long long gt = t0 + npre; gt < t1 && ok; ++gt, ++it) {
                const int st = it % STAGES;
                if (it >= STAGES) ok = mbar_wait_bounded(&empty_bar[st], ((it / STAGES) - 1) & 1, abort_flag, a.status, a.wait_ns);
                if (!ok) break;
                issue(gt, st, true, true, true);
            }
            if (!ok) {
                // Gave up: still wait (bounded) for copies already issued, so that none
                // is in flight into this block's shared memory when it exits.
                for (int j = max(0, it - STAGES); j < it; ++j)
                    mbar_wait_bounded(&full_bar[j % STAGES], (j / STAGES) & 1, abort_flag + 1, a.status, a.wait_ns);
            }
        }
        return;
    }

    if (warp == S::WARPS + 1) {
        // ------------------ hand-over of units that are cut between two blocks ------------------
        // Only when the kernel finishes the units itself (a.out set).  The global round trips of the
        // hand-over are made here, beside the stream: this warp raises the flag of the unit whose
        // second piece this block computed first, and fetches the second piece of the unit whose
        // first piece this block computes last, so that the consumers find it in shared memory.
        if (a.out == nullptr || t0 >= t1) return;
        const bool has_tail = (t0 % a.tpu) != 0, has_head = (t1 % a.tpu) != 0;
        if (!has_tail && !has_head) return;
        pdl_wait();   // the flags are back to zero only once the previous launch has completed
        if (has_tail) {
            if (!mbar_wait_bounded(tail_bar, 0, abort_flag, a.status, a.wait_ns)) return;
            if (lane == 0) st_release_gpu(a.flags + t0 / a.tpu, 1);
        }
        if (has_head) {
            const long long u = (t1 - 1) / a.tpu;
            int ok = 1;
            if (lane == 0) ok = flag_wait_bounded(a.flags + u, 1, abort_flag, a.status, a.wait_ns) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            __syncwarp();    // lane 0's acquire comes before every lane's loads of the piece
            if (!ok) return;
            // written by another SM during this launch: read past L1
            const long long pt = u + blockIdx.x + 1;
            for (int i = lane; i < G * D; i += 32) handover[(i / D) * (D + 2) + (i % D)] = __ldcg(a.part_o + pt * G * D + i);
            for (int i = lane; i < G * 2; i += 32) handover[(i >> 1) * (D + 2) + D + (i & 1)] = __ldcg(a.part_ml + pt * G * 2 + i);
            __syncwarp();
            if (lane == 0) {
                a.flags[u] = 0;          // this block is the flag's only reader
                mbar_arrive(head_bar);
            }
        }
        return;
    }

    // ---------------------------------- consumers ----------------------------------
    pdl_wait();               // partial results of the previous call may still be read until here
    if (tid == 0) KVS_TRACE_STAMP(tr, kTrConsumerGo);
    pdl_launch_dependents();
    int trace_piece = 0;
    const int lig = lane & (LPR - 1);                 // lane within its row group
    const int grp = warp * S::GPW + lane / LPR;       // row group within the block
    const int my_i = lig >> SH;                       // row (of the R) whose score this lane ends up holding

    int it = 0;
    long long gt = t0;
    while (gt < t1) {
        const long long u = gt / a.tpu;
        const int ti0 = (int)(gt - u * a.tpu);
        const int piece_tiles = (int)min((long long)(a.tpu - ti0), t1 - gt);
        const int n_u = a.unit_len ? min(a.unit_len[u], a.cap) : a.n;

        float qf[G > 4 ? 1 : G][EPL];   // larger groups read their queries from q_keep, four heads at a time
        float m[G], lsum[G], acc[G][EPL];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            m[g] = -1.0e30f;
            lsum[g] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
        }

        for (int k = 0; k < piece_tiles; ++k, ++it) {
            const int st = it % STAGES;
            if (!mbar_wait_bounded(&full_bar[st], (it / STAGES) & 1, abort_flag, a.status, a.wait_ns)) return;
            if (tid == 0 && it == 0) KVS_TRACE_STAMP(tr, kTrFirstTile);
            const unsigned char* ks = stage_base + st * S::STAGE_BYTES;
            const unsigned char* vs = ks + kTile;
            if (k == 0) {
                const unsigned char* qs = vs + kTile;
                if constexpr (G > 4) {
                    // every warp is past the previous piece's last tile (the merge barriers), so the
                    // buffer is free; the stage that carries q is released after this tile
                    for (int c = tid; c < G * LPR; c += S::CTHREADS) q_keep[c] = reinterpret_cast<const uint4*>(qs)[c];
                    named_bar_sync(2, S::CTHREADS);
                } else {
#pragma unroll
                    for (int g = 0; g < (G > 4 ? 1 : G); ++g) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(qs + g * RB + lig * 16);
                        Unpack<T>::run(raw, qf[g]);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) qf[g][e] *= a.scale_log2;
                    }
                }
            }
            const int valid = min(TN, n_u - (ti0 + k) * TN);   // <= 0 for tiles past a ragged unit's end
            if (valid <= 0) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
                continue;
            }

            // The q-heads of the group are taken GP at a time over the staged tile (all of them when
            // the group has at most four): with eight heads at once the scores and weights of a tile
            // (2 * 8 * R values) and the queries would not fit in registers beside the running state.
#pragma unroll
            for (int g0 = 0; g0 < G; g0 += GP) {
                // this pass's queries: registers, or (large groups) this lane's chunk from q_keep
                float qp[GP][EPL];
#pragma unroll
                for (int g = 0; g < GP; ++g) {
                    if constexpr (G > 4) {
                        Unpack<T>::run(q_keep[(g0 + g) * LPR + lig], qp[g]);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) qp[g][e] *= a.scale_log2;
                    } else {
#pragma unroll
                        for (int e = 0; e < EPL; ++e) qp[g][e] = qf[g0 + g][e];
                    }
                }
                // scores: partial dot products of this lane's 16-byte chunk
                float s[GP][R];
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const int row = grp + NG * i;
                    const uint4 raw = *reinterpret_cast<const uint4*>(ks + row * RB + lig * 16);
                    float kf[EPL];
                    Unpack<T>::run(raw, kf);
#pragma unroll
                    for (int g = 0; g < GP; ++g) {
                        float d = 0.f;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) d = fmaf(qp[g][e], kf[e], d);
                        s[g][i] = d;
                    }
                }
                // online softmax per q-head, local to the lane group
                float p[GP][R];
                const bool mine_valid = (grp + NG * my_i) < valid;
#pragma unroll
                for (int g = 0; g < GP; ++g) {
                    float sv = reduce_transpose<R, LPR / 2>(s[g], lig);
                    sv = mine_valid ? sv : -INFINITY;
                    float tmax = sv;
#pragma unroll
                    for (int o = LPR / 2; o >= LPR / R; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
                    const float m_new = fmaxf(m[g0 + g], tmax);
                    const float alpha = fast_exp2(m[g0 + g] - m_new);
                    const float pv = fast_exp2(sv - m_new);
                    m[g0 + g] = m_new;
                    lsum[g0 + g] = lsum[g0 + g] * alpha + pv;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[g0 + g][e] *= alpha;
#pragma unroll
                    for (int i = 0; i < R; ++i) p[g][i] = __shfl_sync(0xffffffffu, pv, i << SH, LPR);
                }
                // weighted sum of value rows
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const int row = grp + NG * i;
                    if (row < valid) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(vs + row * RB + lig * 16);
                        float vf[EPL];
                        Unpack<T>::run(raw, vf);
#pragma unroll
                        for (int g = 0; g < GP; ++g)
#pragma unroll
                            for (int e = 0; e < EPL; ++e) acc[g0 + g][e] = fmaf(p[g][i], vf[e], acc[g0 + g][e]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[st]);
        }

        // ---- end of piece: merge the NG lane groups, one q-head at a time ----
        // With a.out set (no unit has more than two pieces) the kernel finishes the units itself: a unit
        // that lies inside this block's share is normalised and written out; of a unit cut in two the
        // second piece, which is the FIRST piece of the next block and so done early in the launch, goes
        // to part_o / part_ml and the hand-over warp raises the unit's flag; the block that holds the
        // first piece comes to it LAST, by when its hand-over warp has fetched the second piece into
        // shared memory; it merges the two in piece order and writes the result.
        const long long pid = u + blockIdx.x;
        if (tid == 0 && trace_piece < 8) KVS_TRACE_STAMP(tr, kTrPiece + 2 * trace_piece);
        const bool finish = a.out != nullptr;
        const bool whole = finish && ti0 == 0 && piece_tiles == a.tpu;
        const bool head = finish && ti0 == 0 && piece_tiles < a.tpu;
        const bool tail = finish && ti0 > 0;
        if (head && !mbar_wait_bounded(head_bar, 0, abort_flag, a.status, a.wait_ns)) return;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            // lanes with equal top bits hold duplicates of lsum; add across the R distinct ones
            float l = lsum[g];
#pragma unroll
            for (int o = LPR / 2; o >= LPR / R; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            named_bar_sync(1, S::CTHREADS);  // scratch free again
            float* row = scratch + grp * (D + 2);
#pragma unroll
            for (int e = 0; e < EPL; ++e) row[lig * EPL + e] = acc[g][e];
            if (lig == 0) {
                row[D] = m[g];
                row[D + 1] = l;
            }
            named_bar_sync(1, S::CTHREADS);
            for (int d = tid; d < D; d += S::CTHREADS) {
                float M = -1.0e30f;
#pragma unroll
                for (int j = 0; j < NG; ++j) M = fmaxf(M, scratch[j * (D + 2) + D]);
                float o = 0.f, den = 0.f;
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    const float w = fast_exp2(scratch[j * (D + 2) + D] - M);
                    o = fmaf(w, scratch[j * (D + 2) + d], o);
                    den = fmaf(w, scratch[j * (D + 2) + D + 1], den);
                }
                if (whole) {
                    a.out[(u * G + g) * D + d] = o / den;
                } else if (head) {
                    const float* hv = handover + g * (D + 2);      // the unit's second piece
                    const float Mx = fmaxf(M, hv[D]);
                    const float w0 = fast_exp2(M - Mx), w1 = fast_exp2(hv[D] - Mx);
                    a.out[(u * G + g) * D + d] = fmaf(w1, hv[d], w0 * o) / fmaf(w1, hv[D + 1], w0 * den);
                } else if (KVS_BOUNDS_OK(pid, 1, a.units + (long long)gridDim.x, a.status)) {
                    a.part_o[(pid * G + g) * D + d] = o;
                    if (d == 0) {
                        a.part_ml[(pid * G + g) * 2] = M;
                        a.part_ml[(pid * G + g) * 2 + 1] = den;
                    }
                }
            }
        }
        if (tail) mbar_arrive(tail_bar);   // this thread's part of the piece is written
        if (tid == 0 && trace_piece < 8) KVS_TRACE_STAMP(tr, kTrPiece + 2 * trace_piece + 1);
        ++trace_piece;
        gt += piece_tiles;
    }
    if (tid == 0) {
        KVS_TRACE_STAMP(tr, kTrEnd);
        KVS_TRACE_VALUE(tr, kTrPieces, trace_piece);
    }
}

// --------------------------------------------------------------------------------------
// K3: combine.  One WARP per (unit, q-head): out = sum_c w_c o_c / sum_c w_c l_c with
// w_c = 2^(m_c - M), M = max_c m_c over the pieces c of the unit.  The output vectors are always
// added in piece order and the denominators in a fixed lane order, so the result does not
// depend on which block finished first.
// Lane j fetches the (max, sum) pair of piece j (independent loads, one round trip to L2) while
// the output vectors of the first pieces are already requested; weights travel by shuffle;
// each lane owns D/32 consecutive output columns.  No shared memory and at most 48 registers:
// the whole grid (eight items per block) becomes resident beside the split-K kernel it follows
// (whose block leaves 14-34 K registers of the SM free), so that the split-K kernel of the NEXT
// call, which may only start once every block of this grid has started, can move onto each SM
// the moment the running split-K block leaves it.
// --------------------------------------------------------------------------------------
// This build serves calls whose units have at most two pieces (every block's share is at least a
// unit long): eight items per block, two vectors requested early.  Longer units: decode_combine_long_kernel.
template <int D, int PRE, int kCombineWarps>
__global__ void __launch_bounds__(kCombineWarps * 32, 5)
    decode_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, float* __restrict__ out,
                          int G, int tpu, long long T, int NC, const int* __restrict__ n_extra, int n, int tile_rows,
                          int units, int cap, int* status, unsigned long long* trace) {
    constexpr int VEC = D / 32;
    struct __align__(VEC * 4) Vec {
        float v[VEC];
    };
    unsigned long long* tr = (trace && threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))
                                 ? trace + (size_t)(150 + (blockIdx.x != 0)) * kTraceSlots : nullptr;
    KVS_TRACE_STAMP(tr, 0);
    pdl_launch_dependents();
    pdl_wait();
    KVS_TRACE_STAMP(tr, 1);
    if (n_extra) {   // replayed launch: recompute the tile line from the grown length
        tpu = (min(n + *n_extra, cap) + tile_rows - 1) / tile_rows;
        T = (long long)units * tpu;
    }
    const long long item = (long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (item >= (long long)units * G) return;
    const long long u = item / G;
    const int g = (int)(item - u * G);
    const int c0 = cta_of_tile(u * tpu, T, NC);
    int np = cta_of_tile((u + 1) * tpu - 1, T, NC) - c0 + 1;             // pieces of this unit
#ifdef KVS_DEBUG_BOUNDS
    if (!KVS_BOUNDS_OK(u + c0, np, (long long)units + NC, status)) np = 1;
#endif
    const float2* ml = reinterpret_cast<const float2*>(part_ml) + (u + c0) * G + g;   // piece c: ml[c * G]
    const Vec* po = reinterpret_cast<const Vec*>(part_o + ((u + c0) * G + g) * D) + lane;   // piece c: po[c * G * 32]
    const int pstride = G * 32;     // offsets within one unit's pieces fit 32 bits
    // first chunk of (max, sum) pairs and, in the same round trip, the first PRE output vectors
    const float2 v0 = lane < np ? ml[lane * G] : make_float2(-1.0e30f, 0.f);
    Vec pre[PRE];
#pragma unroll
    for (int c = 0; c < PRE; ++c)
        if (c < np) pre[c] = po[c * pstride];
    float M = v0.x;
    for (int cb = 32; cb < np; cb += 32)
        if (cb + lane < np) M = fmaxf(M, ml[(cb + lane) * G].x);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    float den = 0.f;     // this lane's share of the denominator (pieces lane, lane + 32, ...)
    for (int cb = 0; cb < np; cb += 32) {
        const float2 v = cb == 0 ? v0 : (cb + lane < np ? ml[(cb + lane) * G] : make_float2(-1.0e30f, 0.f));
        const float w = cb + lane < np ? fast_exp2(v.x - M) : 0.f;
        den = fmaf(w, v.y, den);
        const int cnt = min(32, np - cb);
        int j = 0;
        if (cb == 0) {
#pragma unroll
            for (int c = 0; c < PRE; ++c)
                if (c < cnt) {
                    const float wj = __shfl_sync(0xffffffffu, w, c);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] = fmaf(wj, pre[c].v[e], acc[e]);
                }
            j = min(PRE, cnt);
        }
#pragma unroll 2
        for (; j < cnt; ++j) {
            const float wj = __shfl_sync(0xffffffffu, w, j);
            const Vec x = po[(cb + j) * pstride];
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = fmaf(wj, x.v[e], acc[e]);
        }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    Vec r;
#pragma unroll
    for (int e = 0; e < VEC; ++e) r.v[e] = acc[e] / den;
    reinterpret_cast<Vec*>(out + (u * G + g) * D)[lane] = r;
    KVS_TRACE_STAMP(tr, 2);
}

// Units of three or more pieces (fewer units than blocks): one BLOCK of four warps per (unit, q-head).
// Warp w takes pieces w, w + 4, ...: with up to four pieces per warp in flight a unit of 16 pieces needs
// one round trip for the (max, sum) pairs and one for the vectors (the first of which is requested
// together with the pairs).  The warps' sums are added in warp order by warp 0: a fixed order.
constexpr int kLongWarps = 4;

template <int D>
__global__ void __launch_bounds__(kLongWarps * 32, 8)
    decode_combine_long_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, float* __restrict__ out,
                               int G, int tpu, long long T, int NC, const int* __restrict__ n_extra, int n, int tile_rows,
                               int units, int cap, int* status, unsigned long long* trace) {
    constexpr int VEC = D / 32;
    struct __align__(VEC * 4) Vec {
        float v[VEC];
    };
    __shared__ float s_max[kLongWarps], s_den[kLongWarps];
    __shared__ float s_acc[kLongWarps][D];
    unsigned long long* tr = (trace && threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))
                                 ? trace + (size_t)(150 + (blockIdx.x != 0)) * kTraceSlots : nullptr;
    KVS_TRACE_STAMP(tr, 0);
    pdl_launch_dependents();
    pdl_wait();
    KVS_TRACE_STAMP(tr, 1);
    if (n_extra) {   // replayed launch: recompute the tile line from the grown length
        tpu = (min(n + *n_extra, cap) + tile_rows - 1) / tile_rows;
        T = (long long)units * tpu;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long u = blockIdx.x / G;
    const int g = blockIdx.x - (int)u * G;
    const int c0 = cta_of_tile(u * tpu, T, NC);
    int np = cta_of_tile((u + 1) * tpu - 1, T, NC) - c0 + 1;             // pieces of this unit
#ifdef KVS_DEBUG_BOUNDS
    if (!KVS_BOUNDS_OK(u + c0, np, (long long)units + NC, status)) np = 1;
#endif
    const float2* ml = reinterpret_cast<const float2*>(part_ml) + (u + c0) * G + g;   // piece c: ml[c * G]
    const Vec* po = reinterpret_cast<const Vec*>(part_o + ((u + c0) * G + g) * D) + lane;   // piece c: po[c * G * 32]
    const int pstride = G * 32;
    const int mine = np > warp ? (np - warp + kLongWarps - 1) / kLongWarps : 0;       // pieces warp, warp + 4, ... of this warp
    // this warp's first 32 pairs and, in the same round trip, its first four vectors
    constexpr int PRE = 4;
    const float2 v0 = lane < mine ? ml[(warp + kLongWarps * lane) * G] : make_float2(-1.0e30f, 0.f);
    Vec pre[PRE];
#pragma unroll
    for (int j = 0; j < PRE; ++j)
        if (j < mine) pre[j] = po[(warp + kLongWarps * j) * pstride];
    float M = v0.x;
    for (int jb = 32; jb < mine; jb += 32)
        if (jb + lane < mine) M = fmaxf(M, ml[(warp + kLongWarps * (jb + lane)) * G].x);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    if (lane == 0) s_max[warp] = M;
    __syncthreads();
    M = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));
    float acc[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
    float den = 0.f;
    for (int jb = 0; jb < mine; jb += 32) {
        const float2 v = jb == 0 ? v0 : (jb + lane < mine ? ml[(warp + kLongWarps * (jb + lane)) * G] : make_float2(-1.0e30f, 0.f));
        const float w = jb + lane < mine ? fast_exp2(v.x - M) : 0.f;
        den = fmaf(w, v.y, den);
        const int cnt = min(32, mine - jb);
        int j = 0;
        if (jb == 0) {
#pragma unroll
            for (int t = 0; t < PRE; ++t)
                if (t < cnt) {
                    const float wj = __shfl_sync(0xffffffffu, w, t);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] = fmaf(wj, pre[t].v[e], acc[e]);
                }
            j = min(PRE, cnt);
        }
#pragma unroll 4
        for (; j < cnt; ++j) {
            const float wj = __shfl_sync(0xffffffffu, w, j);
            const Vec x = po[(warp + kLongWarps * (jb + j)) * pstride];
#pragma unroll
            for (int e = 0; e < VEC; ++e) acc[e] = fmaf(wj, x.v[e], acc[e]);
        }
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    if (lane == 0) s_den[warp] = den;
#pragma unroll
    for (int e = 0; e < VEC; ++e) s_acc[warp][lane * VEC + e] = acc[e];
    __syncthreads();
    if (warp == 0) {
        float d = 0.f;
        Vec r;
#pragma unroll
        for (int e = 0; e < VEC; ++e) r.v[e] = 0.f;
#pragma unroll
        for (int wq = 0; wq < kLongWarps; ++wq) {
            d += s_den[wq];
#pragma unroll
            for (int e = 0; e < VEC; ++e) r.v[e] += s_acc[wq][lane * VEC + e];
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) r.v[e] /= d;
        reinterpret_cast<Vec*>(out + (u * G + g) * D)[lane] = r;
        KVS_TRACE_STAMP(tr, 2);
    }
}

template <int D>
static cudaError_t launch_combine_short(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream) {
    constexpr int WARPS = 8;
    const long long items = (long long)a.units * a.G;
    const dim3 grid((unsigned)((items + WARPS - 1) / WARPS)), block(WARPS * 32);
    return launch_kernel(decode_combine_kernel<D, 2, WARPS>, grid, block, 0, stream, a.programmatic, (const float*)a.part_o,
                         (const float*)a.part_ml, a.out, a.G, plan.tpu, plan.T, plan.NC, a.n_extra, a.n, plan.tile_rows,
                         a.units, a.capacity, a.status, a.trace);
}

template <int D>
static cudaError_t launch_combine_long(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream) {
    const dim3 grid((unsigned)(a.units * a.G)), block(kLongWarps * 32);
    return launch_kernel(decode_combine_long_kernel<D>, grid, block, 0, stream, a.programmatic, (const float*)a.part_o,
                         (const float*)a.part_ml, a.out, a.G, plan.tpu, plan.T, plan.NC, a.n_extra, a.n, plan.tile_rows,
                         a.units, a.capacity, a.status, a.trace);
}

cudaError_t launch_combine(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream) {
    // a unit has at most two pieces when no block's share is shorter than a unit, i.e. when there are
    // at least as many units as blocks (whatever the length, also one that grows under graph replay)
    const bool short_units = a.units >= plan.NC;
    if (a.D == 128) return short_units ? launch_combine_short<128>(a, plan, stream) : launch_combine_long<128>(a, plan, stream);
    return short_units ? launch_combine_short<64>(a, plan, stream) : launch_combine_long<64>(a, plan, stream);
}

// --------------------------------------------------------------------------------------
// Launch plumbing for the scalar kernel.
// --------------------------------------------------------------------------------------
template <typename T, int D, int G>
static cudaError_t set_attr_one() {
    cudaError_t e = cudaFuncSetAttribute(decode_splitk_scalar<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ScalarShape<T, D, G>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // the whole L1 / shared-memory array as shared memory, so that the combine kernel's blocks, launched
    // early behind this kernel, find room to become resident beside its blocks (see the tensor-core kernel)
    return cudaFuncSetAttribute(decode_splitk_scalar<T, D, G>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                cudaSharedmemCarveoutMaxShared);
}

template <typename T, int D>
static cudaError_t set_attr_groups() {
    cudaError_t e;
    if ((e = set_attr_one<T, D, 1>()) != cudaSuccess) return e;
    if ((e = set_attr_one<T, D, 2>()) != cudaSuccess) return e;
    if ((e = set_attr_one<T, D, 4>()) != cudaSuccess) return e;
    return set_attr_one<T, D, 8>();
}

template <typename T, int D, int G>
static cudaError_t launch_scalar_one(const ScalarKernelArgs& ka, int NC, bool programmatic, cudaStream_t stream) {
    return launch_kernel(decode_splitk_scalar<T, D, G>, dim3(NC), dim3(ScalarShape<T, D, G>::THREADS),
                         ScalarShape<T, D, G>::SMEM_BYTES, stream, programmatic, ka);
}

template <typename T, int D>
static cudaError_t launch_scalar_groups(int G, const ScalarKernelArgs& ka, int NC, bool pdl, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_scalar_one<T, D, 1>(ka, NC, pdl, stream);
        case 2: return launch_scalar_one<T, D, 2>(ka, NC, pdl, stream);
        case 4: return launch_scalar_one<T, D, 4>(ka, NC, pdl, stream);
        case 8: return launch_scalar_one<T, D, 8>(ka, NC, pdl, stream);
        default: return cudaErrorInvalidValue;
    }
}

void plan_decode_scalar(int units, int n, int G, int D, int dtype, int sm_count, int max_ctas, DecodePlan* plan) {
    const int rb = D * (dtype == 0 ? 2 : 4);
    plan->tile_rows = kTileBytes / rb;
    plan->tpu = (n + plan->tile_rows - 1) / plan->tile_rows;
    plan->T = (long long)units * plan->tpu;
    const int per_sm = (G <= 2) ? KVS_BLOCKS_PER_SM : 1;
    int cap = sm_count * per_sm;
    if (max_ctas > 0) cap = std::min(cap, max_ctas);
    cap = std::min(cap, kMaxCtas);
    plan->NC = (int)std::min<long long>(plan->T, cap);
    plan->kernel = 1;
}

cudaError_t launch_decode_scalar(const DecodeArgs& a, const DecodePlan& plan, cudaStream_t stream) {
    ScalarKernelArgs ka;
    ka.q = (const char*)a.q;
    ka.kplane = (const char*)a.kplane;
    ka.vplane = (const char*)a.vplane;
    ka.part_o = a.part_o;
    ka.part_ml = a.part_ml;
    ka.status = a.status;
    ka.n = a.n;
    ka.row_stride = a.row_stride;
    ka.tpu = plan.tpu;
    ka.T = plan.T;
    ka.scale_log2 = a.scale_log2;
    ka.safe_rows = (a.programmatic && !a.unit_len) ? a.safe_rows : 0;
    ka.unit_len = a.unit_len;
    ka.n_extra = a.n_extra;
    ka.units = a.units;
    ka.cap = a.capacity;
    ka.k_new = (const char*)a.k_new;
    ka.v_new = (const char*)a.v_new;
    ka.out = a.finish_in_kernel ? a.out : nullptr;
    ka.flags = a.flags;
    ka.plane_bytes = a.plane_bytes;
    ka.wait_ns = a.wait_ns;
    ka.stall_tile = a.stall_tile;
    ka.trace = a.trace;
    const bool pdl = a.programmatic;
    if (a.dtype == 0) {
        if (a.D == 128) return launch_scalar_groups<__nv_bfloat16, 128>(a.G, ka, plan.NC, pdl, stream);
        if (a.D == 64) return launch_scalar_groups<__nv_bfloat16, 64>(a.G, ka, plan.NC, pdl, stream);
    } else {
        if (a.D == 128) return launch_scalar_groups<float, 128>(a.G, ka, plan.NC, pdl, stream);
        if (a.D == 64) return launch_scalar_groups<float, 64>(a.G, ka, plan.NC, pdl, stream);
    }
    return cudaErrorInvalidValue;
}

// --------------------------------------------------------------------------------------
// K4: read roof.  Same producer, same ring, consumers only fold the bytes together.
// --------------------------------------------------------------------------------------
constexpr int kRoofStages = 3;
constexpr int kRoofTileBytes = 16384;
constexpr int kRoofStageBytes = 2 * kRoofTileBytes;
constexpr int kRoofSmem = kRoofStages * kRoofStageBytes + 2 * kRoofStages * 8 + 16;

constexpr int kRoofThreads = kConsumerThreads + 32;   // consumer warps + the producer warp

__global__ void __launch_bounds__(kRoofThreads, 2)
    read_roof_kernel(const char* __restrict__ src, long long n_tiles, unsigned long long* checksum) {
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kRoofStages * kRoofStageBytes);
    uint64_t* empty_bar = full_bar + kRoofStages;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kRoofStages);
    __shared__ int local_status;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long t0 = first_tile_of_cta(blockIdx.x, n_tiles, gridDim.x);
    const long long t1 = first_tile_of_cta(blockIdx.x + 1, n_tiles, gridDim.x);
    if (tid == 0) {
        for (int s = 0; s < kRoofStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerWarps);
        }
        *abort_flag = 0;
        local_status = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (warp == kConsumerWarps) {
        if (lane == 0) {
            int it = 0;
            for (long long gt = t0; gt < t1; ++gt, ++it) {
                const int st = it % kRoofStages;
                if (it >= kRoofStages &&
                    !mbar_wait_bounded(&empty_bar[st], ((it / kRoofStages) - 1) & 1, abort_flag, &local_status))
                    break;
                unsigned char* sb = smem + st * kRoofStageBytes;
                mbar_arrive_expect_tx(&full_bar[st], kRoofStageBytes);
                bulk_g2s(sb, src + gt * kRoofStageBytes, kRoofTileBytes, &full_bar[st]);
                bulk_g2s(sb + kRoofTileBytes, src + gt * kRoofStageBytes + kRoofTileBytes, kRoofTileBytes, &full_bar[st]);
            }
        }
        return;
    }
    unsigned int x = 0;
    int it = 0;
    for (long long gt = t0; gt < t1; ++gt, ++it) {
        const int st = it % kRoofStages;
        if (!mbar_wait_bounded(&full_bar[st], (it / kRoofStages) & 1, abort_flag, &local_status)) return;
        const uint4* sb = reinterpret_cast<const uint4*>(smem + st * kRoofStageBytes);
#pragma unroll
        for (int j = 0; j < kRoofStageBytes / 16 / kConsumerThreads; ++j) {
            const uint4 r = sb[j * kConsumerThreads + tid];
            x ^= r.x ^ r.y ^ r.z ^ r.w;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[st]);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) x ^= __shfl_xor_sync(0xffffffffu, x, o);
    if (lane == 0) atomicXor(checksum, (unsigned long long)x);
}

cudaError_t launch_read_roof(const void* src, size_t bytes, unsigned long long* checksum, int sm_count,
                             cudaStream_t stream) {
    const long long n_tiles = (long long)(bytes / kRoofStageBytes);
    const int NC = (int)std::min<long long>(n_tiles, 2LL * sm_count);
    cudaError_t e = cudaMemsetAsync(checksum, 0, 8, stream);
    if (e != cudaSuccess) return e;
    read_roof_kernel<<<NC, kRoofThreads, kRoofSmem, stream>>>((const char*)src, n_tiles, checksum);
    return cudaGetLastError();
}

// --------------------------------------------------------------------------------------
// Self-test of the give-up path of the bounded waits: one thread waits on a barrier that
// nothing ever arrives at, with a short limit, through the same mbar_wait_bounded the
// pipelined kernels use.  No copy is in flight; the wait runs out, the status word becomes
// kDevTimeout and the kernel returns normally.
// --------------------------------------------------------------------------------------
__global__ void wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns, unsigned long long* waited_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = globaltimer_ns();
        const bool ok = mbar_wait_bounded(&bar, 0, &abort_flag, status, limit_ns);
        if (waited_ns) *waited_ns = ok ? 0ull : globaltimer_ns() - t0;
    }
    __syncthreads();
    // the other threads see the give-up through the flag, as the consumer warps of the real kernels do
    if (threadIdx.x == 1 && abort_flag == 0) atomicExch(status, 1);
}

cudaError_t launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, unsigned long long* waited_ns,
                                         cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns, waited_ns);
    return cudaGetLastError();
}

// Self-test of the bounds-checking build: hands the check an offset that lies outside its buffer
// (no memory is touched) and lets it record the violation.  `is_checking_build` tells the host which
// build this is.
__global__ void bounds_selftest_kernel(int* status) {
    // 5 + 8 > 10; in a normal build the check is compiled out and nothing is recorded
    if (threadIdx.x == 0 && KVS_BOUNDS_OK(5, 8, 10, status)) return;
}

bool is_tracing_build() {
#ifdef KVS_TRACE
    return true;
#else
    return false;
#endif
}

bool is_bounds_checking_build() {
#ifdef KVS_DEBUG_BOUNDS
    return true;
#else
    return false;
#endif
}

cudaError_t launch_bounds_selftest(int* status, cudaStream_t stream) {
    bounds_selftest_kernel<<<1, 32, 0, stream>>>(status);
    return cudaGetLastError();
}

cudaError_t init_kernels() {
    cudaError_t e;
    if ((e = set_attr_groups<__nv_bfloat16, 128>()) != cudaSuccess) return e;
    if ((e = set_attr_groups<__nv_bfloat16, 64>()) != cudaSuccess) return e;
    if ((e = set_attr_groups<float, 128>()) != cudaSuccess) return e;
    if ((e = set_attr_groups<float, 64>()) != cudaSuccess) return e;
    return cudaFuncSetAttribute(read_roof_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRoofSmem);
}

}  // namespace kvs
