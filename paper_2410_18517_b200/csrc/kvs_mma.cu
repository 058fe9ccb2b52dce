// K2b: grouped-query split-K decode attention on the tensor cores (bf16 storage only).
//
// The G q-heads that share one kv-head form the (zero-padded) 16-row M side of
// mma.sync.m16n8k16 bf16 -> fp32 tiles: S = Q K^T over 16-token blocks, then O += P V with
// the softmax weights split as P = P_hi + P_lo (two bf16 terms) so that the second
// contraction keeps ~16 bits of P.  K/V tiles arrive by TMA tensor-map copies with the
// 128-byte swizzle, which makes ldmatrix (K) and ldmatrix.trans (V) conflict-free.
// Work decomposition, partial-result layout and the combine kernel are those of the scalar
// path.  One producer warp, four consumer warps; each consumer warp owns 16-token blocks.
#include <cuda.h>

#include <algorithm>

#include "kvs_device.cuh"
#include "kvs_kernels.h"

namespace kvs {

namespace {

// Consumer warps, tile size, ring depth and blocks per SM (compile-time; defaults = measured best).
#ifndef KVS_MMA_WARPS
#define KVS_MMA_WARPS 4
#endif
#ifndef KVS_MMA_TILE_BYTES
#define KVS_MMA_TILE_BYTES 16384
#endif
#ifndef KVS_MMA_STAGES
#define KVS_MMA_STAGES 4
#endif
#ifndef KVS_MMA_BLOCKS_PER_SM
#define KVS_MMA_BLOCKS_PER_SM 1
#endif
constexpr int kMmaWarps = KVS_MMA_WARPS;
constexpr int kMmaConsumerThreads = kMmaWarps * 32;
constexpr int kMmaThreads = kMmaConsumerThreads + 64;   // + the producer warp and the hand-over warp
constexpr int kMmaTileBytes = KVS_MMA_TILE_BYTES;
constexpr int kMmaQBytes = 2048;  // room for 8 heads x 128 x bf16
constexpr int kMmaStages = KVS_MMA_STAGES;
// Second ring geometry, for launches that give every block at least kMmaBigMinTiles of its (larger) tiles: 3
// stages of 32 KiB tiles.  Half as many barrier round trips, piece bookkeeping and tile set-ups per byte: with
// one warp per scheduler all of that is exposed, and the kernel follows the SM clock that the power cap
// leaves (same box at 1.5-1.7 GHz, builds alternating: 32q/8kv, B=4, n=32768 2.77 -> 2.63 ms per step; B=32,
// n=8192 5.46 -> 5.15; B=32, n=1024 0.846 -> 0.835).  Small launches keep the 16 KiB tiles: they need the finer
// split over the blocks.
#ifndef KVS_MMA_BIG_TILE_BYTES
#define KVS_MMA_BIG_TILE_BYTES 32768
#endif
#ifndef KVS_MMA_BIG_STAGES
#define KVS_MMA_BIG_STAGES 3
#endif
#ifndef KVS_MMA_BIG_MIN_TILES
#define KVS_MMA_BIG_MIN_TILES 12
#endif
constexpr int kMmaBigTileBytes = KVS_MMA_BIG_TILE_BYTES;
constexpr int kMmaBigStages = KVS_MMA_BIG_STAGES;
constexpr int kMmaBigMinTiles = KVS_MMA_BIG_MIN_TILES;
constexpr int kBoxRows = 64;      // the pool's tensor map moves boxes of 64 columns x 64 rows (8 KiB)
constexpr int kTailRows = 16;     // a second map moves 16-row boxes: the last, partly filled tile of a unit
                                  // is fetched in as many of these as hold rows (16 = the tokens of one MMA block)

template <int D, int BIG>
struct MmaShape {
    static constexpr int TILE = BIG ? kMmaBigTileBytes : kMmaTileBytes;   // bytes per K tile and per V tile
    static constexpr int STAGES = BIG ? kMmaBigStages : kMmaStages;
    static constexpr int RB = D * 2;
    static constexpr int HALVES = D / 64;                  // 128-byte column blocks per row
    static constexpr int TN = TILE / RB;                   // rows per tile: 64 or 128 (D=128), 128 or 256 (D=64)
    static constexpr int BPW = TN / (kMmaWarps * 16);      // 16-token blocks per warp per tile
    static constexpr int KSTEPS = D / 16;
    static constexpr int NB = D / 8;
    static constexpr int STAGE_BYTES = 2 * TILE + kMmaQBytes;
    static constexpr int SCRATCH_FLOATS = kMmaWarps * 8 * (D + 2);   // [warp][q-head of the group][D + 2]
    static constexpr int HANDOVER_FLOATS = 8 * (D + 2);              // another block's piece of a cut unit: [q-head][D + 2]
    static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + (SCRATCH_FLOATS + HANDOVER_FLOATS) * 4 +
                                      (2 * STAGES + 2) * 8 + 16;
};

__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst_smem)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr));
}

// D(16x8) += A(16x16) B(16x8), rows 8..15 of A are zero padding: their accumulators are
// kept in throw-away registers (c2, c3) that stay zero.
__device__ __forceinline__ void mma_bf16_upper(float& c0, float& c1, uint32_t a_klo, uint32_t a_khi, uint32_t b0,
                                               uint32_t b1) {
    float z2 = 0.f, z3 = 0.f;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c0), "+f"(c1), "+f"(z2), "+f"(z3)
        : "r"(a_klo), "r"(0u), "r"(a_khi), "r"(0u), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

struct MmaKernelArgs {
    const char* q;
    float* part_o;
    float* part_ml;
    int* status;
    int n;
    int row_stride;
    int tpu;
    long long T;
    long long krow0;  // first row of the K plane within the pool-wide row index
    long long vrow0;
    float scale_log2;
    int safe_rows;  // rows of every unit that no kernel possibly still running writes
    const int* unit_len;  // per-unit row counts of a ragged slot, or nullptr (then n holds for all)
    int G;          // q-heads per kv-head, 1..8
    const int* n_extra;  // graph replay: rows every slot has grown by since the launch was recorded, or nullptr
    int units;
    int cap;             // rows a unit can hold: lengths that grew on the device are cut off there
    const char* k_new;   // the step's new rows, appended by this kernel (n counts them), or nullptr
    const char* v_new;
    char* kplane;        // planes of the slot (for the append; the tiles are fetched through the tensor map)
    char* vplane;
    // Finishing inside this kernel (no combine launch): set when no unit has more than two pieces.
    float* out;          // [units][G][D] final results, or nullptr: every piece goes to part_o / part_ml
    int* flags;          // [units], all zero between launches: 1 = the unit's second piece is in part_o / part_ml
    long long plane_rows;   // rows of one plane (what a bounds-checking build checks tile rows against)
    unsigned long long wait_ns;   // limit of every wait inside the kernel
    long long stall_tile;         // self-test only: the K/V copies of this tile are withheld (-1: none)
    unsigned long long* trace;    // tracing build: this launch's rows of time stamps, or nullptr
};

// G (q-heads per kv-head, 1..8) is a run-time argument: it only selects which rows of the padded
// 16-row M side are real, so one kernel per head size serves every group size.
template <int D, int BIG>
__global__ void __launch_bounds__(kMmaThreads, KVS_MMA_BLOCKS_PER_SM)
    decode_splitk_mma(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap_tail,
                      const MmaKernelArgs a_in) {
    using S = MmaShape<D, BIG>;
    constexpr int kTile = S::TILE, kStages = S::STAGES;
    MmaKernelArgs a = a_in;
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
    constexpr int TN = S::TN, KSTEPS = S::KSTEPS, NB = S::NB, BPW = S::BPW;
    const int G = a.G;
    const int QBYTES = G * S::RB;

    extern __shared__ unsigned char smem_raw[];
    // 128-byte swizzled tiles need 1024-byte aligned bases
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    float* scratch = reinterpret_cast<float*>(smem + kStages * S::STAGE_BYTES);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(scratch + S::SCRATCH_FLOATS);
    uint64_t* empty_bar = full_bar + kStages;
    uint64_t* tail_bar = empty_bar + kStages;     // every consumer thread has written this block's second-piece partial
    uint64_t* head_bar = tail_bar + 1;               // the next block's second-piece partial is in handover[]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(head_bar + 1);
    float* handover = const_cast<float*>(reinterpret_cast<volatile float*>(abort_flag + 4));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = gridDim.x;
    const long long t0 = ((long long)blockIdx.x * a.T) / NC;
    const long long t1 = ((long long)(blockIdx.x + 1) * a.T) / NC;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kMmaWarps);
        }
        mbar_init(tail_bar, kMmaConsumerThreads);
        mbar_init(head_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == kMmaWarps) {
        // ------------------------------ producer ------------------------------
        // Lane 0 issues the copies; the whole warp stores the step's new rows when the launch
        // carries an append.
        {
            // Issue the copies of tile `gt` into stage `st` (see the scalar kernel: the barrier
            // is armed once with the stage's full byte count, K/V and q may be issued apart).
            auto issue = [&](long long gt, int st, bool arm, bool kv, bool qpart) {
                const long long u = gt / a.tpu;
                const int ti = (int)(gt - u * a.tpu);
                const bool with_q = (gt == t0) || (ti == 0);
                const int n_u = a.unit_len ? min(a.unit_len[u], a.cap) : a.n;
                const int rows = min(TN, n_u - ti * TN);          // <= 0: a ragged unit ended before this tile
                // a full tile comes in 64-row boxes; a partly filled one in 16-row boxes, only those that hold rows
                const int tail_boxes = rows < TN ? (rows + kTailRows - 1) / kTailRows : 0;
                const uint32_t kv_bytes = rows <= 0 ? 0u : (rows == TN ? 2u * kTile : 2u * tail_boxes * kTailRows * S::RB);
                unsigned char* sb = smem + st * S::STAGE_BYTES;
                if (arm) {
                    const uint32_t total = kv_bytes + (with_q ? QBYTES : 0);
                    if (total) mbar_arrive_expect_tx(&full_bar[st], total);
                    else mbar_arrive(&full_bar[st]);
                }
                if (kv && rows > 0 && gt != a.stall_tile) {
                    long long row = u * a.row_stride + (long long)ti * TN;
                    // (a whole box is fetched even where the unit has fewer rows: it stays inside the unit's row_stride)
                    if (!KVS_BOUNDS_OK(row, rows == TN ? TN : tail_boxes * kTailRows, a.plane_rows, a.status) ||
                        !KVS_BOUNDS_OK(u, 1, a.units, a.status))
                        row = 0;
                    if (rows == TN) {
#pragma unroll
                        for (int h = 0; h < S::HALVES; ++h)
#pragma unroll
                            for (int rb = 0; rb < TN / kBoxRows; ++rb) {
                                const int off = h * (TN * 128) + rb * (kBoxRows * 128);
                                tma_load_2d(sb + off, &tmap, h * 64, (int)(a.krow0 + row) + rb * kBoxRows, &full_bar[st]);
                                tma_load_2d(sb + kTile + off, &tmap, h * 64, (int)(a.vrow0 + row) + rb * kBoxRows,
                                            &full_bar[st]);
                            }
                    } else {
#pragma unroll
                        for (int h = 0; h < S::HALVES; ++h)
                            for (int rb = 0; rb < tail_boxes; ++rb) {
                                const int off = h * (TN * 128) + rb * (kTailRows * 128);
                                tma_load_2d(sb + off, &tmap_tail, h * 64, (int)(a.krow0 + row) + rb * kTailRows, &full_bar[st]);
                                tma_load_2d(sb + kTile + off, &tmap_tail, h * 64,
                                            (int)(a.vrow0 + row) + rb * kTailRows, &full_bar[st]);
                            }
                    }
                }
                if (qpart && with_q)
                    bulk_g2s(sb + 2 * kTile, a.q + (KVS_BOUNDS_OK(u, 1, a.units, a.status) ? u : 0) * (long long)QBYTES,
                             QBYTES, &full_bar[st]);
            };
            // Until the preceding kernel in the stream is known to have finished, fetch only
            // K/V tiles made entirely of rows that no kernel still in flight can be writing.
            int npre = 0;
            if (lane == 0) {
                for (; npre < kStages && t0 + npre < t1; ++npre) {
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
                    store_new_rows<S::RB>(lane, t0, t1, a.tpu, a.n, a.row_stride, a.k_new, a.v_new, a.kplane, a.vplane,
                                          a.plane_rows * S::RB, a.units, a.status);
                else if (lane == 0 && blockIdx.x == 0)
                    atomicExch(a.status, 4);
            }
            if (lane != 0) return;
            int it = npre;
            bool ok = true;
            for (long long gt = t0 + npre; gt < t1; ++gt, ++it) {
                const int st = it % kStages;
                if (it >= kStages)
                    ok = mbar_wait_bounded(&empty_bar[st], ((it / kStages) - 1) & 1, abort_flag, a.status, a.wait_ns);
                if (!ok) break;
                issue(gt, st, true, true, true);
            }
            if (!ok) {
                for (int j = max(0, it - kStages); j < it; ++j)
                    mbar_wait_bounded(&full_bar[j % kStages], (j / kStages) & 1, abort_flag + 1, a.status, a.wait_ns);
            }
        }
        return;
    }

    if (warp == kMmaWarps + 1) {
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
    const int row = lane >> 2;   // q-head row of the accumulator fragment (rows 8..15 are padding)
    const int quad = lane & 3;

    int it = 0;
    long long gt = t0;
    while (gt < t1) {
        const long long u = gt / a.tpu;
        const int ti0 = (int)(gt - u * a.tpu);
        const int piece_tiles = (int)min((long long)(a.tpu - ti0), t1 - gt);
        const int n_u = a.unit_len ? min(a.unit_len[u], a.cap) : a.n;

        uint32_t qa[KSTEPS][2];
        float o[NB][2];
        float m = -1.0e30f, lsum = 0.f;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) o[nb][0] = o[nb][1] = 0.f;

        for (int k = 0; k < piece_tiles; ++k, ++it) {
            const int st = it % kStages;
            if (!mbar_wait_bounded(&full_bar[st], (it / kStages) & 1, abort_flag, a.status, a.wait_ns)) return;
            if (tid == 0 && it == 0) KVS_TRACE_STAMP(tr, kTrFirstTile);
            const unsigned char* ks = smem + st * S::STAGE_BYTES;
            const uint32_t ks_u32 = smem_u32(ks);
            const uint32_t vs_u32 = ks_u32 + kTile;
            if (k == 0) {
                // A fragments of Q: row g < G real, the rest zero
                const uint32_t* qs = reinterpret_cast<const uint32_t*>(ks + 2 * kTile);
#pragma unroll
                for (int s = 0; s < KSTEPS; ++s) {
                    qa[s][0] = row < G ? qs[row * (D / 2) + s * 8 + quad] : 0u;
                    qa[s][1] = row < G ? qs[row * (D / 2) + s * 8 + 4 + quad] : 0u;
                }
            }
            const int valid = n_u - (ti0 + k) * TN;  // rows of this tile that exist (may exceed TN or be <= 0)
            if (valid <= 0) {   // tile past the end of a ragged unit: nothing was loaded, nothing to add
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
                continue;
            }

            if (warp * BPW * 16 >= valid) {   // none of this warp's rows exists in this (partly filled) tile
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
                continue;
            }
            // A warp's BPW blocks of 16 tokens go through the tile in three phases - all score products, one
            // online-softmax update over all of them, all output products - so that the blocks' chains of
            // loads and MMAs overlap and the running state is rescaled once per tile (one warp per scheduler:
            // nothing else hides those latencies).
            // ---- S = Q K^T, per block two 8-token column blocks ----
            // All K fragments of a block are fetched first and the products of even and odd 16-column steps go
            // to separate accumulators, so that neither the shared-memory latency nor the latency of one MMA
            // feeding the next sits KSTEPS times on the path of a tile.
            float s[BPW][2][2];
            float tmax = -INFINITY;
#pragma unroll
            for (int blk = 0; blk < BPW; ++blk) {
                const int tok0 = (warp * BPW + blk) * 16;
#pragma unroll
                for (int nb = 0; nb < 2; ++nb) s[blk][nb][0] = s[blk][nb][1] = 0.f;
                if (tok0 < valid) {   // else no row of this block exists (and a partly filled tile was not fetched that far)
                    const int t = tok0 + ((lane >> 4) << 3) + (lane & 7);
                    const uint32_t rowaddr = ks_u32 + t * 128;
                    const int sw = t & 7;
                    uint32_t b[KSTEPS][4];
#pragma unroll
                    for (int st_k = 0; st_k < KSTEPS; ++st_k) {
                        const int half = st_k >> 2;
                        const int chunk = ((st_k & 3) << 1) + ((lane >> 3) & 1);
                        ldmatrix_x4(b[st_k], rowaddr + half * (TN * 128) + ((chunk ^ sw) << 4));
                    }
                    float s2[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
                    for (int st_k = 0; st_k < KSTEPS; st_k += 2) {
                        mma_bf16_upper(s[blk][0][0], s[blk][0][1], qa[st_k][0], qa[st_k][1], b[st_k][0], b[st_k][1]);
                        mma_bf16_upper(s[blk][1][0], s[blk][1][1], qa[st_k][0], qa[st_k][1], b[st_k][2], b[st_k][3]);
                        mma_bf16_upper(s2[0][0], s2[0][1], qa[st_k + 1][0], qa[st_k + 1][1], b[st_k + 1][0], b[st_k + 1][1]);
                        mma_bf16_upper(s2[1][0], s2[1][1], qa[st_k + 1][0], qa[st_k + 1][1], b[st_k + 1][2], b[st_k + 1][3]);
                    }
#pragma unroll
                    for (int nb = 0; nb < 2; ++nb) {
                        s[blk][nb][0] += s2[nb][0];
                        s[blk][nb][1] += s2[nb][1];
                    }
                }
                // scores in the log2 domain; tokens that do not exist count as minus infinity
#pragma unroll
                for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int tok = tok0 + nb * 8 + quad * 2 + j;
                        s[blk][nb][j] = tok < valid ? s[blk][nb][j] * a.scale_log2 : -INFINITY;
                        tmax = fmaxf(tmax, s[blk][nb][j]);
                    }
            }
            // ---- one online-softmax update for row `row` over the warp's tokens of this tile ----
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
            const float m_new = fmaxf(m, tmax);
            const float alpha = fast_exp2(m - m_new);
            m = m_new;
            float p[BPW][2][2];
            float psum = 0.f;
#pragma unroll
            for (int blk = 0; blk < BPW; ++blk)
#pragma unroll
                for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        p[blk][nb][j] = fast_exp2(s[blk][nb][j] - m_new);
                        psum += p[blk][nb][j];
                    }
            lsum = lsum * alpha + psum;
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                o[nb][0] *= alpha;
                o[nb][1] *= alpha;
            }
            // ---- O += P V, per block 16 tokens x D, two 8-wide column blocks per ldmatrix ----
#pragma unroll
            for (int blk = 0; blk < BPW; ++blk) {
                const int tok0 = (warp * BPW + blk) * 16;
                if (tok0 >= valid) continue;
                // P = P_hi + P_lo as A fragments (k = tokens): klo = tokens 0..7, khi = tokens 8..15
                const float h00 = bf16_round(p[blk][0][0]), h01 = bf16_round(p[blk][0][1]);
                const float h10 = bf16_round(p[blk][1][0]), h11 = bf16_round(p[blk][1][1]);
                const uint32_t phi_lo = pack_bf16(h00, h01), phi_hi = pack_bf16(h10, h11);
                const uint32_t plo_lo = pack_bf16(p[blk][0][0] - h00, p[blk][0][1] - h01);
                const uint32_t plo_hi = pack_bf16(p[blk][1][0] - h10, p[blk][1][1] - h11);
                // Four column blocks at a time: their P_hi products are issued before their P_lo products, so
                // that an MMA never waits for the one just before it (same accumulator).
                const int t = tok0 + (((lane >> 3) & 1) << 3) + (lane & 7);
                const uint32_t rowaddr = vs_u32 + t * 128;
                const int sw = t & 7;
#pragma unroll
                for (int nbp = 0; nbp < NB / 2; nbp += 2) {
                    uint32_t b[2][4];
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        const int chunkg = (nbp + x) * 2 + (lane >> 4);
                        const int half = chunkg >> 3;
                        const int chunk = chunkg & 7;
                        ldmatrix_x4_trans(b[x], rowaddr + half * (TN * 128) + ((chunk ^ sw) << 4));
                    }
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        mma_bf16_upper(o[2 * (nbp + x)][0], o[2 * (nbp + x)][1], phi_lo, phi_hi, b[x][0], b[x][1]);
                        mma_bf16_upper(o[2 * (nbp + x) + 1][0], o[2 * (nbp + x) + 1][1], phi_lo, phi_hi, b[x][2], b[x][3]);
                    }
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        mma_bf16_upper(o[2 * (nbp + x)][0], o[2 * (nbp + x)][1], plo_lo, plo_hi, b[x][0], b[x][1]);
                        mma_bf16_upper(o[2 * (nbp + x) + 1][0], o[2 * (nbp + x) + 1][1], plo_lo, plo_hi, b[x][2], b[x][3]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[st]);
        }

        // ---- end of piece: merge the consumer warps, all q-heads of the group in one round ----
        // scratch[warp][q-head][D + 2]: one barrier before (the previous piece's readers are done),
        // one after the writes.
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
        float l = lsum;
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        named_bar_sync(1, kMmaConsumerThreads);
        if (row < G) {
            float* dst = scratch + (warp * 8 + row) * (D + 2);
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
                dst[nb * 8 + quad * 2] = o[nb][0];
                dst[nb * 8 + quad * 2 + 1] = o[nb][1];
            }
            if (quad == 0) {
                dst[D] = m;
                dst[D + 1] = l;
            }
        }
        if (head && !mbar_wait_bounded(head_bar, 0, abort_flag, a.status, a.wait_ns)) return;
        named_bar_sync(1, kMmaConsumerThreads);
        for (int idx = tid; idx < G * D; idx += kMmaConsumerThreads) {
            const int g = idx / D, d = idx - g * D;
            const float* src = scratch + g * (D + 2);
            constexpr int WS = 8 * (D + 2);            // floats between the warps' rows of one q-head
            float M = -1.0e30f;
#pragma unroll
            for (int j = 0; j < kMmaWarps; ++j) M = fmaxf(M, src[j * WS + D]);
            float acc = 0.f, den = 0.f;
#pragma unroll
            for (int j = 0; j < kMmaWarps; ++j) {
                const float w = fast_exp2(src[j * WS + D] - M);
                acc = fmaf(w, src[j * WS + d], acc);
                den = fmaf(w, src[j * WS + D + 1], den);
            }
            if (whole) {
                a.out[(u * G + g) * D + d] = acc / den;
            } else if (head) {
                const float* hv = handover + g * (D + 2);      // the unit's second piece
                const float Mx = fmaxf(M, hv[D]);
                const float w0 = fast_exp2(M - Mx), w1 = fast_exp2(hv[D] - Mx);
                a.out[(u * G + g) * D + d] = fmaf(w1, hv[d], w0 * acc) / fmaf(w1, hv[D + 1], w0 * den);
            } else if (KVS_BOUNDS_OK(pid, 1, a.units + (long long)gridDim.x, a.status)) {
                a.part_o[(pid * G + g) * D + d] = acc;
                if (d == 0) {
                    a.part_ml[(pid * G + g) * 2] = M;
                    a.part_ml[(pid * G + g) * 2 + 1] = den;
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

template <int D, int BIG>
cudaError_t set_attr() {
    cudaError_t e = cudaFuncSetAttribute(decode_splitk_mma<D, BIG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         MmaShape<D, BIG>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // All of the SM's L1 / shared-memory array as shared memory: the kernel gains nothing from L1
    // (its loads are bulk copies), and the blocks of the small kernels launched early behind it
    // (combine) only become resident beside it if the carve-out has room for them.  Measured: with
    // the default carve-out a footprint of 157 KiB instead of 142 KiB cost 2.8 us per layer.
    return cudaFuncSetAttribute(decode_splitk_mma<D, BIG>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                cudaSharedmemCarveoutMaxShared);
}

template <int D, int BIG>
cudaError_t launch_one(const CUtensorMap& tm, const CUtensorMap& tm_tail, const MmaKernelArgs& ka, int NC, bool pdl,
                       cudaStream_t stream) {
    return launch_kernel(decode_splitk_mma<D, BIG>, dim3(NC), dim3(kMmaThreads), MmaShape<D, BIG>::SMEM_BYTES, stream, pdl, tm,
                         tm_tail, ka);
}

}  // namespace

cudaError_t init_mma_kernels() {
    cudaError_t e;
    if ((e = set_attr<128, 0>()) != cudaSuccess || (e = set_attr<128, 1>()) != cudaSuccess ||
        (e = set_attr<64, 0>()) != cudaSuccess)
        return e;
    return set_attr<64, 1>();
}

// Tensor map over the whole pool seen as [total_rows][D] bf16, box = 64 columns x 64 rows (or, with
// `tail`, x 16 rows), 128-byte swizzle.  `storage` must be 64-byte aligned and hold
// sizeof(CUtensorMap) = 128 bytes.
cudaError_t make_pool_tensor_map(void* storage, void* pool, long long total_rows, int D, bool tail) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)total_rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)(tail ? kTailRows : kBoxRows)};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = reinterpret_cast<EncodeFn>(fn)(reinterpret_cast<CUtensorMap*>(storage), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                                2, pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

void plan_decode_mma(int units, int n, int D, int sm_count, int max_ctas, DecodePlan* plan) {
    int cap = sm_count * KVS_MMA_BLOCKS_PER_SM;
    if (max_ctas > 0) cap = std::min(cap, max_ctas);
    cap = std::min(cap, kMaxCtas);
    // the larger tiles when every block still gets kMmaBigMinTiles of them
    const int big_rows = kMmaBigTileBytes / (D * 2);
    const long long big_T = (long long)units * ((n + big_rows - 1) / big_rows);
    plan->tile_rows = big_T >= (long long)kMmaBigMinTiles * cap ? big_rows : kMmaTileBytes / (D * 2);
    plan->tpu = (n + plan->tile_rows - 1) / plan->tile_rows;
    plan->T = (long long)units * plan->tpu;
    plan->NC = (int)std::min<long long>(plan->T, cap);
    plan->kernel = 2;
}

cudaError_t launch_decode_mma(const DecodeArgs& a, const DecodePlan& plan, const void* tensor_map,
                              const void* tensor_map_tail, long long krow0, long long vrow0, cudaStream_t stream) {
    MmaKernelArgs ka;
    ka.q = (const char*)a.q;
    ka.part_o = a.part_o;
    ka.part_ml = a.part_ml;
    ka.status = a.status;
    ka.n = a.n;
    ka.row_stride = a.row_stride;
    ka.tpu = plan.tpu;
    ka.T = plan.T;
    ka.krow0 = krow0;
    ka.vrow0 = vrow0;
    ka.scale_log2 = a.scale_log2;
    ka.safe_rows = (a.programmatic && !a.unit_len) ? a.safe_rows : 0;
    ka.unit_len = a.unit_len;
    const CUtensorMap& tm = *reinterpret_cast<const CUtensorMap*>(tensor_map);
    const CUtensorMap& tm_tail = *reinterpret_cast<const CUtensorMap*>(tensor_map_tail);
    ka.G = a.G;
    ka.n_extra = a.n_extra;
    ka.units = a.units;
    ka.cap = a.capacity;
    ka.k_new = (const char*)a.k_new;
    ka.v_new = (const char*)a.v_new;
    ka.kplane = (char*)const_cast<void*>(a.kplane);
    ka.vplane = (char*)const_cast<void*>(a.vplane);
    ka.out = a.finish_in_kernel ? a.out : nullptr;
    ka.flags = a.flags;
    ka.plane_rows = a.plane_bytes / (a.D * 2);
    ka.wait_ns = a.wait_ns;
    ka.stall_tile = a.stall_tile;
    ka.trace = a.trace;
    if (a.G < 1 || a.G > 8) return cudaErrorInvalidValue;
    const bool big = plan.tile_rows * a.D * 2 == kMmaBigTileBytes && kMmaBigTileBytes != kMmaTileBytes;
    if (a.D == 128)
        return big ? launch_one<128, 1>(tm, tm_tail, ka, plan.NC, a.programmatic, stream)
                   : launch_one<128, 0>(tm, tm_tail, ka, plan.NC, a.programmatic, stream);
    if (a.D == 64)
        return big ? launch_one<64, 1>(tm, tm_tail, ka, plan.NC, a.programmatic, stream)
                   : launch_one<64, 0>(tm, tm_tail, ka, plan.NC, a.programmatic, stream);
    return cudaErrorInvalidValue;
}

}  // namespace kvs
