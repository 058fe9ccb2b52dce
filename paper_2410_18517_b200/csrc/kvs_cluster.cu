// One-kernel decode step of a layer for launches that latency, not bandwidth, bounds (few
// sequences, short caches): append of the new token's K/V row, split-K attention and the merge
// of the pieces in a single launch.
//
// A (sequence, kv-head) unit is handled by one thread-block cluster: block `rank` of the
// cluster takes an even share of the unit's 16 KiB tiles through the same bulk-copy ring and
// the same fp32 arithmetic as the persistent split-K kernel, then writes its piece
// (o[D], max, sum per q-head) into the shared memory of the cluster's first block
// (distributed shared memory) and arrives on that block's mbarrier; the first block waits for
// all pieces, merges them in rank order and writes the output.  No partial result goes through
// global memory and there is no combine kernel.
//
// With an append fused in, the row that the step adds (row n-1 of the unit) is not in the pool
// yet: the block whose share holds it fetches that row from the caller's k/v buffers straight
// into its place in the tile, and also stores it to the pool for later steps and for layers
// that share the slot.
#include <algorithm>

#include "kvs_device.cuh"
#include "kvs_kernels.h"
#include "kvs_scalar.cuh"

namespace kvs {

namespace {

constexpr int kClWarps = 8;
constexpr int kClConsumers = kClWarps * 32;
constexpr int kClThreads = kClConsumers + 32;
constexpr int kClTileBytes = 16384;       // per K tile and per V tile
constexpr int kClStages = 3;

template <typename T, int D, int G>
struct ClusterShape {
    static constexpr int RB = D * (int)sizeof(T);
    static constexpr int LPR = RB / 16;
    static constexpr int GPW = 32 / LPR;
    static constexpr int NG = kClWarps * GPW;
    static constexpr int TN = kClTileBytes / RB;
    static constexpr int QBYTES = G * RB;
    static constexpr int STAGE_BYTES = 2 * kClTileBytes + QBYTES;
    static constexpr int SCRATCH_FLOATS = NG * (D + 2);
    static constexpr int PIECE_FLOATS = G * (D + 2);                   // one block's piece
    static constexpr int RECV_FLOATS = kMaxClusterSize * PIECE_FLOATS; // pieces of the whole cluster
    static constexpr int SMEM_BYTES =
        kClStages * STAGE_BYTES + (SCRATCH_FLOATS + RECV_FLOATS) * 4 + (2 * kClStages + 1) * 8 + 16;
};

struct ClusterArgs {
    const char* q;
    const char* kplane;
    const char* vplane;
    const char* k_new;     // [B][1][Hkv][D] rows to append, or nullptr: attention only
    const char* v_new;
    float* out;
    int* status;
    int n;                 // rows per unit, the appended one included
    int row_stride;
    int tpu;               // tiles per unit
    int capacity;          // max_seq
    float scale_log2;
    int safe_rows;
    const int* n_extra;    // graph replay: rows the slot has grown by since the launch was recorded, or nullptr
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive (release, cluster scope) on an mbarrier in another block's shared memory.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kClThreads, 1) decode_cluster_kernel(const ClusterArgs a_in) {
    using S = ClusterShape<T, D, G>;
    using Math = ScalarMath<T, D, G, S::NG, S::TN>;
    constexpr int RB = S::RB, LPR = S::LPR, TN = S::TN;
    ClusterArgs a = a_in;
    const bool append = a.k_new != nullptr;
    bool over = false;
    if (a.n_extra != nullptr) {   // a replayed launch (see the split-K kernel): lengths have grown on the device
        a.n += *a.n_extra;
        over = a.n > a.capacity;  // only a replay can outrun the capacity: nothing is appended then
        if (over) a.n = a.capacity;
        a.tpu = (a.n + TN - 1) / TN;
    }

    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* stage_base = smem;
    float* scratch = reinterpret_cast<float*>(smem + kClStages * S::STAGE_BYTES);
    float* recv = scratch + S::SCRATCH_FLOATS;                 // [cluster size][G][D + 2], used in rank 0 only
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(recv + S::RECV_FLOATS);
    uint64_t* empty_bar = full_bar + kClStages;
    uint64_t* pieces_bar = empty_bar + kClStages;              // one arrival per block of the cluster
    volatile int* abort_flag = reinterpret_cast<volatile int*>(pieces_bar + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
    const long long u = blockIdx.x / csize;                    // the cluster's unit
    const int t0 = (int)(((long long)rank * a.tpu) / csize);   // this block's tiles of the unit
    const int t1 = (int)(((long long)(rank + 1) * a.tpu) / csize);
    const int new_tile = append && !over ? (a.n - 1) / TN : -1;   // tile that holds the appended row

    if (tid == 0) {
        for (int s = 0; s < kClStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kClWarps);
        }
        mbar_init(pieces_bar, csize);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        fence_mbar_init();
    }
    __syncthreads();
    cluster_sync_all();      // rank 0's barrier exists before any block arrives on it

    if (warp == kClWarps) {
        // ------------------------------ producer ------------------------------
        // lane 0 issues the copies; after the wait for the previous kernel all lanes store the
        // appended row to the pool if this block's share holds it
        bool ok = true;
        int it = 0;
        auto issue = [&](int ti, int st, bool arm, bool kv, bool qpart) {
            const int row0 = ti * TN;
            const int rows = min(TN, a.n - row0);
            const bool has_new = ti == new_tile;
            const int old_rows = has_new ? rows - 1 : rows;      // rows that are in the pool already
            const bool with_q = ti == t0;
            unsigned char* sb = stage_base + st * S::STAGE_BYTES;
            if (arm) mbar_arrive_expect_tx(&full_bar[st], 2u * rows * RB + (with_q ? S::QBYTES : 0));
            if (kv) {
                if (old_rows > 0) {
                    const long long off = (u * a.row_stride + row0) * (long long)RB;
                    bulk_g2s(sb, a.kplane + off, (uint32_t)old_rows * RB, &full_bar[st]);
                    bulk_g2s(sb + kClTileBytes, a.vplane + off, (uint32_t)old_rows * RB, &full_bar[st]);
                }
                if (has_new) {
                    bulk_g2s(sb + old_rows * RB, a.k_new + u * RB, RB, &full_bar[st]);
                    bulk_g2s(sb + kClTileBytes + old_rows * RB, a.v_new + u * RB, RB, &full_bar[st]);
                }
            }
            if (qpart && with_q) bulk_g2s(sb + 2 * kClTileBytes, a.q + u * (long long)S::QBYTES, S::QBYTES, &full_bar[st]);
        };
        int npre = 0;
        if (lane == 0) {
            // before the previous kernel is known to have finished: only tiles made of rows that
            // nothing in flight writes; q, newer rows and the appended row come after the wait
            for (; npre < kClStages && t0 + npre < t1; ++npre) {
                const int ti = t0 + npre;
                if ((long long)(ti + 1) * TN > a.safe_rows || ti == new_tile) break;
                issue(ti, npre, true, true, false);
            }
        }
        pdl_wait();
        pdl_launch_dependents();
        if (over) {
            if (append && lane == 0 && rank == 0) atomicExch(a.status, 4);
        } else if (new_tile >= t0 && new_tile < t1) {
            const long long dst = (u * a.row_stride + (a.n - 1)) * (long long)RB;
            for (int i = lane; i < 2 * LPR; i += 32) {
                const bool isv = i >= LPR;
                const int c = isv ? i - LPR : i;
                const uint4 val = *reinterpret_cast<const uint4*>((isv ? a.v_new : a.k_new) + u * RB + c * 16);
                *reinterpret_cast<uint4*>(const_cast<char*>(isv ? a.vplane : a.kplane) + dst + c * 16) = val;
            }
        }
        if (lane == 0) {
            for (int j = 0; j < npre; ++j) issue(t0 + j, j, false, false, true);
            it = npre;
            for (int ti = t0 + npre; ti < t1 && ok; ++ti, ++it) {
                const int st = it % kClStages;
                if (it >= kClStages) ok = mbar_wait_bounded(&empty_bar[st], ((it / kClStages) - 1) & 1, abort_flag, a.status);
                if (!ok) break;
                issue(ti, st, true, true, true);
            }
            if (!ok) {
                for (int j = max(0, it - kClStages); j < it; ++j)
                    mbar_wait_bounded(&full_bar[j % kClStages], (j / kClStages) & 1, abort_flag + 1, a.status);
            }
        }
        return;
    }

    // ---------------------------------- consumers ----------------------------------
    pdl_wait();
    pdl_launch_dependents();
    const int lig = lane & (LPR - 1);
    const int grp = warp * S::GPW + lane / LPR;
    typename Math::State st_;
    Math::reset(st_);
    int it = 0;
    for (int ti = t0; ti < t1; ++ti, ++it) {
        const int st = it % kClStages;
        if (!mbar_wait_bounded(&full_bar[st], (it / kClStages) & 1, abort_flag, a.status)) return;
        const unsigned char* ks = stage_base + st * S::STAGE_BYTES;
        const unsigned char* vs = ks + kClTileBytes;
        if (ti == t0) Math::load_q(st_, vs + kClTileBytes, lig, a.scale_log2);
        Math::tile(st_, ks, vs, min(TN, a.n - ti * TN), lig, grp);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[st]);
    }
    // this block's piece goes to slot `rank` of rank 0's receive buffer (a block without tiles
    // sends the neutral piece: max -1e30, sum 0)
    const uint32_t slot = map_to_rank(smem_u32(recv), 0) + rank * S::PIECE_FLOATS * 4;
    Math::template merge<kClConsumers>(st_, scratch, tid, lig, grp, [&](int g, int d, float o, float M, float den) {
        const uint32_t row = slot + g * (D + 2) * 4;
        st_cluster_f32(row + d * 4, o);
        if (d == 0) {
            st_cluster_f32(row + D * 4, M);
            st_cluster_f32(row + (D + 1) * 4, den);
        }
    });
    named_bar_sync(1, kClConsumers);      // every store of the piece has been issued
    if (tid == 0) mbar_arrive_remote(map_to_rank(smem_u32(pieces_bar), 0));   // release: the piece is visible to rank 0
    if (rank != 0) return;

    // ---- rank 0: all pieces are here; merge them in rank order ----
    if (!mbar_try_wait_cluster(pieces_bar, 0)) {
        const unsigned long long tstart = globaltimer_ns();
        uint32_t spins = 0;
        while (!mbar_try_wait_cluster(pieces_bar, 0)) {
            if ((++spins & 0xffu) == 0 && (abort_flag[0] != 0 || globaltimer_ns() - tstart > kWaitLimitNs)) {
                abort_flag[0] = 1;
                atomicExch(a.status, kDevTimeout);
                return;
            }
        }
    }
    for (int idx = tid; idx < G * D; idx += kClConsumers) {
        const int g = idx / D, d = idx - g * D;
        float M = -1.0e30f;
        for (uint32_t c = 0; c < csize; ++c) M = fmaxf(M, recv[(c * G + g) * (D + 2) + D]);
        float o = 0.f, den = 0.f;
        for (uint32_t c = 0; c < csize; ++c) {
            const float* p = recv + (c * G + g) * (D + 2);
            const float w = fast_exp2(p[D] - M);
            o = fmaf(w, p[d], o);
            den = fmaf(w, p[D + 1], den);
        }
        a.out[(u * G + g) * D + d] = o / den;
    }
}

template <typename T, int D, int G>
cudaError_t set_attr_cluster() {
    cudaError_t e = cudaFuncSetAttribute(decode_cluster_kernel<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ClusterShape<T, D, G>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_cluster_kernel<T, D, G>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
}

template <typename T, int D>
cudaError_t set_attr_cluster_groups() {
    cudaError_t e;
    if ((e = set_attr_cluster<T, D, 1>()) != cudaSuccess) return e;
    if ((e = set_attr_cluster<T, D, 2>()) != cudaSuccess) return e;
    if ((e = set_attr_cluster<T, D, 4>()) != cudaSuccess) return e;
    return set_attr_cluster<T, D, 8>();
}

template <typename T, int D, int G>
cudaError_t launch_cluster_one(const ClusterArgs& ka, int units, int csize, bool programmatic, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * csize));
    cfg.blockDim = dim3(kClThreads);
    cfg.dynamicSmemBytes = ClusterShape<T, D, G>::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, decode_cluster_kernel<T, D, G>, ka);
}

template <typename T, int D>
cudaError_t launch_cluster_groups(int G, const ClusterArgs& ka, int units, int csize, bool pdl, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_cluster_one<T, D, 1>(ka, units, csize, pdl, stream);
        case 2: return launch_cluster_one<T, D, 2>(ka, units, csize, pdl, stream);
        case 4: return launch_cluster_one<T, D, 4>(ka, units, csize, pdl, stream);
        case 8: return launch_cluster_one<T, D, 8>(ka, units, csize, pdl, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t init_cluster_kernels(int* max_cluster_size) {
    cudaError_t e;
    if ((e = set_attr_cluster_groups<__nv_bfloat16, 128>()) != cudaSuccess) return e;
    if ((e = set_attr_cluster_groups<__nv_bfloat16, 64>()) != cudaSuccess) return e;
    if ((e = set_attr_cluster_groups<float, 128>()) != cudaSuccess) return e;
    if ((e = set_attr_cluster_groups<float, 64>()) != cudaSuccess) return e;
    // the largest cluster the device can place with this kernel's shared-memory footprint
    *max_cluster_size = 1;
    for (int cs = kMaxClusterSize; cs >= 2; cs >>= 1) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)cs);
        cfg.blockDim = dim3(kClThreads);
        cfg.dynamicSmemBytes = ClusterShape<__nv_bfloat16, 128, 8>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, decode_cluster_kernel<__nv_bfloat16, 128, 8>, &cfg) == cudaSuccess &&
            clusters > 0) {
            *max_cluster_size = cs;
            break;
        }
        (void)cudaGetLastError();
    }
    return cudaSuccess;
}

int cluster_tile_rows(int D, int dtype) { return kClTileBytes / (D * (dtype == 0 ? 2 : 4)); }

bool plan_decode_cluster(int units, int n, int G, int D, int dtype, int sm_count, int max_cluster_size,
                         DecodePlan* plan) {
    if (G != 1 && G != 2 && G != 4 && G != 8) return false;
    if (max_cluster_size < 2) return false;
    plan->tile_rows = cluster_tile_rows(D, dtype);
    plan->tpu = (n + plan->tile_rows - 1) / plan->tile_rows;
    plan->T = (long long)units * plan->tpu;
    // blocks per unit: a power of two up to 16, no more than the unit has tiles, and no more
    // blocks in all than about two per SM
    int cs = 1;
    while (cs * 2 <= max_cluster_size && cs * 2 <= plan->tpu && (long long)units * cs * 2 <= 2LL * sm_count) cs *= 2;
    plan->NC = units * cs;
    plan->kernel = 3;
    plan->geom = cs;
    return true;
}

cudaError_t launch_decode_cluster(const DecodeArgs& a, const DecodePlan& plan, const void* k_new, const void* v_new,
                                  int capacity, cudaStream_t stream) {
    ClusterArgs ka;
    ka.q = (const char*)a.q;
    ka.kplane = (const char*)a.kplane;
    ka.vplane = (const char*)a.vplane;
    ka.k_new = (const char*)k_new;
    ka.v_new = (const char*)v_new;
    ka.out = a.out;
    ka.status = a.status;
    ka.n = a.n;
    ka.row_stride = a.row_stride;
    ka.tpu = plan.tpu;
    ka.capacity = capacity;
    ka.scale_log2 = a.scale_log2;
    ka.safe_rows = a.programmatic ? a.safe_rows : 0;
    ka.n_extra = a.n_extra;
    const bool pdl = a.programmatic;
    const int cs = plan.geom;
    if (a.dtype == 0) {
        if (a.D == 128) return launch_cluster_groups<__nv_bfloat16, 128>(a.G, ka, a.units, cs, pdl, stream);
        if (a.D == 64) return launch_cluster_groups<__nv_bfloat16, 64>(a.G, ka, a.units, cs, pdl, stream);
    } else {
        if (a.D == 128) return launch_cluster_groups<float, 128>(a.G, ka, a.units, cs, pdl, stream);
        if (a.D == 64) return launch_cluster_groups<float, 64>(a.G, ka, a.units, cs, pdl, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace kvs
