// Device-side building blocks for sm_100a: mbarrier, 1-D bulk async copy
// (global -> this CTA's shared memory), bounded waits.  Inline PTX only.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kvs {

// Device status word values (mirrors kvs_status in the public header).
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 7;
constexpr int kDevBounds = 9;

// Tracing build (-DKVS_TRACE): the split-K and combine kernels stamp %globaltimer into a caller-provided
// buffer at fixed points (one row of kTraceSlots words per thread block and launch), from which the
// per-block timeline of a launch can be read.  In a normal build the stamps compile to nothing.
constexpr int kTraceSlots = 32;     // words per (launch, block)
constexpr int kTraceBlocks = 160;   // rows per launch: blocks 0..147 of the split-K kernel, rows 150 / 151 the
                                    // first / last block of the combine kernel
enum TraceSlot {
    kTrEntry = 0,          // kernel entry (thread 0)
    kTrProducerGo = 1,     // producer: its wait for the previous kernel has returned
    kTrConsumerGo = 2,     // consumers: their wait has returned
    kTrFirstTile = 3,      // the first tile (with q) has arrived
    kTrPiece = 4,          // 4 + 2k: piece k's tiles are done, 5 + 2k: piece k is merged and written (k < 8)
    kTrEnd = 20,           // consumers are done
    kTrPieces = 21,        // number of pieces of the block
    kTrProducerPre = 22,   // producer: early tiles issued, about to wait
    kTrSm = 23,            // the SM the block ran on
};
#ifdef KVS_TRACE
#define KVS_TRACE_STAMP(row, slot) do { if ((row) != nullptr) (row)[slot] = ::kvs::globaltimer_ns(); } while (0)
#define KVS_TRACE_VALUE(row, slot, v) do { if ((row) != nullptr) (row)[slot] = (unsigned long long)(v); } while (0)
#else
#define KVS_TRACE_STAMP(row, slot) do { (void)(row); } while (0)
#define KVS_TRACE_VALUE(row, slot, v) do { (void)(row); (void)(v); } while (0)
#endif

// Bounds-checking build (-DKVS_DEBUG_BOUNDS): every global offset the kernels compute for a pool
// plane, the query / new-row buffers or the partial results is checked against the buffer it
// must fall in.  The first violation is recorded in the status word (kDevBounds; nothing traps)
// and the access is redirected to offset 0 of the same buffer (reads) or dropped (writes), so
// that the launch still runs to its end.  In a normal build the checks compile to nothing.
#ifdef KVS_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(long long off, long long len, long long limit, int* status) {
    if (off >= 0 && len >= 0 && off + len <= limit) return true;
    atomicCAS(status, kDevOk, kDevBounds);
    return false;
}
#define KVS_BOUNDS_OK(off, len, limit, status) ::kvs::bounds_ok((long long)(off), (long long)(len), (long long)(limit), (status))
#else
#define KVS_BOUNDS_OK(off, len, limit, status) true
#endif

// A wait gives up after this many nanoseconds of wall time on the GPU.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned int sm_id() {
    unsigned int v;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(v));
    return v;
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
    // make the initialised barriers visible to the async (bulk-copy) proxy
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for the phase with the given parity to complete.  Bounded: gives up when
// limit_ns (by default kWaitLimitNs) have passed or when another thread of the CTA
// has already given up (*abort_flag != 0).  Returns false on giving up; the caller
// must then stop consuming data, and the status word is set to kDevTimeout.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                  int* status, unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 0xffu) == 0) {
            if (*abort_flag != 0) return false;
            if (globaltimer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicExch(status, kDevTimeout);
                return false;
            }
        }
    }
}

// A flag in global memory through which one thread block tells another, inside one launch, that
// data it wrote is ready: the writer stores with release semantics after a barrier with the threads
// that wrote the data, the reader polls with acquire semantics and then passes a barrier with the
// threads that will read it.
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
    asm volatile("st.release.gpu.global.b32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded like mbar_wait_bounded: false (status word set, *abort_flag raised) when the flag has not
// taken the value within the limit.
__device__ __forceinline__ bool flag_wait_bounded(const int* flag, int want, volatile int* abort_flag, int* status,
                                                  unsigned long long limit_ns = kWaitLimitNs) {
    if (ld_acquire_gpu(flag) == want) return true;
    const unsigned long long t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (ld_acquire_gpu(flag) == want) return true;
        if ((++spins & 0x3fu) == 0) {
            if (*abort_flag != 0) return false;
            if (globaltimer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicExch(status, kDevTimeout);
                return false;
            }
        }
    }
}

// 1-D bulk copy global -> shared memory of this CTA; completion is reported as
// `bytes` transaction bytes on `bar`.  Both addresses must be 16-byte aligned
// and `bytes` a non-zero multiple of 16.  (The destination state space is
// spelled shared::cluster; with no cluster launched that is this CTA's own
// shared memory.)
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Named barrier among `nthreads` threads (all of whole warps), id 1..15.
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 16 bytes of storage -> floats.  bf16 widens exactly (shift into the high half).
template <typename T>
struct Unpack;

template <>
struct Unpack<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void run(const uint4& r, float (&f)[8]) {
        f[0] = __uint_as_float(r.x << 16);
        f[1] = __uint_as_float(r.x & 0xffff0000u);
        f[2] = __uint_as_float(r.y << 16);
        f[3] = __uint_as_float(r.y & 0xffff0000u);
        f[4] = __uint_as_float(r.z << 16);
        f[5] = __uint_as_float(r.z & 0xffff0000u);
        f[6] = __uint_as_float(r.w << 16);
        f[7] = __uint_as_float(r.w & 0xffff0000u);
    }
};

template <>
struct Unpack<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void run(const uint4& r, float (&f)[4]) {
        f[0] = __uint_as_float(r.x);
        f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z);
        f[3] = __uint_as_float(r.w);
    }
};

}  // namespace kvs

namespace kvs {

// Programmatic dependent launch: a kernel launched with the programmatic-serialization
// attribute may start while its predecessor in the stream still runs.  pdl_wait() blocks
// until the predecessor has completed and its writes are visible (a no-op for a normal
// launch); pdl_launch_dependents() lets the successor's blocks be scheduled early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with or without the programmatic-serialization attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool programmatic, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace kvs

namespace kvs {

// The append of a decode step done by the attention kernel itself.  Called by all lanes of the
// producer warp of a split-K kernel, after the wait for the previous kernel: for every unit whose
// last tile lies in this block's share [t0, t1) of the tile line, the unit's new row (row n-1, not
// in the pool yet) is stored from the caller's buffers k_new / v_new ([units][RB] bytes) to the K
// and V planes.  Only this block ever fetches that tile, and it does so after this call: the
// proxy fence orders the warp's plain stores before the bulk (asynchronous-proxy) copies that
// lane 0 issues next.
template <int RB>
__device__ __forceinline__ void store_new_rows(int lane, long long t0, long long t1, int tpu, int n, int row_stride,
                                               const char* k_new, const char* v_new, char* kplane, char* vplane,
                                               long long plane_bytes, int units, int* status) {
    constexpr int LPR = RB / 16;
    if (t1 > t0) {
        const long long u0 = t0 / tpu, u1 = (t1 - 1) / tpu;
        for (long long u = u0; u <= u1; ++u) {
            const long long last = u * tpu + tpu - 1;
            if (last < t0 || last >= t1) continue;
            const long long dst = (u * row_stride + (n - 1)) * (long long)RB;
            if (!KVS_BOUNDS_OK(dst, RB, plane_bytes, status) || !KVS_BOUNDS_OK(u, 1, units, status)) continue;
            for (int i = lane; i < 2 * LPR; i += 32) {
                const bool isv = i >= LPR;
                const int c = isv ? i - LPR : i;
                const uint4 val = *reinterpret_cast<const uint4*>((isv ? v_new : k_new) + u * RB + c * 16);
                *reinterpret_cast<uint4*>((isv ? vplane : kplane) + dst + c * 16) = val;
            }
        }
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __syncwarp();
}

}  // namespace kvs
