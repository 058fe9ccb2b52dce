// The data-parallel reductions of KVSharer's strategy search (Section 3.1, Algorithm 1), run
// on caches already resident in the pool:
//   layer_mean_kernel       sample-mean K/V representation of every cache slot over a slab of
//                           positions, streamed in long contiguous runs (one pass over the pool)
//   mean_distance_kernel    squared Euclidean distances of every pair of slots over that slab,
//                           from the means (which stay in L2 between the two kernels)
//   distance_sum_kernel     fixed-order sum of the per-block partial matrices
//   distance_finish_kernel  square roots, slot pairs expanded to layer pairs
//   mean_cosine_kernel      cosine similarity of the sample-means of two [S][dim] tensors
// All are bandwidth-bound: every cached element is read exactly once.
#include "kvs_device.cuh"
#include "kvs_kernels.h"

#include <algorithm>

namespace kvs {

namespace {

constexpr int kMeanThreads = 256;
constexpr int kMeanChunk = kMeanThreads * 8;   // positions per work item of the mean kernel: 8 per thread (16-byte loads of bf16)
constexpr int kDistThreads = 256;
constexpr int kDistChunk = 256;                // positions per chunk of the distance kernel: one per thread
constexpr int kDistStride = kDistChunk + 1;    // padded row of the mean tile (bank = slot + position)

// As many thread groups as the block has threads for (at most 16) share the positions of a chunk, so that
// every thread has a 4x4 block of slot pairs to work on.
__host__ __device__ inline int dist_groups(int items) {
    const int g = kDistThreads / items;
    return g < 1 ? 1 : (g > 16 ? 16 : g);
}

template <typename T>
__device__ __forceinline__ float2 load2(const T* p);
template <>
__device__ __forceinline__ float2 load2<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint32_t r = *reinterpret_cast<const uint32_t*>(p);
    return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
}
template <>
__device__ __forceinline__ float2 load2<float>(const float* p) {
    return *reinterpret_cast<const float2*>(p);
}

// Eight consecutive elements (16 bytes of bf16, 32 bytes of fp32) as floats, added into s.  The data is read
// exactly once: streaming loads, so that it is the first to leave the caches.
template <typename T>
__device__ __forceinline__ void add8_once(const T* p, float (&s)[8]);
template <>
__device__ __forceinline__ void add8_once<__nv_bfloat16>(const __nv_bfloat16* p, float (&s)[8]) {
    const uint4 r = __ldcs(reinterpret_cast<const uint4*>(p));
    float f[8];
    Unpack<__nv_bfloat16>::run(r, f);
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] += f[i];
}
template <>
__device__ __forceinline__ void add8_once<float>(const float* p, float (&s)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p + 4));
    s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w;
    s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
}

// ---- pass 1: sample means --------------------------------------------------------------------
// Positions p of a layer's representation run over (K or V, kv-head, row, column): P = 2 * Hkv * n * D.
// A work item is (slot, chunk of kMeanChunk positions of the slab [p0, p1)): every thread owns 8
// consecutive positions and adds the B samples' values, which lie one (sequence) stride apart, so a
// block reads B runs of 4 KiB (bf16) and neighbouring blocks continue the same runs.  The means go
// to `mean` as [slot][p - p0] fp32: small enough (the slab is sized for it) to stay in L2 until the
// distance kernel has read them.
struct MeanArgs {
    const char* pool;
    float* mean;               // [n_slots][slab]
    long long plane_bytes;
    int n_slots, B, Hkv, n, row_stride, D;
    long long p0, p1, slab;    // slab = positions per slot row of `mean` (>= p1 - p0)
};

template <typename T>
__global__ void __launch_bounds__(kMeanThreads) layer_mean_kernel(const MeanArgs a) {
    const long long unit_elems = (long long)a.n * a.D;            // cached elements of one (sequence, head)
    const long long kv_elems = (long long)a.Hkv * unit_elems;
    const long long bstride = (long long)a.Hkv * a.row_stride * a.D;
    const long long chunks = (a.p1 - a.p0 + kMeanChunk - 1) / kMeanChunk;
    const float inv_b = 1.0f / a.B;
    for (long long item = blockIdx.x; item < chunks * a.n_slots; item += gridDim.x) {
        const int slot = (int)(item / chunks);
        const long long p = a.p0 + (item - slot * chunks) * kMeanChunk + 8 * threadIdx.x;
        if (p >= a.p1) continue;
        // a unit holds a multiple of 8 elements, so the 8 positions never straddle two units
        const int kv = (int)(p / kv_elems);
        const long long rem = p - kv * kv_elems;
        const int h = (int)(rem / unit_elems);
        const long long e = rem - h * unit_elems;
        const T* base = reinterpret_cast<const T*>(a.pool + (long long)(2 * slot + kv) * a.plane_bytes) +
                        (long long)h * a.row_stride * a.D + e;
        float s8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 10
        for (int b = 0; b < a.B; ++b) add8_once<T>(base + b * bstride, s8);
        float4* dst = reinterpret_cast<float4*>(a.mean + (long long)slot * a.slab + (p - a.p0));
        dst[0] = make_float4(s8[0] * inv_b, s8[1] * inv_b, s8[2] * inv_b, s8[3] * inv_b);
        dst[1] = make_float4(s8[4] * inv_b, s8[5] * inv_b, s8[6] * inv_b, s8[7] * inv_b);
    }
}

// ---- pass 2: squared differences of every slot pair over the slab ---------------------------
// Per 512-position chunk a block copies every slot's means into a shared-memory tile ([slots][513],
// padded so that slot-pair reads are conflict-free), then 4x4 register blocks of slot pairs (upper
// triangle only: the matrix is symmetric) accumulate squared differences of the means (differences,
// not a Gram matrix, so near-identical layers do not cancel).  A block adds its chunks' sums to its
// own partial matrix, slab after slab, always in the same order.
struct DistArgs {
    const float* mean;         // [n_slots][slab]
    float* partial;            // [blocks][Sp*Sp]
    int S, Sp;                 // slots, rounded up to a multiple of 4
    long long count, slab;     // positions of this slab, row length of `mean`
    int first;                 // 1: the partial matrices start from zero with this launch
};

__global__ void __launch_bounds__(kDistThreads) mean_distance_kernel(const DistArgs a) {
    // The mean pass of the next slab is launched behind this kernel as a programmatic dependent: it may move
    // onto the SMs as soon as every block of this kernel has got here (it reads nothing this kernel writes).
    pdl_launch_dependents();
    extern __shared__ float M[];
    const int tid = threadIdx.x;
    const int tiles = a.Sp / 4;
    const int items = tiles * (tiles + 1) / 2;                     // 4x4 blocks of slot pairs with ti <= tj
    const int groups = dist_groups(items);                         // thread groups splitting the positions
    // A thread keeps one 4x4 block of slot pairs and one share of every chunk's positions for the whole launch
    // (groups * items <= threads), so its sixteen sums stay in registers from the first chunk to the last.
    const bool active = tid < groups * items;
    const int g = active ? tid / items : 0;
    int it = active ? tid - g * items : 0, ti = 0;
    while (it >= tiles - ti) {               // row ti of the upper triangle holds tiles - ti blocks
        it -= tiles - ti;
        ++ti;
    }
    const int tj = ti + it;
    const int per = (kDistChunk + groups - 1) / groups;
    const int q0 = g * per, q1 = min(kDistChunk, q0 + per);
    float d[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) d[x][y] = 0.f;
    for (int i = tid; i < (a.Sp - a.S) * kDistStride; i += kDistThreads) M[a.S * kDistStride + i] = 0.f;  // padding slots
    const long long chunks = (a.count + kDistChunk - 1) / kDistChunk;
    for (long long c = blockIdx.x; c < chunks; c += gridDim.x) {
        const long long p = c * kDistChunk;
        const int have = (int)min((long long)kDistChunk, a.count - p);
        __syncthreads();                     // the tile is free again (and, the first time, the padding is in place)
        // a warp reads 32 consecutive positions of one slot and stores them to 32 different banks; sixteen loads
        // are in flight per thread (the means come from L2)
#pragma unroll 16
        for (int i = tid; i < a.S * kDistChunk; i += kDistThreads) {
            const int sl = i / kDistChunk, q = i - sl * kDistChunk;
            M[sl * kDistStride + q] = q < have ? __ldcg(a.mean + (long long)sl * a.slab + p + q) : 0.f;
        }
        __syncthreads();
        if (active) {
            const float* mi_row = M + (4 * ti) * kDistStride;
            const float* mj_row = M + (4 * tj) * kDistStride;
#pragma unroll 2
            for (int q = q0; q < q1; ++q) {
                float mi[4];
                float2 mj[2];
#pragma unroll
                for (int x = 0; x < 4; ++x) mi[x] = mi_row[x * kDistStride + q];
                mj[0] = make_float2(mj_row[q], mj_row[kDistStride + q]);
                mj[1] = make_float2(mj_row[2 * kDistStride + q], mj_row[3 * kDistStride + q]);
                // two slot pairs per instruction (packed fp32): t = mi - mj, d += t * t
                const float2 minus1 = make_float2(-1.f, -1.f);
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 2; ++y) {
                        const float2 t = __ffma2_rn(mj[y], minus1, make_float2(mi[x], mi[x]));
                        const float2 r = __ffma2_rn(t, t, make_float2(d[x][2 * y], d[x][2 * y + 1]));
                        d[x][2 * y] = r.x;
                        d[x][2 * y + 1] = r.y;
                    }
            }
        }
    }
    // The groups' sums meet in shared memory (in the tile's place: the launch sizes it for both), are added
    // in group order and go to the block's own partial matrix.
    __syncthreads();
    for (int i = tid; i < groups * a.Sp * a.Sp; i += kDistThreads) M[i] = 0.f;
    __syncthreads();
    if (active) {
        float* dst = M + g * a.Sp * a.Sp;
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) dst[(4 * ti + x) * a.Sp + 4 * tj + y] = d[x][y];   // (g, block) has one owner
    }
    __syncthreads();
    for (int i = tid; i < a.Sp * a.Sp; i += kDistThreads) {
        float s = 0.f;
        for (int gg = 0; gg < groups; ++gg) s += M[gg * a.Sp * a.Sp + i];
        float* dst = a.partial + (long long)blockIdx.x * a.Sp * a.Sp + i;
        *dst = a.first ? s : *dst + s;
    }
}

// slot_dist2[r][c] (r < c) = sum over blocks of the (r, c) entries of their partial matrices: one warp
// per entry, lane l adds blocks l, l + 32, ... and the lanes are added in a fixed order.
__global__ void __launch_bounds__(256) distance_sum_kernel(const float* __restrict__ partial, double* __restrict__ slot_dist2,
                                                           int S, int Sp, int blocks) {
    const int entry = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (entry >= S * S) return;
    const int r = entry / S, c = entry - r * S;
    double s = 0.0;
    if (r < c)
        for (int b = lane; b < blocks; b += 32) s += partial[(long long)b * Sp * Sp + r * Sp + c];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) slot_dist2[entry] = s;
}

struct FinishArgs {
    int slot_of_layer[kMaxLayersSearch];
};

// dist[i][j] = sqrt of the entry of the two layers' slots (zero for two layers on one slot).
__global__ void distance_finish_kernel(const double* __restrict__ slot_dist2, float* __restrict__ dist, int L, int S,
                                       const FinishArgs f) {
    const int i = blockIdx.x, j = threadIdx.x;
    if (j >= L) return;
    const int si = f.slot_of_layer[i], sj = f.slot_of_layer[j];
    const int r = min(si, sj), c = max(si, sj);
    dist[i * L + j] = r == c ? 0.f : (float)sqrt(slot_dist2[r * S + c]);
}

// ---- mean cosine --------------------------------------------------------------------------
// A work item is a run of 2048 consecutive elements (8 per thread): the block adds the S samples of both
// tensors over it (2 * S runs of 4 KiB for bf16, each read once: streaming loads, ten in flight per thread),
// and neighbouring blocks continue the same runs.  Blocks are short-lived (an item or two each) rather than
// persistent: measured on the layer means, that keeps more distinct runs open at any moment and is a
// quarter faster.  Tensors that do not allow 16-byte loads go two elements at a time.
template <typename T>
__global__ void __launch_bounds__(256) mean_cosine_kernel(const T* __restrict__ a, const T* __restrict__ b, int S,
                                                          long long dim, double* __restrict__ partial) {
    float dot = 0.f, na = 0.f, nb = 0.f;
    const float inv = 1.0f / S;
    const bool wide = (dim % 8 == 0) && ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) % 32 == 0);
    if (wide) {
        for (long long e = 8 * ((long long)blockIdx.x * blockDim.x + threadIdx.x); e < dim; e += 8LL * gridDim.x * blockDim.x) {
            float sa[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, sb[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 5
            for (int s = 0; s < S; ++s) {
                add8_once<T>(a + s * dim + e, sa);
                add8_once<T>(b + s * dim + e, sb);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float x = sa[i] * inv, y = sb[i] * inv;
                dot = fmaf(x, y, dot);
                na = fmaf(x, x, na);
                nb = fmaf(y, y, nb);
            }
        }
    } else {
        for (long long e = 2 * ((long long)blockIdx.x * blockDim.x + threadIdx.x); e < dim; e += 2LL * gridDim.x * blockDim.x) {
            float ax = 0.f, ay = 0.f, bx = 0.f, by = 0.f;
            for (int s = 0; s < S; ++s) {
                const float2 va = load2<T>(a + s * dim + e), vb = load2<T>(b + s * dim + e);
                ax += va.x; ay += va.y; bx += vb.x; by += vb.y;
            }
            ax *= inv; ay *= inv; bx *= inv; by *= inv;
            dot = fmaf(ax, bx, fmaf(ay, by, dot));
            na = fmaf(ax, ax, fmaf(ay, ay, na));
            nb = fmaf(bx, bx, fmaf(by, by, nb));
        }
    }
    __shared__ float red[3][8];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        dot += __shfl_xor_sync(0xffffffffu, dot, o);
        na += __shfl_xor_sync(0xffffffffu, na, o);
        nb += __shfl_xor_sync(0xffffffffu, nb, o);
    }
    if ((threadIdx.x & 31) == 0) {
        red[0][threadIdx.x >> 5] = dot;
        red[1][threadIdx.x >> 5] = na;
        red[2][threadIdx.x >> 5] = nb;
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += red[threadIdx.x][w];
        partial[(long long)blockIdx.x * 3 + threadIdx.x] = s;
    }
}

// One block: thread t adds the partial sums of blocks t, t + 256, ... in that order, then the threads' sums
// are added pairwise in a fixed tree.
__global__ void __launch_bounds__(256) cosine_finish_kernel(const double* __restrict__ partial, int blocks,
                                                            float* __restrict__ out) {
    __shared__ double red[3][256];
    double dot = 0.0, na = 0.0, nb = 0.0;
    for (int c = threadIdx.x; c < blocks; c += 256) {
        dot += partial[3 * c];
        na += partial[3 * c + 1];
        nb += partial[3 * c + 2];
    }
    red[0][threadIdx.x] = dot;
    red[1][threadIdx.x] = na;
    red[2][threadIdx.x] = nb;
    __syncthreads();
    for (int o = 128; o >= 1; o >>= 1) {
        if (threadIdx.x < o)
#pragma unroll
            for (int k = 0; k < 3; ++k) red[k][threadIdx.x] += red[k][threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = (float)(red[0][0] / (sqrt(red[1][0]) * sqrt(red[2][0])));
}

}  // namespace

// Scratch layout: per-block partial matrices, then TWO slabs of means (the distance pass of one slab runs
// beside the mean pass of the next).
static size_t distance_partial_bytes(int n_slots) {
    const int Sp = (n_slots + 3) / 4 * 4;
    return ((size_t)kSearchMaxBlocks * Sp * Sp * sizeof(float) + 255) / 256 * 256;
}

size_t distance_scratch_bytes(int n_slots, long long positions) {
    // as many positions per slot as fit half the budget, in whole mean-kernel chunks
    long long slab = std::min<long long>(kMeanSlabBytes / 2 / ((long long)n_slots * 4), positions);
    slab = std::max<long long>((slab + kMeanChunk - 1) / kMeanChunk * kMeanChunk, kMeanChunk);
    return distance_partial_bytes(n_slots) + 2 * (size_t)n_slots * slab * sizeof(float);
}

cudaError_t launch_layer_distances(const void* pool, long long plane_bytes, const int* slot_of_layer, int L, int n_slots,
                                   int B, int Hkv, int n, int row_stride, int D, int dtype, float* scratch,
                                   size_t scratch_bytes, float* dist, int sm_count, int* launches, cudaStream_t stream) {
    if (L > kMaxLayersSearch) return cudaErrorInvalidValue;
    const int S = n_slots, Sp = (S + 3) / 4 * 4;
    const long long P = 2LL * Hkv * n * D;
    const size_t partial_bytes = distance_partial_bytes(S);
    if (scratch_bytes < partial_bytes + 2 * (size_t)S * kMeanChunk * sizeof(float)) return cudaErrorInvalidValue;
    // positions per slab: what half of the scratch holds, in whole mean-kernel chunks; slabs of equal size
    long long slab = (long long)((scratch_bytes - partial_bytes) / 2 / sizeof(float) / S) / kMeanChunk * kMeanChunk;
    const long long n_slabs = (P + slab - 1) / slab;
    slab = ((P + n_slabs - 1) / n_slabs + kMeanChunk - 1) / kMeanChunk * kMeanChunk;
    float* partial = scratch;
    float* mean[2];
    mean[0] = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + partial_bytes);
    mean[1] = mean[0] + (size_t)S * slab;

    const int tiles = Sp / 4, items = tiles * (tiles + 1) / 2;
    const int groups = dist_groups(items);
    const size_t smem = std::max((size_t)Sp * kDistStride, (size_t)groups * Sp * Sp) * sizeof(float);
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(mean_distance_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess)
        return e;
    // Two distance blocks per SM when there are few slabs (the last distance pass runs alone and should be
    // short); one when there are many: each pass then has a whole mean pass to hide behind, and the fewer
    // registers it holds the more mean blocks stay resident beside it (measured on 3, 4 and 21 slabs).
    const int per_sm = n_slabs >= 8 ? 1 : 2;
    const int dist_blocks = (int)std::min<long long>((std::min(slab, P) + kDistChunk - 1) / kDistChunk,
                                                     std::min(per_sm * sm_count, kSearchMaxBlocks));
    // One stream.  The distance pass of slab k is a plain launch (it waits for the mean pass of slab k and for
    // the distance pass before it); the mean pass of slab k + 1 follows it as a programmatic dependent that
    // never waits: it starts as soon as the distance blocks are resident and streams beside them.  It writes
    // the buffer that the distance pass of slab k - 1 read, which has completed by then.
    *launches = 0;
    int k = 0;
    for (long long p0 = 0; p0 < P; p0 += slab, ++k) {
        const int buf = k & 1;
        MeanArgs m;
        m.pool = (const char*)pool;
        m.mean = mean[buf];
        m.plane_bytes = plane_bytes;
        m.n_slots = S; m.B = B; m.Hkv = Hkv; m.n = n; m.row_stride = row_stride; m.D = D;
        m.p0 = p0; m.p1 = std::min(P, p0 + slab); m.slab = slab;
        const long long mean_items = (m.p1 - m.p0 + kMeanChunk - 1) / kMeanChunk * S;
        const int blocks = (int)std::min<long long>(mean_items, 16LL * sm_count);
        e = dtype == 0 ? launch_kernel(layer_mean_kernel<__nv_bfloat16>, dim3(blocks), dim3(kMeanThreads), 0, stream, k > 0, m)
                       : launch_kernel(layer_mean_kernel<float>, dim3(blocks), dim3(kMeanThreads), 0, stream, k > 0, m);
        if (e != cudaSuccess) return e;
        DistArgs a;
        a.mean = mean[buf];
        a.partial = partial;
        a.S = S; a.Sp = Sp;
        a.count = m.p1 - m.p0; a.slab = slab;
        a.first = p0 == 0 ? 1 : 0;
        // the same number of blocks for every slab: block b's partial matrix is its own, slab after slab
        mean_distance_kernel<<<dist_blocks, kDistThreads, smem, stream>>>(a);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        *launches += 2;
    }
    // the slabs of means are no longer needed: the first bytes hold the slot-pair sums for a moment
    double* slot_dist2 = reinterpret_cast<double*>(mean[0]);
    distance_sum_kernel<<<(S * S + 7) / 8, 256, 0, stream>>>(partial, slot_dist2, S, Sp, dist_blocks);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    FinishArgs f;
    for (int l = 0; l < L; ++l) f.slot_of_layer[l] = slot_of_layer[l];
    distance_finish_kernel<<<L, (L + 31) / 32 * 32, 0, stream>>>(slot_dist2, dist, L, S, f);
    *launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_mean_cosine(const void* a, const void* b, int S, long long dim, int dtype, double* partial,
                               float* out, int sm_count, cudaStream_t stream) {
    const long long pairs = (dim + 7) / 8;
    const int blocks = (int)std::max<long long>(1, std::min<long long>((pairs + 255) / 256, std::min(16 * sm_count, kCosineMaxBlocks)));
    if (dtype == 0)
        mean_cosine_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, S,
                                                                     dim, partial);
    else
        mean_cosine_kernel<float><<<blocks, 256, 0, stream>>>((const float*)a, (const float*)b, S, dim, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cosine_finish_kernel<<<1, 256, 0, stream>>>(partial, blocks, out);
    return cudaGetLastError();
}

}  // namespace kvs
