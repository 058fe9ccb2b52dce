// The data-parallel reductions of KVSharer's strategy search (Section 3.1, Algorithm 1), run
// on caches already resident in the pool:
//   layer_distance_kernel   sample-mean K/V representation of every layer, then the squared
//                           Euclidean distance of every pair of layers (one pass over the pool)
//   distance_finish_kernel  fixed-order sum of the per-block partial matrices, square root
//   mean_cosine_kernel      cosine similarity of the sample-means of two [S][dim] tensors
// Both are bandwidth-bound: every cached element is read exactly once.
#include "kvs_device.cuh"
#include "kvs_kernels.h"

#include <algorithm>

namespace kvs {

namespace {

constexpr int kDistThreads = 256;
constexpr int kDistChunk = 512;          // positions per chunk: two per thread
constexpr int kDistStride = kDistChunk + 1;   // padded row of the mean tile (bank = layer + position)

// 1, 2, 4 or 8 thread groups share the positions of a chunk when there are few layer-pair blocks.
__host__ __device__ inline int dist_groups(int items) {
    int g = 1;
    while (g < 8 && 2 * g * items <= kDistThreads) g *= 2;
    return g;
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

// Eight consecutive elements as floats (16 bytes of bf16, 32 bytes of fp32), added into s.
template <typename T>
__device__ __forceinline__ void add8(const T* p, float (&s)[8]);
template <>
__device__ __forceinline__ void add8<__nv_bfloat16>(const __nv_bfloat16* p, float (&s)[8]) {
    const uint4 r = *reinterpret_cast<const uint4*>(p);
    float f[8];
    Unpack<__nv_bfloat16>::run(r, f);
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] += f[i];
}
template <>
__device__ __forceinline__ void add8<float>(const float* p, float (&s)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    s[0] += a.x; s[1] += a.y; s[2] += a.z; s[3] += a.w;
    s[4] += b.x; s[5] += b.y; s[6] += b.z; s[7] += b.w;
}

struct DistArgs {
    const char* pool;
    float* partial;            // [blocks][Lp*Lp]
    long long plane_bytes;
    int slot_of_layer[kMaxLayersSearch];
    int L, Lp;                 // layers, rounded up to a multiple of 4
    int B, Hkv, n, row_stride, D;
    long long P;               // positions: 2 * Hkv * n * D
};

// Shared memory: mean tile M[Lp][kDistStride] fp32, then accumulators acc[groups][Lp*Lp].
template <typename T>
__global__ void __launch_bounds__(kDistThreads) layer_distance_kernel(const DistArgs a) {
    extern __shared__ float sm[];
    float* M = sm;
    float* acc = sm + a.Lp * kDistStride;
    const int tid = threadIdx.x;
    const int tiles = a.Lp / 4;
    const int items = tiles * tiles;                               // 4x4 blocks of layer pairs
    const int groups = dist_groups(items);                         // thread groups splitting the positions
    for (int i = tid; i < groups * a.Lp * a.Lp; i += kDistThreads) acc[i] = 0.f;
    for (int i = tid; i < (a.Lp - a.L) * kDistStride; i += kDistThreads) M[a.L * kDistStride + i] = 0.f;  // padding layers
    __syncthreads();

    const long long unit_elems = (long long)a.n * a.D;            // cached elements of one (sequence, head)
    const long long kv_elems = (long long)a.Hkv * unit_elems;
    const long long chunks = (a.P + kDistChunk - 1) / kDistChunk;
    const float inv_b = 1.0f / a.B;
    for (long long c = blockIdx.x; c < chunks; c += gridDim.x) {
        // ---- means of this chunk's positions, all layers ----
        // 64 groups of 8 consecutive positions (16-byte loads); the 4 quarters of the block take
        // every fourth layer.  A unit holds a multiple of 8 elements, so a group never straddles two.
        // Position 8*pg + i of the chunk is stored at column 64*i + pg: the order of positions inside
        // a chunk is irrelevant to the sums and this one keeps the stores conflict-free.
        {
            const int pg = tid & 63, lq = tid >> 6;
            const long long p = c * kDistChunk + 8 * pg;
            if (p < a.P) {
                const int kv = (int)(p / kv_elems);
                const long long rem = p - kv * kv_elems;
                const int h = (int)(rem / unit_elems);
                const long long e = rem - h * unit_elems;
                const long long bstride = (long long)a.Hkv * a.row_stride * a.D;
                for (int l = lq; l < a.L; l += 4) {
                    const T* base = reinterpret_cast<const T*>(a.pool + (long long)(2 * a.slot_of_layer[l] + kv) * a.plane_bytes) +
                                    (long long)h * a.row_stride * a.D + e;
                    float s8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
                    for (int b = 0; b < a.B; ++b) add8<T>(base + b * bstride, s8);
#pragma unroll
                    for (int i = 0; i < 8; ++i) M[l * kDistStride + 64 * i + pg] = s8[i] * inv_b;
                }
            } else {
                for (int l = lq; l < a.L; l += 4)
#pragma unroll
                    for (int i = 0; i < 8; ++i) M[l * kDistStride + 64 * i + pg] = 0.f;
            }
        }
        __syncthreads();
        // ---- squared differences of every layer pair over the chunk ----
        for (int w = tid; w < groups * items; w += kDistThreads) {
            const int g = w / items, it = w - g * items;
            const int ti = (it / tiles) * 4, tj = (it % tiles) * 4;
            float d[4][4];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) d[x][y] = 0.f;
            const int per = kDistChunk / groups;
            for (int q = g * per; q < (g + 1) * per; ++q) {
                float mi[4], mj[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    mi[x] = M[(ti + x) * kDistStride + q];
                    mj[x] = M[(tj + x) * kDistStride + q];
                }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) {
                        const float t = mi[x] - mj[y];
                        d[x][y] = fmaf(t, t, d[x][y]);
                    }
            }
            float* dst = acc + g * a.Lp * a.Lp;
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) dst[(ti + x) * a.Lp + tj + y] += d[x][y];   // (g, item) has one owner
        }
        __syncthreads();
    }
    for (int i = tid; i < a.Lp * a.Lp; i += kDistThreads) {
        float s = 0.f;
        for (int g = 0; g < groups; ++g) s += acc[g * a.Lp * a.Lp + i];
        a.partial[(long long)blockIdx.x * a.Lp * a.Lp + i] = s;
    }
}

__global__ void distance_finish_kernel(const float* __restrict__ partial, float* __restrict__ dist, int L, int Lp,
                                       int blocks) {
    const int i = blockIdx.x, j = threadIdx.x;
    if (j >= L) return;
    double s = 0.0;
    for (int c = 0; c < blocks; ++c) s += partial[(long long)c * Lp * Lp + i * Lp + j];
    dist[i * L + j] = (i == j) ? 0.f : (float)sqrt(s);
}

// ---- mean cosine --------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) mean_cosine_kernel(const T* __restrict__ a, const T* __restrict__ b, int S,
                                                          long long dim, double* __restrict__ partial) {
    float dot = 0.f, na = 0.f, nb = 0.f;
    const float inv = 1.0f / S;
    const bool wide = (dim % 8 == 0) && ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) % 32 == 0);
    if (wide) {
        for (long long e = 8 * ((long long)blockIdx.x * blockDim.x + threadIdx.x); e < dim; e += 8LL * gridDim.x * blockDim.x) {
            float sa[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, sb[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int s = 0; s < S; ++s) {
                add8<T>(a + s * dim + e, sa);
                add8<T>(b + s * dim + e, sb);
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

__global__ void cosine_finish_kernel(const double* __restrict__ partial, int blocks, float* __restrict__ out) {
    double dot = 0.0, na = 0.0, nb = 0.0;
    for (int c = 0; c < blocks; ++c) {
        dot += partial[3 * c];
        na += partial[3 * c + 1];
        nb += partial[3 * c + 2];
    }
    *out = (float)(dot / (sqrt(na) * sqrt(nb)));
}

}  // namespace

size_t distance_partial_bytes(int L) {
    const int Lp = (L + 3) / 4 * 4;
    return (size_t)kSearchMaxBlocks * Lp * Lp * sizeof(float);
}

cudaError_t launch_layer_distances(const void* pool, long long plane_bytes, const int* slot_of_layer, int L, int B,
                                   int Hkv, int n, int row_stride, int D, int dtype, float* partial, float* dist,
                                   int sm_count, cudaStream_t stream) {
    if (L > kMaxLayersSearch) return cudaErrorInvalidValue;
    DistArgs a;
    a.pool = (const char*)pool;
    a.partial = partial;
    a.plane_bytes = plane_bytes;
    for (int l = 0; l < L; ++l) a.slot_of_layer[l] = slot_of_layer[l];
    a.L = L;
    a.Lp = (L + 3) / 4 * 4;
    a.B = B; a.Hkv = Hkv; a.n = n; a.row_stride = row_stride; a.D = D;
    a.P = 2LL * Hkv * n * D;
    const int tiles = a.Lp / 4, items = tiles * tiles;
    const int groups = dist_groups(items);
    const size_t smem = ((size_t)a.Lp * kDistStride + (size_t)groups * a.Lp * a.Lp) * sizeof(float);
    const long long chunks = (a.P + kDistChunk - 1) / kDistChunk;
    const int blocks = (int)std::min<long long>(chunks, std::min(2 * sm_count, kSearchMaxBlocks));
    cudaError_t e;
    if (dtype == 0) {
        if ((e = cudaFuncSetAttribute(layer_distance_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem)) != cudaSuccess)
            return e;
        layer_distance_kernel<__nv_bfloat16><<<blocks, kDistThreads, smem, stream>>>(a);
    } else {
        if ((e = cudaFuncSetAttribute(layer_distance_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem)) != cudaSuccess)
            return e;
        layer_distance_kernel<float><<<blocks, kDistThreads, smem, stream>>>(a);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    distance_finish_kernel<<<L, a.Lp, 0, stream>>>(partial, dist, L, a.Lp, blocks);
    return cudaGetLastError();
}

cudaError_t launch_mean_cosine(const void* a, const void* b, int S, long long dim, int dtype, double* partial,
                               float* out, int sm_count, cudaStream_t stream) {
    const long long pairs = (dim + 7) / 8;
    const int blocks = (int)std::max<long long>(1, std::min<long long>((pairs + 255) / 256, std::min(4 * sm_count, kSearchMaxBlocks)));
    if (dtype == 0)
        mean_cosine_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, S,
                                                                     dim, partial);
    else
        mean_cosine_kernel<float><<<blocks, 256, 0, stream>>>((const float*)a, (const float*)b, S, dim, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cosine_finish_kernel<<<1, 1, 0, stream>>>(partial, blocks, out);
    return cudaGetLastError();
}

}  // namespace kvs
