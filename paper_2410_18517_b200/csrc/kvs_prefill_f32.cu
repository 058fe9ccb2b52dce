// Prefill attention for fp32 storage (the small configuration with fp32 Q/K/V): the same causal
// attention as the tensor-core kernel, computed with fp32 FMAs.  Prompts in fp32 are small by
// nature, so this is a plain kernel: one warp per query, keys in tiles of 32.
//   scores:  lane j takes key (tile * 32 + j): dot product of the query (in shared memory) with
//            the key's row
//   softmax: running maximum and sum per query, combined over the warp with shuffles
//   output:  lane l owns columns l, l + 32, ... of the output row and adds p_j * V[j][column] for
//            the tile's keys (coalesced reads of every value row)
#include "kvs_device.cuh"
#include "kvs_kernels.h"

namespace kvs {

namespace {

constexpr int kPf32Warps = 4;   // queries per block

struct Prefill32Args {
    const float* q;        // [B][T][Hq][D]
    float* out;            // [B][T][Hq][D]
    const float* kplane;   // [B][Hkv][row_stride][D]
    const float* vplane;
    int B, T, Hq, G, n, row_stride;
    float scale_log2;
};

template <int D>
__global__ void __launch_bounds__(kPf32Warps * 32) prefill_attention_f32(const Prefill32Args a) {
    constexpr int CPL = D / 32;                    // output columns per lane
    __shared__ float qs[kPf32Warps][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * kPf32Warps + warp;     // (b, i, hq), hq fastest: the q layout
    if (item >= (long long)a.B * a.T * a.Hq) return;
    const int hq = (int)(item % a.Hq);
    const long long bi = item / a.Hq;
    const int i = (int)(bi % a.T), b = (int)(bi / a.T);
    const float* qrow = a.q + item * D;
#pragma unroll
    for (int c = 0; c < CPL; ++c) qs[warp][lane + 32 * c] = qrow[lane + 32 * c] * a.scale_log2;
    __syncwarp();
    const long long unit = ((long long)b * (a.Hq / a.G) + hq / a.G) * a.row_stride * D;
    const float* K = a.kplane + unit;
    const float* V = a.vplane + unit;
    const int limit = a.n - a.T + i;               // last key this query may see (causal)
    float m = -1.0e30f, l = 0.f, acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
    for (int j0 = 0; j0 <= limit; j0 += 32) {
        const int j = j0 + lane;
        float s = -INFINITY;
        if (j <= limit) {
            const float4* kr = reinterpret_cast<const float4*>(K + (long long)j * D);
            float d = 0.f;
#pragma unroll 8
            for (int e = 0; e < D / 4; ++e) {
                const float4 kv = kr[e];
                d = fmaf(qs[warp][4 * e], kv.x, d);
                d = fmaf(qs[warp][4 * e + 1], kv.y, d);
                d = fmaf(qs[warp][4 * e + 2], kv.z, d);
                d = fmaf(qs[warp][4 * e + 3], kv.w, d);
            }
            s = d;
        }
        float tmax = s;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
        const float m_new = fmaxf(m, tmax);
        const float alpha = fast_exp2(m - m_new);
        const float p = fast_exp2(s - m_new);      // 0 for the lanes past the limit
        float psum = p;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
        l = l * alpha + psum;
        m = m_new;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] *= alpha;
        const int cnt = min(32, limit - j0 + 1);
        for (int t = 0; t < cnt; ++t) {
            const float pt = __shfl_sync(0xffffffffu, p, t);
            const float* vr = V + (long long)(j0 + t) * D;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] = fmaf(pt, vr[lane + 32 * c], acc[c]);
        }
    }
    float* orow = a.out + item * D;
    const float inv = 1.0f / l;
#pragma unroll
    for (int c = 0; c < CPL; ++c) orow[lane + 32 * c] = acc[c] * inv;
}

}  // namespace

cudaError_t launch_prefill_f32(const void* q, float* out, const void* kplane, const void* vplane, int B, int T, int Hq,
                               int G, int D, int n, int row_stride, float scale_log2, cudaStream_t stream) {
    Prefill32Args a;
    a.q = static_cast<const float*>(q);
    a.out = out;
    a.kplane = static_cast<const float*>(kplane);
    a.vplane = static_cast<const float*>(vplane);
    a.B = B; a.T = T; a.Hq = Hq; a.G = G; a.n = n; a.row_stride = row_stride;
    a.scale_log2 = scale_log2;
    const long long items = (long long)B * T * Hq;
    const unsigned blocks = (unsigned)((items + kPf32Warps - 1) / kPf32Warps);
    if (D == 128) prefill_attention_f32<128><<<blocks, kPf32Warps * 32, 0, stream>>>(a);
    else if (D == 64) prefill_attention_f32<64><<<blocks, kPf32Warps * 32, 0, stream>>>(a);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace kvs
