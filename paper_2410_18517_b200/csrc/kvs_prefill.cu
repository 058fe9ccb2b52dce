// Prefill attention with the sharing strategy on the 5th-generation tensor cores.
//
// n_q queries per head (the newest n_q positions of the slot the layer reads, causal mask)
// against the slot's K/V rows: a dense contraction, so it runs on tcgen05.mma with the
// accumulators in tensor memory.  One thread block = 128 queries of one (sequence, q-head):
//   warp 4 (one lane)  TMA producer: Q tile once, then K/V tiles of 128 keys, 2 stages
//   warp 5 (one lane)  MMA issuer:   S = Q K^T  (128x128x128, bf16 -> fp32 in TMEM)
//                                    O_tile = P V with P = P_hi + P_lo (two bf16 terms)
//   warps 0..3         softmax: thread r owns query row r = TMEM lane r; reads S with
//                      tcgen05.ld, keeps the running max / sum / output row in registers,
//                      writes P_hi, P_lo to shared memory in the swizzled K-major layout
// K/V/Q tiles land in the 128-byte-swizzled layout the MMA shared-memory descriptors expect
// (K and Q K-major, V MN-major).  bf16 storage, head size 128.
#include <cuda.h>

#include <algorithm>

#include "kvs_device.cuh"
#include "kvs_kernels.h"

namespace kvs {

namespace {

constexpr int kPfThreads = 192;
constexpr int kPfTile = 128;                 // queries per block and keys per tile
constexpr int kPfHalfBytes = kPfTile * 128;  // 128 rows x 64 bf16: one swizzled column block
constexpr int kPfMatBytes = 2 * kPfHalfBytes;  // a 128 x 128 bf16 operand
constexpr int kPfStages = 2;
constexpr int kPfSmemBytes = 1024 + kPfMatBytes /*Q*/ + kPfStages * 2 * kPfMatBytes /*K,V*/ + 2 * kPfMatBytes /*P*/ + 256;
constexpr uint32_t kTmemCols = 256;          // S: columns [0,128), O tile: [128,256)

__device__ __forceinline__ void tma_load_2d_pf(void* dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* tmap, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], "
        "[%6];" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate, bf16 A and B, A K-major,
// B K-major (b_mn = 0) or MN-major (b_mn = 1), M = 128, N = 128.
__device__ __forceinline__ uint32_t instr_desc_bf16(int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t"
        "}\n" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
        "%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct PrefillArgs {
    float* out;      // [B][T][Hq][128]
    int* status;
    int n;           // rows cached in the slot (after this pass's append)
    int T;           // queries per head
    int Hq, G;
    int row_stride;
    long long krow0, vrow0;  // first row of the slot's K / V plane in the pool-wide row numbering
    float scale_log2;
};

__global__ void __launch_bounds__(kPfThreads, 1)
    prefill_attention_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                         const PrefillArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sQ = smem;
    unsigned char* sKV = sQ + kPfMatBytes;                       // stage s: K at +s*2*Mat, V right after it
    unsigned char* sPhi = sKV + kPfStages * 2 * kPfMatBytes;
    unsigned char* sPlo = sPhi + kPfMatBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sPlo + kPfMatBytes);
    uint64_t* q_full = bars;            // 1
    uint64_t* kv_full = bars + 1;       // 2
    uint64_t* kv_empty = bars + 3;      // 2
    uint64_t* s_full = bars + 5;        // 1
    uint64_t* p_full = bars + 6;        // 1 (128 arrivals)
    uint64_t* o_full = bars + 7;        // 1
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 9);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qb = gridDim.x - 1 - blockIdx.x;       // blocks with the most keys first
    const int hq = blockIdx.y, b = blockIdx.z;
    const int hk = hq / a.G;
    const int Hkv = a.Hq / a.G;
    const int q0 = qb * kPfTile;
    // last key any query of this block may see, and the tiles that cover keys 0..that
    const int last_key = min(a.n - a.T + q0 + kPfTile - 1, a.n - 1);
    const int nt = last_key / kPfTile + 1;

    if (tid == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < kPfStages; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], 1);
        }
        mbar_init(s_full, 1);
        mbar_init(p_full, 128);
        mbar_init(o_full, 1);
        abort_flag[0] = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_s = tmem_base;
    const uint32_t tmem_o = tmem_base + 128;

    if (warp == 4) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            mbar_arrive_expect_tx(q_full, kPfMatBytes);
            tma_load_4d(sQ, &tmap_q, 0, hq, q0, b, q_full);
            tma_load_4d(sQ + kPfHalfBytes, &tmap_q, 64, hq, q0, b, q_full);
            const long long unit_row = ((long long)b * Hkv + hk) * a.row_stride;
            for (int j = 0; j < nt; ++j) {
                const int s = j & 1;
                if (j >= kPfStages &&
                    !mbar_wait_bounded(&kv_empty[s], ((j >> 1) - 1) & 1, abort_flag, a.status))
                    break;
                unsigned char* sK = sKV + s * 2 * kPfMatBytes;
                unsigned char* sV = sK + kPfMatBytes;
                mbar_arrive_expect_tx(&kv_full[s], 2 * kPfMatBytes);
                const long long row = unit_row + (long long)j * kPfTile;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int rb = 0; rb < 2; ++rb) {
                        tma_load_2d_pf(sK + h * kPfHalfBytes + rb * 8192, &tmap_kv, h * 64, (int)(a.krow0 + row + rb * 64),
                                       &kv_full[s]);
                        tma_load_2d_pf(sV + h * kPfHalfBytes + rb * 8192, &tmap_kv, h * 64, (int)(a.vrow0 + row + rb * 64),
                                       &kv_full[s]);
                    }
            }
        }
    } else if (warp == 5) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(0);
            const uint32_t idesc_o = instr_desc_bf16(1);
            const uint32_t q_addr = smem_u32(sQ), phi_addr = smem_u32(sPhi), plo_addr = smem_u32(sPlo);
            auto issue_s = [&](int j) {
                const uint32_t k_addr = smem_u32(sKV + (j & 1) * 2 * kPfMatBytes);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 head-dim columns per step; 4 steps per 64-column block
                    const uint32_t off = (ks >> 2) * kPfHalfBytes + (ks & 3) * 32;
                    umma_bf16(tmem_s, smem_desc_sw128(q_addr + off, 16, 1024), smem_desc_sw128(k_addr + off, 16, 1024),
                              idesc_s, ks > 0);
                }
                umma_commit(s_full);
            };
            bool ok = mbar_wait_bounded(q_full, 0, abort_flag, a.status) &&
                      mbar_wait_bounded(&kv_full[0], 0, abort_flag, a.status);
            if (ok) {
                tc_fence_after();
                issue_s(0);
            }
            for (int j = 0; j < nt && ok; ++j) {
                ok = mbar_wait_bounded(p_full, j & 1, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t v_addr = smem_u32(sKV + (j & 1) * 2 * kPfMatBytes + kPfMatBytes);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 keys per step
                    const uint32_t a_off = (ks >> 2) * kPfHalfBytes + (ks & 3) * 32;
                    // V is MN-major: 64 head-dim columns contiguous per key row, the other 64 one
                    // column block (LBO) away; 8-key groups 1024 bytes (SBO) apart
                    const uint64_t vdesc = smem_desc_sw128(v_addr + ks * 16 * 128, kPfHalfBytes, 1024);
                    umma_bf16(tmem_o, smem_desc_sw128(phi_addr + a_off, 16, 1024), vdesc, idesc_o, ks > 0);
                    umma_bf16(tmem_o, smem_desc_sw128(plo_addr + a_off, 16, 1024), vdesc, idesc_o, 1);
                }
                umma_commit(o_full);
                umma_commit(&kv_empty[j & 1]);
                if (j + 1 < nt) {
                    ok = mbar_wait_bounded(&kv_full[(j + 1) & 1], ((j + 1) >> 1) & 1, abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_s(j + 1);
                }
            }
        }
    } else {
        // ------------------------------ softmax / output rows ------------------------------
        const int r = tid;                                   // query row in the block = TMEM lane
        const int qpos = min(q0 + r, a.T - 1);               // padding rows repeat the last query
        const int limit = a.n - a.T + qpos;                  // last key this query may see
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        float acc[128];
#pragma unroll
        for (int i = 0; i < 128; ++i) acc[i] = 0.f;
        float m = -1.0e30f, l = 0.f;
        bool ok = true;
        for (int j = 0; j < nt; ++j) {
            ok = mbar_wait_bounded(s_full, j & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const int key0 = j * kPfTile;
            // pass 1: row maximum of the masked, scaled scores
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float x[32];
                tmem_ld32(tmem_s + lane_addr + c * 32, x);
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    mx = fmaxf(mx, (key0 + c * 32 + i <= limit) ? x[i] * a.scale_log2 : -INFINITY);
            }
            const float m_new = fmaxf(m, mx);
            const float alpha = fast_exp2(m - m_new);
            // pass 2: p = 2^(x - m_new), split into two bf16 terms, into the swizzled A-operand layout
            float lsum = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float x[32];
                tmem_ld32(tmem_s + lane_addr + c * 32, x);
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = (key0 + c * 32 + i <= limit) ? fast_exp2(x[i] * a.scale_log2 - m_new) : 0.f;
                    const float p1 = (key0 + c * 32 + i + 1 <= limit) ? fast_exp2(x[i + 1] * a.scale_log2 - m_new) : 0.f;
                    lsum += p0 + p1;
                    const float h0 = __bfloat162float(__float2bfloat16_rn(p0));
                    const float h1 = __bfloat162float(__float2bfloat16_rn(p1));
                    hi[i >> 1] = pack2_bf16(h0, h1);
                    lo[i >> 1] = pack2_bf16(p0 - h0, p1 - h1);
                }
                // keys c*32 .. c*32+31 = column block c/2, 16-byte chunks (c%2)*4 .. +3 of row r
                const uint32_t row_off = (c >> 1) * kPfHalfBytes + r * 128;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t chunk = ((c & 1) * 4 + k) ^ (r & 7);
                    *reinterpret_cast<uint4*>(sPhi + row_off + chunk * 16) =
                        make_uint4(hi[4 * k], hi[4 * k + 1], hi[4 * k + 2], hi[4 * k + 3]);
                    *reinterpret_cast<uint4*>(sPlo + row_off + chunk * 16) =
                        make_uint4(lo[4 * k], lo[4 * k + 1], lo[4 * k + 2], lo[4 * k + 3]);
                }
            }
            l = l * alpha + lsum;
            m = m_new;
            tc_fence_before();
            fence_async_smem();
            mbar_arrive(p_full);
            // O_tile = P V of this tile, folded into the running output row
            ok = mbar_wait_bounded(o_full, j & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float o[32];
                tmem_ld32(tmem_o + lane_addr + c * 32, o);
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[c * 32 + i] = fmaf(acc[c * 32 + i], alpha, o[i]);
            }
            tc_fence_before();
        }
        if (ok && q0 + r < a.T) {
            const float inv = 1.0f / l;
            float4* dst = reinterpret_cast<float4*>(a.out + (((long long)b * a.T + (q0 + r)) * a.Hq + hq) * 128);
#pragma unroll
            for (int i = 0; i < 32; ++i)
                dst[i] = make_float4(acc[4 * i] * inv, acc[4 * i + 1] * inv, acc[4 * i + 2] * inv, acc[4 * i + 3] * inv);
        }
    }
    // every thread of every role ends here; tensor memory is released by the warp that took it
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t get_encode(EncodeFn* out) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
    *out = reinterpret_cast<EncodeFn>(fn);
    return cudaSuccess;
}

}  // namespace

cudaError_t init_prefill_kernels() {
    return cudaFuncSetAttribute(prefill_attention_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes);
}

// q: [B][T][Hq][128] bf16.  One block per (128 queries, q-head, sequence).
cudaError_t launch_prefill(const void* q, float* out, int* status, const void* pool_tensor_map, int B, int T, int Hq,
                           int G, int n, int row_stride, long long krow0, long long vrow0, float scale_log2,
                           cudaStream_t stream) {
    EncodeFn encode = nullptr;
    cudaError_t e = get_encode(&encode);
    if (e != cudaSuccess) return e;
    alignas(64) CUtensorMap tq;
    cuuint64_t dims[4] = {128, (cuuint64_t)Hq, (cuuint64_t)T, (cuuint64_t)B};
    cuuint64_t strides[3] = {128 * 2, (cuuint64_t)Hq * 128 * 2, (cuuint64_t)T * Hq * 128 * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kPfTile, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    PrefillArgs a;
    a.out = out;
    a.status = status;
    a.n = n;
    a.T = T;
    a.Hq = Hq;
    a.G = G;
    a.row_stride = row_stride;
    a.krow0 = krow0;
    a.vrow0 = vrow0;
    a.scale_log2 = scale_log2;
    dim3 grid((T + kPfTile - 1) / kPfTile, Hq, B);
    prefill_attention_tc<<<grid, kPfThreads, kPfSmemBytes, stream>>>(
        tq, *reinterpret_cast<const CUtensorMap*>(pool_tensor_map), a);
    return cudaGetLastError();
}

}  // namespace kvs
