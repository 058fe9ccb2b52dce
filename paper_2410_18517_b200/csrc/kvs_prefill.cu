// Prefill attention with the sharing strategy on the 5th-generation tensor cores.
//
// n_q queries per head (the newest n_q positions of the slot the layer reads, causal mask)
// against the slot's K/V rows: a dense contraction, so it runs on tcgen05.mma with the
// accumulators in tensor memory.  One thread block = 128 queries of one (sequence, q-head):
//   warp 4 (one lane)  TMA producer: Q tile once, then K and V tiles of 128 keys
//   warp 5 (one lane)  MMA issuer:   S = Q K^T  (128x128x128, bf16 -> fp32 in TMEM)
//                                    O += P V with P = P_hi + P_lo (two bf16 terms, read from TMEM)
//   warps 0..3         softmax: thread r owns query row r = TMEM lane r; reads S with
//                      tcgen05.ld, writes P_hi / P_lo over S with tcgen05.st, and rescales the
//                      output row in TMEM only when the running maximum grows by more than 2^8
// Two blocks share an SM (96 KiB of shared memory and 256 TMEM columns each), so one block's
// softmax overlaps the other's tensor-core work.  K/V/Q tiles land in the 128-byte-swizzled
// layout the MMA shared-memory descriptors expect (K and Q K-major, V MN-major).
// bf16 storage, head size 128.
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
constexpr int kPfSmemBytes = 1024 + 3 * kPfMatBytes /*Q, K, V*/ + 256;
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

// Same, with the A operand read from tensor memory (row = lane, two bf16 per 32-bit column).
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t"
        "}\n" ::"r"(tmem_d),
        "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

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

// 32 fp32 columns of this thread's TMEM lane, written back.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,"
        "%31,%32};" ::"r"(taddr),
        "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), "f"(v[9]),
        "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "f"(v[16]), "f"(v[17]), "f"(v[18]),
        "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]), "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]),
        "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
        : "memory");
}

// 16 packed 32-bit columns (32 bf16 values) of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
        "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
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

// One softmax pass over a 32-column chunk of S: p = 2^(x*scale - m_ref) (0 where masked),
// split into bf16 hi and lo words (2 keys per word).  Returns the chunk's sum of p.
// max(a, b, c) in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// One softmax pass over a 32-column chunk of S: p = 2^(x*scale - m_ref) (0 where masked),
// split into bf16 hi and lo words (2 keys per word).  Returns the chunk's sum of p.  The scale,
// the sum and the hi/lo split use the packed two-float instructions.
template <bool MASK>
__device__ __forceinline__ float softmax_chunk(const float (&x)[32], float scale_log2, float m_ref, int key_first,
                                               int limit, uint32_t (&hi)[16], uint32_t (&lo)[16]) {
    const float2 sc = make_float2(scale_log2, scale_log2), nm = make_float2(-m_ref, -m_ref);
    const float2 minus1 = make_float2(-1.f, -1.f);
    float2 sum = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const float2 t = __ffma2_rn(make_float2(x[i], x[i + 1]), sc, nm);
        float2 p = make_float2(fast_exp2(t.x), fast_exp2(t.y));
        if (MASK) {
            p.x = (key_first + i <= limit) ? p.x : 0.f;
            p.y = (key_first + i + 1 <= limit) ? p.y : 0.f;
        }
        sum = __fadd2_rn(sum, p);
        const uint32_t h = pack2_bf16(p.x, p.y);
        hi[i >> 1] = h;
        const float2 r = __ffma2_rn(make_float2(__uint_as_float(h << 16), __uint_as_float(h & 0xffff0000u)), minus1, p);
        lo[i >> 1] = pack2_bf16(r.x, r.y);
    }
    return sum.x + sum.y;
}

__global__ void __launch_bounds__(kPfThreads, 2)
    prefill_attention_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                         const PrefillArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sQ = smem;
    unsigned char* sK = sQ + kPfMatBytes;
    unsigned char* sV = sK + kPfMatBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + kPfMatBytes);
    uint64_t* q_full = bars;
    uint64_t* k_full = bars + 1;
    uint64_t* k_empty = bars + 2;
    uint64_t* v_full = bars + 3;
    uint64_t* v_empty = bars + 4;
    uint64_t* s_full = bars + 5;
    uint64_t* p_full = bars + 6;        // 128 arrivals
    uint64_t* o_full = bars + 7;
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
        for (int i = 0; i < 8; ++i) mbar_init(&bars[i], i == 6 ? 128 : 1);
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
    const uint32_t tmem_s = tmem_base;         // S (fp32, 128 columns); P_hi / P_lo (bf16 pairs) overwrite it
    const uint32_t tmem_o = tmem_base + 128;   // running output rows

    if (warp == 4) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            mbar_arrive_expect_tx(q_full, kPfMatBytes);
            tma_load_4d(sQ, &tmap_q, 0, hq, q0, b, q_full);
            tma_load_4d(sQ + kPfHalfBytes, &tmap_q, 64, hq, q0, b, q_full);
            const long long unit_row = ((long long)b * Hkv + hk) * a.row_stride;
            for (int j = 0; j < nt; ++j) {
                const long long row = unit_row + (long long)j * kPfTile;
                if (j >= 1 && !mbar_wait_bounded(k_empty, (j - 1) & 1, abort_flag, a.status)) break;
                mbar_arrive_expect_tx(k_full, kPfMatBytes);
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int rb = 0; rb < 2; ++rb)
                        tma_load_2d_pf(sK + h * kPfHalfBytes + rb * 8192, &tmap_kv, h * 64, (int)(a.krow0 + row + rb * 64),
                                       k_full);
                if (j >= 1 && !mbar_wait_bounded(v_empty, (j - 1) & 1, abort_flag, a.status)) break;
                mbar_arrive_expect_tx(v_full, kPfMatBytes);
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int rb = 0; rb < 2; ++rb)
                        tma_load_2d_pf(sV + h * kPfHalfBytes + rb * 8192, &tmap_kv, h * 64, (int)(a.vrow0 + row + rb * 64),
                                       v_full);
            }
        }
    } else if (warp == 5) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(0);
            const uint32_t idesc_o = instr_desc_bf16(1);
            const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
            auto issue_s = [&]() {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 head-dim columns per step; 4 steps per 64-column block
                    const uint32_t off = (ks >> 2) * kPfHalfBytes + (ks & 3) * 32;
                    umma_bf16(tmem_s, smem_desc_sw128(q_addr + off, 16, 1024), smem_desc_sw128(k_addr + off, 16, 1024),
                              idesc_s, ks > 0);
                }
                umma_commit(s_full);
                umma_commit(k_empty);     // the K tile may be overwritten once S is done
            };
            bool ok = mbar_wait_bounded(q_full, 0, abort_flag, a.status) &&
                      mbar_wait_bounded(k_full, 0, abort_flag, a.status);
            if (ok) {
                tc_fence_after();
                issue_s();
            }
            for (int j = 0; j < nt && ok; ++j) {
                ok = mbar_wait_bounded(p_full, j & 1, abort_flag, a.status) &&
                     mbar_wait_bounded(v_full, j & 1, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 keys per step: 8 TMEM columns of bf16 pairs
                    // V is MN-major: 64 head-dim columns contiguous per key row, the other 64 one
                    // column block (LBO) away; 8-key groups 1024 bytes (SBO) apart
                    const uint64_t vdesc = smem_desc_sw128(v_addr + ks * 16 * 128, kPfHalfBytes, 1024);
                    umma_bf16_ts(tmem_o, tmem_s + ks * 8, vdesc, idesc_o, (j > 0) || (ks > 0));        // P_hi
                    umma_bf16_ts(tmem_o, tmem_s + 64 + ks * 8, vdesc, idesc_o, 1);                   // P_lo
                }
                umma_commit(o_full);
                umma_commit(v_empty);
                if (j + 1 < nt) {
                    ok = mbar_wait_bounded(k_full, (j + 1) & 1, abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    issue_s();
                }
            }
        }
    } else {
        // ------------------------------ softmax / output rows ------------------------------
        const int r = tid;                                   // query row in the block = TMEM lane
        const int qpos = min(q0 + r, a.T - 1);               // padding rows repeat the last query
        const int limit = a.n - a.T + qpos;                  // last key this query may see
        const int block_min_limit = a.n - a.T + q0;          // smallest limit of any row of the block
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const uint32_t ts = tmem_s + lane_addr, to = tmem_o + lane_addr;
        float m_ref = -1.0e30f, l = 0.f;                     // p is taken relative to m_ref (log2 domain)
        bool ok = true;
        for (int j = 0; j < nt; ++j) {
            ok = mbar_wait_bounded(s_full, j & 1, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            const int key0 = j * kPfTile;
            const bool mask = key0 + kPfTile - 1 > block_min_limit;   // block-uniform
            // pass 1: row maximum of the (masked) scores
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float x[32];
                tmem_ld32(ts + c * 32, x);
                if (mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, (key0 + c * 32 + i <= limit) ? x[i] : -INFINITY);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) mx = fmax3(mx, x[i], x[i + 1]);
                }
            }
            mx *= a.scale_log2;
            // The reference maximum only moves when the new one is more than 8 (a factor 256) above
            // it; then the output row and the sum accumulated so far are rescaled.  PV of the
            // previous tile has finished (S of this tile was issued after it), so O is quiet.
            const bool grow = mx > m_ref + 8.0f;
            if (__any_sync(0xffffffffu, grow)) {
                const float m_new = grow ? mx : m_ref;
                const float alpha = fast_exp2(m_ref - m_new);
                if (j > 0) {
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        float o[32];
                        tmem_ld32(to + c * 32, o);
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= alpha;
                        tmem_st32(to + c * 32, o);
                    }
                }
                l *= alpha;
                m_ref = m_new;
            }
            // pass 2, upper key half first: P_hi / P_lo overwrite S, so a column may only be written
            // once the scores in it have been read.  P_hi[keys k] -> columns k/2, P_lo -> 64 + k/2.
            uint32_t hi3[16], hi2[16], hi1[16], hi0[16], lo[16];
            float lsum = 0.f;
            {
                float x[32];
                tmem_ld32(ts + 96, x);
                lsum += mask ? softmax_chunk<true>(x, a.scale_log2, m_ref, key0 + 96, limit, hi3, lo)
                             : softmax_chunk<false>(x, a.scale_log2, m_ref, key0 + 96, limit, hi3, lo);
                tmem_ld32(ts + 64, x);          // all scores of columns 64..127 are now in registers
                tmem_st16(ts + 64 + 48, lo);
                lsum += mask ? softmax_chunk<true>(x, a.scale_log2, m_ref, key0 + 64, limit, hi2, lo)
                             : softmax_chunk<false>(x, a.scale_log2, m_ref, key0 + 64, limit, hi2, lo);
                tmem_st16(ts + 64 + 32, lo);
                tmem_ld32(ts + 32, x);
                lsum += mask ? softmax_chunk<true>(x, a.scale_log2, m_ref, key0 + 32, limit, hi1, lo)
                             : softmax_chunk<false>(x, a.scale_log2, m_ref, key0 + 32, limit, hi1, lo);
                tmem_st16(ts + 64 + 16, lo);
                tmem_ld32(ts, x);               // columns 0..63 are now in registers too
                tmem_st16(ts + 32, hi2);
                tmem_st16(ts + 48, hi3);
                tmem_st16(ts + 16, hi1);
                lsum += mask ? softmax_chunk<true>(x, a.scale_log2, m_ref, key0, limit, hi0, lo)
                             : softmax_chunk<false>(x, a.scale_log2, m_ref, key0, limit, hi0, lo);
                tmem_st16(ts, hi0);
                tmem_st16(ts + 64, lo);
            }
            l += lsum;
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            mbar_arrive(p_full);
        }
        if (ok) ok = mbar_wait_bounded(o_full, (nt - 1) & 1, abort_flag, a.status);
        if (ok) {
            tc_fence_after();
            const float inv = 1.0f / l;
            const bool store = q0 + r < a.T;
            float4* dst = reinterpret_cast<float4*>(a.out + (((long long)b * a.T + min(q0 + r, a.T - 1)) * a.Hq + hq) * 128);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float o[32];
                tmem_ld32(to + c * 32, o);
                if (store) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[c * 8 + i] = make_float4(o[4 * i] * inv, o[4 * i + 1] * inv, o[4 * i + 2] * inv, o[4 * i + 3] * inv);
                }
            }
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
