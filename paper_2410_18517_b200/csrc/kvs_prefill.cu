// Prefill attention with the sharing strategy on the 5th-generation tensor cores.
//
// n_q queries per head (the newest n_q positions of the slot the layer reads, causal mask)
// against the slot's K/V rows: a dense contraction, so it runs on tcgen05.mma with the
// accumulators in tensor memory.  One thread block = 128 queries of one (sequence, q-head),
// walking over the keys in tiles of 64:
//   warp 8 (one lane)  TMA producer: Q tile once, then K and V tiles, two stages each
//   warp 9 (one lane)  MMA issuer:   S = Q K^T  (128x64x128, bf16 -> fp32 in TMEM), into one
//                                    of two score buffers, so that S of tile j+1 is computed
//                                    while the softmax of tile j runs;
//                                    O += P V with P = P_hi + P_lo (two bf16 terms, read from TMEM)
//   warps 0..7         softmax: two threads per query row (= TMEM lane), warp w and warp w+4,
//                      32 keys of the tile each.  A thread reads its scores with tcgen05.ld,
//                      the two exchange their maxima through shared memory, then each writes
//                      its part of P_hi / P_lo over S with tcgen05.st; the output row in TMEM is
//                      rescaled only when the running maximum grows by more than 2^8
// Two blocks share an SM (99 KiB of shared memory and 256 TMEM columns each), so four key
// tiles are in flight per SM.  K/V/Q tiles land in the 128-byte-swizzled layout the MMA
// shared-memory descriptors expect (K and Q K-major, V MN-major).
// bf16 storage, head size 64 or 128.
#include <cuda.h>

#include <algorithm>

#include "kvs_device.cuh"
#include "kvs_kernels.h"

namespace kvs {

namespace {

constexpr int kPfSoftmaxWarps = 8;
constexpr int kPfThreads = (kPfSoftmaxWarps + 2) * 32;
constexpr int kPfTile = 128;                 // queries per block
constexpr int kPfKeys = 64;                  // keys per tile
constexpr int kPfQBlock = kPfTile * 128;     // one swizzled block of Q: 128 rows x 64 bf16 columns
constexpr int kPfKvBlock = kPfKeys * 128;    // one swizzled block of K or V: 64 rows x 64 bf16 columns
// Head size D = 64 or 128: rows are D/64 swizzled blocks wide.
template <int D>
struct PfShape {
    static constexpr int HALVES = D / 64;
    static constexpr int Q_BYTES = HALVES * kPfQBlock;
    static constexpr int KV_BYTES = HALVES * kPfKvBlock;
    static constexpr int Q_BUF = 2 * kPfQBlock;   // the Q tile; later two [128 rows][32 floats] blocks of staged output
    static constexpr int SMEM_BYTES = 1024 + Q_BUF + 4 * KV_BYTES /*K, V: two stages each*/ + 256 +
                                      6 * kPfTile * 4 /*row maxima, row sums*/;
    static constexpr int OC = D / 2;              // output columns per softmax thread
    static constexpr int ROUNDS = OC / 32;        // staging rounds of 32 columns per thread
};
constexpr uint32_t kTmemCols = 256;          // two score buffers: columns [0,64), [64,128); O tile: [128,128+D)

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
// B K-major (b_mn = 0) or MN-major (b_mn = 1), M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int b_mn, uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
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

// Multiply 8 fp32 columns of this thread's TMEM lane by alpha in place.
__device__ __forceinline__ void tmem_scale8(uint32_t taddr, float alpha) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

// 8 packed 32-bit columns (16 bf16 values) of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&v)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(v[0]),
                 "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct PrefillArgs {
    int* status;
    int* sched;      // work counter, zero when the kernel starts
    int n;           // rows cached in the slot (after this pass's append)
    int T;           // queries per head
    int Hq, G, B;
    int group_heads; // q-heads per scheduling group (a multiple of G)
    int row_stride;
    long long krow0, vrow0;  // first row of the slot's K / V plane in the pool-wide row numbering
    long long plane_rows;    // rows of one plane (what a bounds-checking build checks tile rows against)
    float scale_log2;
};

// A work item = 128 queries of one (sequence, q-head).  The q-heads (numbered sequence-major, so
// the heads of one kv-head are adjacent) are taken in groups of `group_heads`; inside a group the
// items run from the query blocks with the most keys down, all heads of the group per block.
// The group is sized on the host so that the K/V rows its heads stream fit in L2 together, while
// the blocks running at one moment still spread over as many kv-heads as that allows.
struct PrefillItem {
    int q0, hq, b, nt;
};
__device__ __forceinline__ PrefillItem decode_item(int w, const PrefillArgs& a) {
    const int nqb = (a.T + kPfTile - 1) / kPfTile;
    const int nheads = a.Hq * a.B;
    const int ipg = nqb * a.group_heads;                       // items of a full group
    const int g = min(w / ipg, (nheads - 1) / a.group_heads);
    const int r = w - g * ipg;
    const int gh = min(a.group_heads, nheads - g * a.group_heads);   // the last group may be smaller
    const int qb = nqb - 1 - r / gh;
    const int head = g * a.group_heads + r % gh;
    PrefillItem it;
    it.q0 = qb * kPfTile;
    it.hq = head % a.Hq;
    it.b = head / a.Hq;
    // last key any query of the block may see, and the key tiles that cover keys 0..that
    const int last_key = min(a.n - a.T + it.q0 + kPfTile - 1, a.n - 1);
    it.nt = last_key / kPfKeys + 1;
    return it;
}

// TMA store of one [128 rows][32 floats] block (128-byte swizzle) of the output tile.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tmap, const void* src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(
                     reinterpret_cast<uint64_t>(tmap)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(src))
                 : "memory");
}

// max(a, b, c) in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// One softmax pass over 16 scores x[OFF .. OFF+15]: p = 2^(x*scale - m_ref) (0 where masked),
// split into bf16 hi and lo words (2 keys per word).  Returns the sum of p.  The scale, the
// sum and the hi/lo split use the packed two-float instructions.
template <bool MASK, int OFF>
__device__ __forceinline__ float softmax_chunk(const float (&x)[32], float scale_log2, float m_ref, int key_first,
                                               int limit, uint32_t (&hi)[8], uint32_t (&lo)[8]) {
    const float2 sc = make_float2(scale_log2, scale_log2), nm = make_float2(-m_ref, -m_ref);
    const float2 minus1 = make_float2(-1.f, -1.f);
    float2 sum = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const float2 t = __ffma2_rn(make_float2(x[OFF + i], x[OFF + i + 1]), sc, nm);
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

template <int D>
__global__ void __launch_bounds__(kPfThreads, 2)
    prefill_attention_tc(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
                         const __grid_constant__ CUtensorMap tmap_out, const PrefillArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* sQ = smem;                       // Q tile; after an item's last MMA, staging for its output
    using S = PfShape<D>;
    constexpr int kKvBytes = S::KV_BYTES;
    unsigned char* sK = sQ + S::Q_BUF;              // two stages
    unsigned char* sV = sK + 2 * kKvBytes;          // two stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + 2 * kKvBytes);
    uint64_t* q_full = bars;
    uint64_t* q_free = bars + 1;        // the output staged in the Q buffer has been read by the TMA store
    // o_full[tile & 1]: one phase per PV group of a tile of that parity (the tile's contribution is in O).
    // Two barriers, because the PV groups of two consecutive tiles can be outstanding at once and a
    // parity wait cannot tell a phase from the one two before it.
    uint64_t* o_full = bars + 28;
    uint64_t* epi_bar = bars + 3;       // all softmax threads, used around the output staging
    uint64_t* k_full = bars + 4;        // [2] per K stage
    uint64_t* k_empty = bars + 6;
    uint64_t* v_full = bars + 8;        // [2] per V stage
    uint64_t* v_empty = bars + 10;
    uint64_t* s_full = bars + 12;       // [2] per score buffer
    uint64_t* p_full = bars + 14;       // [2] per score buffer, one arrival per softmax thread
    uint64_t* pair_bar = bars + 16;     // [4]: the two warps that share 32 query rows, 64 arrivals
    uint64_t* item_full = bars + 20;    // [2] work-item ring: written by the producer lane
    uint64_t* item_empty = bars + 22;   // [2] released by the MMA lane and every softmax thread
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 25);
    volatile int* ring = reinterpret_cast<volatile int*>(bars + 26);   // [2] item numbers, -1 = no more work
    float* exch_m = reinterpret_cast<float*>(bars + 32);   // [2 tile parities][2 key halves][128] row maxima
    float* exch_l = exch_m + 4 * kPfTile;                  // [2 key halves][128] row sums

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = a.Hq / a.G;
    const int total_items = ((a.T + kPfTile - 1) / kPfTile) * a.Hq * a.B;
    constexpr int kSoftmaxThreads = kPfSoftmaxWarps * 32;

    if (tid == 0) {
        for (int i = 0; i < 24; ++i) mbar_init(&bars[i], 1);
        mbar_init(&o_full[0], 1);
        mbar_init(&o_full[1], 1);
        mbar_init(epi_bar, kSoftmaxThreads);
        mbar_init(&p_full[0], kSoftmaxThreads);
        mbar_init(&p_full[1], kSoftmaxThreads);
        for (int i = 0; i < 4; ++i) mbar_init(&pair_bar[i], 64);
        mbar_init(&item_empty[0], kSoftmaxThreads + 1);
        mbar_init(&item_empty[1], kSoftmaxThreads + 1);
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
    const uint32_t tmem_s = tmem_base;         // two score buffers of 64 fp32 columns; P_hi / P_lo overwrite them
    const uint32_t tmem_o = tmem_base + 128;   // running output rows

    // Every role walks the same sequence of work items (numbers handed out by the producer lane
    // through a two-entry ring) and keeps its own count `t` of key tiles done in earlier items:
    // stage = t & 1, and a stage's barrier is in phase (t >> 1) & 1.
    if (warp == kPfSoftmaxWarps) {
        // ------------------------------ scheduler + TMA producer ------------------------------
        if (lane == 0) {
            int t = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int slot = it & 1;
                if (it >= 2) ok = mbar_wait_bounded(&item_empty[slot], (uint32_t)((it >> 1) - 1) & 1u, abort_flag, a.status);
                if (!ok) break;
                int w = atomicAdd(a.sched, 1);
                if (w >= total_items) w = -1;
                ring[slot] = w;
                mbar_arrive(&item_full[slot]);
                if (w < 0) break;
                const PrefillItem item = decode_item(w, a);
                const long long unit_row = ((long long)item.b * Hkv + item.hq / a.G) * a.row_stride;
                auto load_q = [&]() {
                    // the Q buffer doubles as the previous item's output staging
                    if (it >= 1 && !mbar_wait_bounded(q_free, (uint32_t)(it - 1) & 1u, abort_flag, a.status)) return false;
                    mbar_arrive_expect_tx(q_full, S::Q_BYTES);
#pragma unroll
                    for (int h = 0; h < S::HALVES; ++h)
                        tma_load_4d(sQ + h * kPfQBlock, &tmap_q, h * 64, item.hq, item.q0, item.b, q_full);
                    return true;
                };
                for (int j = 0; j < item.nt && ok; ++j) {
                    // the first two K/V tiles do not depend on the previous item's output being
                    // gone from the Q buffer, so they are fetched before Q
                    if (j == 2) ok = load_q();
                    if (!ok) break;
                    const int tt = t + j, st = tt & 1;
                    const uint32_t prev = (uint32_t)((tt >> 1) - 1) & 1u;   // phase in which tile tt-2 released the stage
                    long long row = unit_row + (long long)j * kPfKeys;
                    if (!KVS_BOUNDS_OK(row, kPfKeys, a.plane_rows, a.status)) row = 0;
                    if (tt >= 2 && !mbar_wait_bounded(&k_empty[st], prev, abort_flag, a.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(&k_full[st], kKvBytes);
#pragma unroll
                    for (int h = 0; h < S::HALVES; ++h)
                        tma_load_2d_pf(sK + st * kKvBytes + h * kPfKvBlock, &tmap_kv, h * 64, (int)(a.krow0 + row),
                                       &k_full[st]);
                    if (tt >= 2 && !mbar_wait_bounded(&v_empty[st], prev, abort_flag, a.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(&v_full[st], kKvBytes);
#pragma unroll
                    for (int h = 0; h < S::HALVES; ++h)
                        tma_load_2d_pf(sV + st * kKvBytes + h * kPfKvBlock, &tmap_kv, h * 64, (int)(a.vrow0 + row),
                                       &v_full[st]);
                }
                if (ok && item.nt <= 2) ok = load_q();
                t += item.nt;
            }
        }
    } else if (warp == kPfSoftmaxWarps + 1) {
        // ------------------------------ MMA issuer ------------------------------
        // Order on the tensor pipe: S_0, then per tile j: S_{j+1} (into the other score buffer, so
        // that the softmax of tile j+1 can start the moment the one of tile j ends), PV_j.  The
        // pipe runs one thread's MMAs in issue order, so S_{j+1} overwrites its buffer only after
        // PV_{j-1} has read P_{j-1} from it.  PV_0 of an item starts a fresh output tile; the
        // softmax threads arrive for it only after they have read the previous item's output.
        if (lane == 0) {
            const uint32_t idesc_s = instr_desc_bf16(0, kPfKeys);
            const uint32_t idesc_o = instr_desc_bf16(1, D);
            const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
            auto issue_s = [&](int tt) {
                const int st = tt & 1;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {   // 16 head-dim columns per step; 4 steps per 64-column block
                    const uint32_t qoff = (ks >> 2) * kPfQBlock + (ks & 3) * 32;
                    const uint32_t koff = st * kKvBytes + (ks >> 2) * kPfKvBlock + (ks & 3) * 32;
                    umma_bf16(tmem_s + st * kPfKeys, smem_desc_sw128(q_addr + qoff, 16, 1024),
                              smem_desc_sw128(k_addr + koff, 16, 1024), idesc_s, ks > 0);
                }
                umma_commit(&s_full[st]);
                umma_commit(&k_empty[st]);     // the K stage may be overwritten once S is done
            };
            int t = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int slot = it & 1;
                ok = mbar_wait_bounded(&item_full[slot], (uint32_t)(it >> 1) & 1u, abort_flag, a.status);
                if (!ok) break;
                const int w = ring[slot];
                if (w < 0) break;
                const int nt = decode_item(w, a).nt;
                ok = mbar_wait_bounded(q_full, (uint32_t)it & 1u, abort_flag, a.status) &&
                     mbar_wait_bounded(&k_full[t & 1], (uint32_t)(t >> 1) & 1u, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                issue_s(t);
                for (int j = 0; j < nt; ++j) {
                    const int tt = t + j, st = tt & 1;
                    const uint32_t ph = (uint32_t)(tt >> 1) & 1u;
                    if (j + 1 < nt) {
                        ok = mbar_wait_bounded(&k_full[st ^ 1], (uint32_t)((tt + 1) >> 1) & 1u, abort_flag, a.status);
                        if (!ok) break;
                        tc_fence_after();
                        issue_s(tt + 1);
                    }
                    ok = mbar_wait_bounded(&p_full[st], ph, abort_flag, a.status) &&
                         mbar_wait_bounded(&v_full[st], ph, abort_flag, a.status);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kPfKeys / 16; ++ks) {   // 16 keys per step: 8 TMEM columns of bf16 pairs
                        // V is MN-major: 64 head-dim columns contiguous per key row, the other 64 (D = 128)
                        // one column block (LBO) away; 8-key groups 1024 bytes (SBO) apart
                        const uint64_t vdesc = smem_desc_sw128(v_addr + st * kKvBytes + ks * 16 * 128, kPfKvBlock, 1024);
                        umma_bf16_ts(tmem_o, tmem_s + st * kPfKeys + ks * 8, vdesc, idesc_o, (j > 0) || (ks > 0));   // P_hi
                        umma_bf16_ts(tmem_o, tmem_s + st * kPfKeys + kPfKeys / 2 + ks * 8, vdesc, idesc_o, 1);     // P_lo
                    }
                    umma_commit(&o_full[st]);
                    umma_commit(&v_empty[st]);
                }
                if (!ok) break;
                mbar_arrive(&item_empty[slot]);
                t += nt;
            }
        }
    } else {
        // ------------------------------ softmax / output rows ------------------------------
        const int w4 = warp & 3, hf = warp >> 2;             // TMEM lane quarter, key half of a tile
        const int r = w4 * 32 + lane;                        // query row in the block = TMEM lane
        const uint32_t lane_addr = (uint32_t)(w4 * 32) << 16;
        const uint32_t to = tmem_o + lane_addr + hf * S::OC;     // this thread's D/2 columns of the output row
        // output staging: [128 rows][32 floats] blocks, 128-byte swizzle; this thread's row of the
        // block its key half owns
        unsigned char* stage_row = sQ + hf * kPfQBlock + r * 128;
        int t = 0;
        uint32_t pp = 0, ep = 0;                             // phases used so far of pair_bar[w4] and epi_bar
        bool ok = true;
        for (int it = 0; ok; ++it) {
            const int slot = it & 1;
            ok = mbar_wait_bounded(&item_full[slot], (uint32_t)(it >> 1) & 1u, abort_flag, a.status);
            if (!ok) break;
            const int w = ring[slot];
            if (w < 0) break;
            const PrefillItem item = decode_item(w, a);
            const int nt = item.nt;
            const int qpos = min(item.q0 + r, a.T - 1);          // padding rows repeat the last query
            const int limit = a.n - a.T + qpos;                  // last key this query may see
            const int block_min_limit = a.n - a.T + item.q0;     // smallest limit of any row of the block
            float m_ref = -1.0e30f, l = 0.f;                     // p is taken relative to m_ref (log2 domain)
            for (int j = 0; j < nt; ++j) {
                const int tt = t + j, st = tt & 1;
                ok = mbar_wait_bounded(&s_full[st], (uint32_t)(tt >> 1) & 1u, abort_flag, a.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sb = tmem_s + lane_addr + st * kPfKeys;
                const uint32_t ts = sb + hf * 32;                     // this thread's 32 scores
                const uint32_t tph = sb + hf * 16;                    // P_hi words of its keys (key k -> column k/2)
                const uint32_t tpl = sb + kPfKeys / 2 + hf * 16;      // P_lo words (column 32 + k/2)
                const int key0 = j * kPfKeys + hf * 32;
                const bool mask = j * kPfKeys + kPfKeys - 1 > block_min_limit;   // block-uniform
                float x[32];
                tmem_ld32(ts, x);
                // row maximum of the (masked) scores: own half, then the partner warp's through shared
                // memory.  After the pair barrier both halves of S have been read, so P may overwrite it.
                float mx = -INFINITY;
                if (mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, (key0 + i <= limit) ? x[i] : -INFINITY);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) mx = fmax3(mx, x[i], x[i + 1]);
                }
                float* em = exch_m + st * 2 * kPfTile;
                em[hf * kPfTile + r] = mx;
                tc_fence_before();
                mbar_arrive(&pair_bar[w4]);
                ok = mbar_wait_bounded(&pair_bar[w4], pp & 1u, abort_flag, a.status);
                ++pp;
                if (!ok) break;
                tc_fence_after();
                mx = fmaxf(mx, em[(hf ^ 1) * kPfTile + r]) * a.scale_log2;
                // The reference maximum only moves when the new one is more than 8 (a factor 256) above
                // it; then the output row and the sum accumulated so far are rescaled, once every PV
                // issued so far has landed in O (PV of this tile cannot start before this thread's
                // arrival below).  Both threads of a row take the same decision from the same numbers.
                const bool grow = mx > m_ref + 8.0f;
                if (__any_sync(0xffffffffu, grow)) {
                    const float m_new = grow ? mx : m_ref;
                    const float alpha = fast_exp2(m_ref - m_new);
                    if (j > 0) {
                        ok = mbar_wait_bounded(&o_full[(tt - 1) & 1], (uint32_t)((tt - 1) >> 1) & 1u, abort_flag, a.status);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll 1
                        for (int c = 0; c < S::OC / 8; ++c) tmem_scale8(to + c * 8, alpha);
                    }
                    l *= alpha;
                    m_ref = m_new;
                }
                float lsum = 0.f;
#define KVS_PF_CHUNK(OFF)                                                                                      \
    {                                                                                                          \
        uint32_t hi[8], lo[8];                                                                                 \
        lsum += mask ? softmax_chunk<true, OFF>(x, a.scale_log2, m_ref, key0 + OFF, limit, hi, lo)             \
                     : softmax_chunk<false, OFF>(x, a.scale_log2, m_ref, key0 + OFF, limit, hi, lo);           \
        tmem_st8(tph + OFF / 2, hi);                                                                           \
        tmem_st8(tpl + OFF / 2, lo);                                                                           \
    }
                KVS_PF_CHUNK(0)
                KVS_PF_CHUNK(16)
#undef KVS_PF_CHUNK
                l += lsum;
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive(&p_full[st]);
            }
            if (!ok) break;
            // the row's sum is the two halves' sums (both relative to the same reference maximum)
            exch_l[hf * kPfTile + r] = l;
            mbar_arrive(&pair_bar[w4]);
            ok = mbar_wait_bounded(&pair_bar[w4], pp & 1u, abort_flag, a.status);
            ++pp;
            if (!ok) break;
            l += exch_l[(hf ^ 1) * kPfTile + r];
            // the last tile's PV group is behind every other MMA of the item on the pipe
            ok = mbar_wait_bounded(&o_full[(t + nt - 1) & 1], (uint32_t)((t + nt - 1) >> 1) & 1u, abort_flag, a.status);
            if (!ok) break;
            tc_fence_after();
            // Output: every MMA of the item is done, so the Q buffer is free.  Each thread scales its
            // D/2 columns and stages them there, 32 columns per round, in the swizzled layout of a TMA
            // store; one thread issues the stores (rows past the last query are clipped by the
            // tensor map) and waits until they have read the buffer.
            const float inv = 1.0f / l;
#pragma unroll 1
            for (int c = 0; c < S::ROUNDS; ++c) {
                float o[32];
                tmem_ld32(to + c * 32, o);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float4*>(stage_row + ((i ^ (r & 7)) << 4)) =
                        make_float4(o[4 * i] * inv, o[4 * i + 1] * inv, o[4 * i + 2] * inv, o[4 * i + 3] * inv);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(epi_bar);
                ok = mbar_wait_bounded(epi_bar, ep & 1u, abort_flag, a.status);
                ++ep;
                if (!ok) break;
                if (tid == 0) {
                    tma_store_4d(&tmap_out, sQ, c * 32, item.hq, item.q0, item.b);
                    tma_store_4d(&tmap_out, sQ + kPfQBlock, S::OC + c * 32, item.hq, item.q0, item.b);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    if (c == S::ROUNDS - 1) mbar_arrive(q_free);
                }
                if (c < S::ROUNDS - 1) {   // the buffer is reused by the next round
                    mbar_arrive(epi_bar);
                    ok = mbar_wait_bounded(epi_bar, ep & 1u, abort_flag, a.status);
                    ++ep;
                    if (!ok) break;
                }
            }
            if (!ok) break;
            tc_fence_before();
            mbar_arrive(&item_empty[slot]);
            t += nt;
        }
        if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the stores have reached memory
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
    cudaError_t e = cudaFuncSetAttribute(prefill_attention_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PfShape<128>::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(prefill_attention_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                PfShape<64>::SMEM_BYTES);
}

// q: [B][T][Hq][D] bf16, D = 64 or 128.  Persistent blocks (two per SM) take (128 queries, q-head,
// sequence) items from a counter, heaviest first.  `sched` is a device int the launch zeroes on `stream`.
cudaError_t launch_prefill(const void* q, float* out, int* status, int* sched, const void* pool_tensor_map, int B, int T,
                           int Hq, int G, int D, int n, int row_stride, long long krow0, long long vrow0,
                           long long plane_rows, float scale_log2, int sm_count, long long l2_bytes, cudaStream_t stream) {
    if (D != 64 && D != 128) return cudaErrorInvalidValue;
    EncodeFn encode = nullptr;
    cudaError_t e = get_encode(&encode);
    if (e != cudaSuccess) return e;
    alignas(64) CUtensorMap tq, to;
    const cuuint64_t d = (cuuint64_t)D;
    cuuint64_t dims[4] = {d, (cuuint64_t)Hq, (cuuint64_t)T, (cuuint64_t)B};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    {
        cuuint64_t strides[3] = {d * 2, (cuuint64_t)Hq * d * 2, (cuuint64_t)T * Hq * d * 2};
        cuuint32_t box[4] = {64, 1, (cuuint32_t)kPfTile, 1};
        if (encode(&tq, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t strides[3] = {d * 4, (cuuint64_t)Hq * d * 4, (cuuint64_t)T * Hq * d * 4};
        cuuint32_t box[4] = {32, 1, (cuuint32_t)kPfTile, 1};
        if (encode(&to, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
            CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    PrefillArgs a;
    a.status = status;
    a.sched = sched;
    a.n = n;
    a.T = T;
    a.Hq = Hq;
    a.G = G;
    a.B = B;
    a.row_stride = row_stride;
    a.krow0 = krow0;
    a.vrow0 = vrow0;
    a.plane_rows = plane_rows;
    a.scale_log2 = scale_log2;
    {
        // kv-heads whose K/V rows (n rows of 2 D bytes, K and V) fit in three quarters of L2
        // together; groups of equal size
        const long long streams = (long long)B * (Hq / G);
        const long long stream_bytes = 2LL * n * D * 2;
        const long long fit = std::max<long long>(1, (l2_bytes / 4 * 3) / stream_bytes);
        const long long groups = (streams + fit - 1) / fit;
        a.group_heads = (int)((streams + groups - 1) / groups) * G;
    }
    if ((e = cudaMemsetAsync(sched, 0, sizeof(int), stream)) != cudaSuccess) return e;
    const long long items = (long long)((T + kPfTile - 1) / kPfTile) * Hq * B;
    const int blocks = (int)std::min<long long>(items, 2LL * sm_count);
    const CUtensorMap& tkv = *reinterpret_cast<const CUtensorMap*>(pool_tensor_map);
    if (D == 128)
        prefill_attention_tc<128><<<blocks, kPfThreads, PfShape<128>::SMEM_BYTES, stream>>>(tq, tkv, to, a);
    else
        prefill_attention_tc<64><<<blocks, kPfThreads, PfShape<64>::SMEM_BYTES, stream>>>(tq, tkv, to, a);
    return cudaGetLastError();
}

}  // namespace kvs
