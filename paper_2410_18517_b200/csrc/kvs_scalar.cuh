// Arithmetic of the scalar (fp32 FMA) decode-attention kernels, shared by the persistent split-K
// kernel and the cluster kernel: a token row of RB = D*sizeof(T) bytes is read by LPR = RB/16
// lanes, 16 bytes each; a lane group owns rows grp, grp + NG, ... of a tile and keeps its own
// online-softmax state (running max in the log2 domain, sum, un-normalised output chunk).
#pragma once
#include "kvs_device.cuh"

namespace kvs {

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

// T = storage type, D = head size, G = q-heads per kv-head, NG = lane groups per block,
// TN = rows per tile.
template <typename T, int D, int G, int NG, int TN>
struct ScalarMath {
    static constexpr int RB = D * (int)sizeof(T);
    static constexpr int LPR = RB / 16;
    static constexpr int EPL = 16 / (int)sizeof(T);
    static constexpr int R = TN / NG;                                    // rows per group per tile
    static constexpr int SH = Log2<LPR>::value - Log2<R>::value;         // lane-in-group >> SH = row held after the reduction
    static_assert(R >= 1 && R <= LPR && (R & (R - 1)) == 0, "rows per group must be a power of two <= lanes per row");
    static_assert(TN % NG == 0, "tile rows must divide evenly among lane groups");

    struct State {
        float qf[G][EPL];
        float m[G], lsum[G], acc[G][EPL];
    };

    static __device__ __forceinline__ void reset(State& s) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            s.m[g] = -1.0e30f;
            s.lsum[g] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) s.acc[g][e] = 0.f;
        }
    }

    // q rows of the unit (G x RB bytes at qs), pre-multiplied by scale * log2(e)
    static __device__ __forceinline__ void load_q(State& s, const unsigned char* qs, int lig, float scale_log2) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 raw = *reinterpret_cast<const uint4*>(qs + g * RB + lig * 16);
            Unpack<T>::run(raw, s.qf[g]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) s.qf[g][e] *= scale_log2;
        }
    }

    // One tile of `valid` (1..TN) rows: K at ks, V at vs.  lig = lane within its row group,
    // grp = row group within the block.
    static __device__ __forceinline__ void tile(State& st, const unsigned char* ks, const unsigned char* vs, int valid,
                                                int lig, int grp) {
        const int my_i = lig >> SH;   // row (of the R) whose score this lane ends up holding
        // scores: partial dot products of this lane's 16-byte chunk
        float s[G][R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = grp + NG * i;
            const uint4 raw = *reinterpret_cast<const uint4*>(ks + row * RB + lig * 16);
            float kf[EPL];
            Unpack<T>::run(raw, kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) d = fmaf(st.qf[g][e], kf[e], d);
                s[g][i] = d;
            }
        }
        // online softmax per q-head, local to the lane group
        float p[G][R];
        const bool mine_valid = (grp + NG * my_i) < valid;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float sv = reduce_transpose<R, LPR / 2>(s[g], lig);
            sv = mine_valid ? sv : -INFINITY;
            float tmax = sv;
#pragma unroll
            for (int o = LPR / 2; o >= LPR / R; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            const float m_new = fmaxf(st.m[g], tmax);
            const float alpha = fast_exp2(st.m[g] - m_new);
            const float pv = fast_exp2(sv - m_new);
            st.m[g] = m_new;
            st.lsum[g] = st.lsum[g] * alpha + pv;
#pragma unroll
            for (int e = 0; e < EPL; ++e) st.acc[g][e] *= alpha;
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
                for (int g = 0; g < G; ++g)
#pragma unroll
                    for (int e = 0; e < EPL; ++e) st.acc[g][e] = fmaf(p[g][i], vf[e], st.acc[g][e]);
            }
        }
    }

    // End of a piece: merge the NG lane groups of the block, one q-head at a time, through
    // `scratch` (NG x (D + 2) floats); store(g, d, o, M, den) is called by thread d < D with the
    // merged un-normalised output element, and M (max, log2 domain) and den (sum) of the piece.
    // All NT consumer threads call this (named barrier 1).
    template <int NT, typename Store>
    static __device__ __forceinline__ void merge(State& st, float* scratch, int tid, int lig, int grp, Store store) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            // lanes with equal top bits hold duplicates of lsum; add across the R distinct ones
            float l = st.lsum[g];
#pragma unroll
            for (int o = LPR / 2; o >= LPR / R; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            named_bar_sync(1, NT);  // scratch free again
            float* row = scratch + grp * (D + 2);
#pragma unroll
            for (int e = 0; e < EPL; ++e) row[lig * EPL + e] = st.acc[g][e];
            if (lig == 0) {
                row[D] = st.m[g];
                row[D + 1] = l;
            }
            named_bar_sync(1, NT);
            for (int d = tid; d < D; d += NT) {
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
                store(g, d, o, M, den);
            }
        }
    }
};

}  // namespace kvs
