// Tensor-core inner loop of the split-K decode attention (head_dim 64 or 128).
//
// For one KV head the G query heads that share it form the rows of a 16-row MMA tile (rows >= G are zero), so
//   S^T[head, pos] = Q[head, :] . K[pos, :]      is  mma.m16n8k16 with A = Q (bf16 hi + lo halves), B = K rows
//   O[head, :]    += P[head, pos] * V[pos, :]    is  mma.m16n8k16 with A = P (bf16),               B = V rows
// and the accumulator layout of S^T is already the A-operand layout of P, so the probabilities never leave the
// registers.  K and V rows arrive in the ring as 128-byte-swizzled TMA boxes ([positions] x [64 columns]); the
// swizzle makes the 8 x 16 B row fragments of ldmatrix fall into distinct banks although consecutive positions
// are a multiple of 128 bytes apart.  Compared with the CUDA-core loop this removes the per-position butterfly
// shuffles and the 16-fold replicated softmax arithmetic.
//
// Precision: q and the probabilities are each split into two bf16 numbers (x = hi + lo to ~2^-17), K and V are
// bf16 values by definition, all accumulation is fp32: the result matches an fp32 CUDA-core loop to ~1e-5.
#pragma once

// Included by kl_device.cuh once its PTX helpers, ex2() and rescale() are defined.
namespace kl {

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D += A * B for one m16n8k16 tile; rows 8..15 of A are zero (a1 = a3 = 0).
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    const uint32_t z = 0u;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}

// Byte offset of the 16-byte piece `c16` (0..7) of row `r` inside a swizzled box set: boxes of `box_bytes`
// (rows x 128 B) follow each other, one per 64 columns.
__device__ __forceinline__ uint32_t swz_off(uint32_t box_bytes, uint32_t r, uint32_t cc) {
    return (cc >> 3) * box_bytes + r * 128u + (((cc & 7u) ^ (r & 7u)) << 4);
}

template <int HD>
struct AttnTcState {
    static constexpr int NKB = HD / 16;  // k blocks of the score product
    static constexpr int NNT = HD / 8;   // n tiles of the value product
    uint32_t qh[NKB][2], ql[NKB][2];     // A fragments of Q (rows 0..7 only), hi and lo bf16 halves
    float o[NNT][4];                     // O accumulators ([.][2], [.][3] belong to the zero rows)
    float m, l;                          // running maximum (base-2 scores) and this lane's part of the row sum
};

// One tile of 16 positions starting at row `row0` of the box set at (kbase, vbase); rows j with lo <= j < hi hold
// valid positions, every other row is ignored whatever it contains.
template <int HD>
__device__ __forceinline__ void attn_tc_tile(AttnTcState<HD>& st, uint32_t kbase, uint32_t vbase, uint32_t box_bytes,
                                             uint32_t row0, uint32_t lo, uint32_t hi, uint32_t lane) {
    constexpr int NKB = HD / 16, NNT = HD / 8;
    const uint32_t t = lane & 3u, mi = lane >> 3, mr = lane & 7u;
    float sA[4] = {0.f, 0.f, 0.f, 0.f}, sB[4] = {0.f, 0.f, 0.f, 0.f};
    {
        const uint32_t r = row0 + (mi >> 1) * 8u + mr;
#pragma unroll
        for (int kb = 0; kb < NKB; ++kb) {
            uint32_t b[4];
            ldmatrix_x4(b, kbase + swz_off(box_bytes, r, 2u * kb + (mi & 1u)));
            mma_16816(sA, st.qh[kb][0], st.qh[kb][1], b[0], b[1]);
            mma_16816(sA, st.ql[kb][0], st.ql[kb][1], b[0], b[1]);
            mma_16816(sB, st.qh[kb][0], st.qh[kb][1], b[2], b[3]);
            mma_16816(sB, st.ql[kb][0], st.ql[kb][1], b[2], b[3]);
        }
    }
    // this lane holds, for head (lane >> 2), the scores of positions row0 + {2t, 2t+1, 8+2t, 9+2t}
    const uint32_t j0 = row0 + 2u * t;
    const bool v0 = j0 >= lo && j0 < hi, v1 = j0 + 1 >= lo && j0 + 1 < hi;
    const bool v2 = j0 + 8 >= lo && j0 + 8 < hi, v3 = j0 + 9 >= lo && j0 + 9 < hi;
    float mx = fmaxf(fmaxf(v0 ? sA[0] : -INFINITY, v1 ? sA[1] : -INFINITY),
                     fmaxf(v2 ? sB[0] : -INFINITY, v3 ? sB[1] : -INFINITY));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float mn = fmaxf(st.m, mx);
    const float c = rescale(st.m, mn);
    const float p0 = v0 ? ex2(sA[0] - mn) : 0.f, p1 = v1 ? ex2(sA[1] - mn) : 0.f;
    const float p2 = v2 ? ex2(sB[0] - mn) : 0.f, p3 = v3 ? ex2(sB[1] - mn) : 0.f;
    st.l = st.l * c + ((p0 + p1) + (p2 + p3));
    st.m = mn;
#pragma unroll
    for (int n = 0; n < NNT; ++n) {
        st.o[n][0] *= c;
        st.o[n][1] *= c;
    }
    // probabilities as bf16 hi + lo halves (like q), so the value product keeps fp32-level accuracy
    const uint32_t pa0 = pack_bf16(p0, p1), pa2 = pack_bf16(p2, p3);
    const uint32_t pl0 = pack_bf16(p0 - bf_lo(pa0), p1 - bf_hi(pa0)), pl2 = pack_bf16(p2 - bf_lo(pa2), p3 - bf_hi(pa2));
    // V rows of ignored positions may hold anything (even NaN payloads): clear them, 0 * NaN would poison O
    const bool partial = (lo > row0) || (hi < row0 + 16u);
    const uint32_t mlo = (v0 ? 0x0000ffffu : 0u) | (v1 ? 0xffff0000u : 0u);
    const uint32_t mhi = (v2 ? 0x0000ffffu : 0u) | (v3 ? 0xffff0000u : 0u);
    {
        const uint32_t r = row0 + (mi & 1u) * 8u + mr;
#pragma unroll
        for (int db = 0; db < NNT / 2; ++db) {
            uint32_t v[4];
            ldmatrix_x4_trans(v, vbase + swz_off(box_bytes, r, 2u * db + (mi >> 1)));
            if (partial) {
                v[0] &= mlo;
                v[1] &= mhi;
                v[2] &= mlo;
                v[3] &= mhi;
            }
            mma_16816(st.o[2 * db], pa0, pa2, v[0], v[1]);
            mma_16816(st.o[2 * db], pl0, pl2, v[0], v[1]);
            mma_16816(st.o[2 * db + 1], pa0, pa2, v[2], v[3]);
            mma_16816(st.o[2 * db + 1], pl0, pl2, v[2], v[3]);
        }
    }
}

}  // namespace kl
