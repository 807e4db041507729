// Tensor-core inner loop of the split-K decode attention (head_dim 64 or 128).
//
// For one KV head and a tile of 16 cached positions:
//   S[pos, head]   = K[pos, :] . Q[head, :]       mma.m16n8k16, A = K rows (ldmatrix), B = Q (bf16 hi + lo halves)
//   O^T[d, head]  += V^T[d, pos] * P[pos, head]   mma.m16n8k16, A = V rows (ldmatrix.trans), B = P (bf16 hi + lo)
// The 16 rows of every MMA are real data (positions, value columns); the G <= 8 query heads that share the KV head
// are the 8 columns.  P leaves the S accumulators as packed bf16 pairs and reaches the B-operand layout with one
// movmatrix transpose per 8 x 8 block, so the probabilities never touch shared memory.  K and V rows arrive in the
// ring as 128-byte-swizzled TMA boxes ([positions] x [64 columns]); the swizzle makes the 8 x 16 B row fragments of
// ldmatrix fall into distinct banks although consecutive positions are a multiple of 128 bytes apart.
//
// Precision: q and the probabilities are each split into two bf16 numbers (x = hi + lo to ~2^-17), K and V are
// bf16 values by definition, all accumulation is fp32: the result matches an fp32 CUDA-core loop to ~1e-5.
//
// PACK (G <= 4): the eight columns of an MMA hold the hi halves of the (up to four) heads in columns 0..3 and their lo
// halves in columns 4..7, so one MMA does the work of two.  The two partial scores of a head then sit in lanes
// t and t ^ 2 of a quad and are added with one shuffle; the hi and lo parts of O^T are accumulated in separate
// columns and added once, when the unit's chunks are done.  (mma.sync is slow on this part -- about 70 cycles per
// instruction from a single warp -- so the instruction count is what the loop costs.)
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
// D += A * B for one m16n8k16 tile.
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Transposes an 8 x 8 matrix of 16-bit elements held one row per lane group (row lane/4, columns 2*(lane%4), +1).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// Byte offset of the 16-byte piece `c16` (0..7) of row `r` inside a swizzled box set: boxes of `box_bytes`
// (rows x 128 B) follow each other, one per 64 columns.
__device__ __forceinline__ uint32_t swz_off(uint32_t box_bytes, uint32_t r, uint32_t cc) {
    return (cc >> 3) * box_bytes + r * 128u + (((cc & 7u) ^ (r & 7u)) << 4);
}

template <int HD>
struct AttnTcState {
    static constexpr int NKB = HD / 16;  // k blocks of the score product
    static constexpr int NMT = HD / 16;  // m tiles (16 value columns each) of the value product
    uint32_t qh[NKB][2], ql[NKB][2];     // B fragments of Q for head lane/4 (zero beyond G), hi and lo bf16 halves
                                         // (PACK: qh holds column lane/4 of the packed operand, ql is unused)
    float o[NMT][4];                     // O^T accumulators: value columns mt*16 + lane/4 (+8), heads 2*(lane%4), +1
                                         // (PACK: columns 2*(lane%4), +1 of the packed result)
    float m[2], l[2];                    // running maximum (base-2 scores) and this lane's part of the row sums, for
                                         // heads 2*(lane%4) and 2*(lane%4)+1 (PACK: heads 2*(lane%2), +1)
};

// One tile of 16 positions starting at row `row0` of the box set at (kbase, vbase); rows j with lo <= j < hi hold
// valid positions, every other row is ignored whatever it contains.
template <int HD, bool PACK>
__device__ __forceinline__ void attn_tc_tile(AttnTcState<HD>& st, uint32_t kbase, uint32_t vbase, uint32_t box_bytes,
                                             uint32_t row0, uint32_t lo, uint32_t hi, uint32_t lane) {
    constexpr int NKB = HD / 16, NMT = HD / 16;
    const uint32_t g = lane >> 2, mi = lane >> 3, mr = lane & 7u;
    // scores: two accumulators (even / odd k blocks) halve the dependent MMA chain
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
    {
        const uint32_t r = row0 + (mi & 1u) * 8u + mr;
#pragma unroll
        for (int kb = 0; kb < NKB; ++kb) {
            uint32_t a[4];
            ldmatrix_x4(a, kbase + swz_off(box_bytes, r, 2u * kb + (mi >> 1)));
            if (kb & 1) {
                mma_16816(s1, a, st.qh[kb][0], st.qh[kb][1]);
                if (!PACK) mma_16816(s1, a, st.ql[kb][0], st.ql[kb][1]);
            } else {
                mma_16816(s0, a, st.qh[kb][0], st.qh[kb][1]);
                if (!PACK) mma_16816(s0, a, st.ql[kb][0], st.ql[kb][1]);
            }
        }
    }
    // this lane holds the scores of positions row0 + g and row0 + g + 8 for heads 2t and 2t + 1
    const uint32_t j0 = row0 + g;
    const bool v0 = j0 >= lo && j0 < hi, v1 = j0 + 8 >= lo && j0 + 8 < hi;
    float sa0 = s0[0] + s1[0], sa1 = s0[1] + s1[1], sb0 = s0[2] + s1[2], sb1 = s0[3] + s1[3];
    if (PACK) {   // hi and lo partial scores of a head sit in lanes t and t ^ 2
        sa0 += __shfl_xor_sync(0xffffffffu, sa0, 2);
        sa1 += __shfl_xor_sync(0xffffffffu, sa1, 2);
        sb0 += __shfl_xor_sync(0xffffffffu, sb0, 2);
        sb1 += __shfl_xor_sync(0xffffffffu, sb1, 2);
    }
    float mx0 = fmaxf(v0 ? sa0 : -INFINITY, v1 ? sb0 : -INFINITY);
    float mx1 = fmaxf(v0 ? sa1 : -INFINITY, v1 ? sb1 : -INFINITY);
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    const float mn0 = fmaxf(st.m[0], mx0), mn1 = fmaxf(st.m[1], mx1);
    const float c0 = rescale(st.m[0], mn0), c1 = rescale(st.m[1], mn1);
    const float p00 = v0 ? ex2(sa0 - mn0) : 0.f, p01 = v0 ? ex2(sa1 - mn1) : 0.f;
    const float p10 = v1 ? ex2(sb0 - mn0) : 0.f, p11 = v1 ? ex2(sb1 - mn1) : 0.f;
    st.l[0] = st.l[0] * c0 + (p00 + p10);
    st.l[1] = st.l[1] * c1 + (p01 + p11);
    st.m[0] = mn0;
    st.m[1] = mn1;
#pragma unroll
    for (int n = 0; n < NMT; ++n) {
        st.o[n][0] *= c0;
        st.o[n][1] *= c1;
        st.o[n][2] *= c0;
        st.o[n][3] *= c1;
    }
    // probabilities as bf16 hi + lo halves (like q); the S layout (row = position, columns = two heads) is
    // transposed into the B-operand layout (rows = two positions, column = head)
    const uint32_t ph0 = pack_bf16(p00, p01), ph1 = pack_bf16(p10, p11);
    const uint32_t pl0 = pack_bf16(p00 - bf_lo(ph0), p01 - bf_hi(ph0)), pl1 = pack_bf16(p10 - bf_lo(ph1), p11 - bf_hi(ph1));
    uint32_t bh0, bh1, bl0 = 0u, bl1 = 0u;
    if (PACK) {   // columns 0..3 (lanes t < 2) carry the hi halves, columns 4..7 the lo halves
        const bool lo_cols = (lane & 2u) != 0u;
        bh0 = movmatrix_trans(lo_cols ? pl0 : ph0);
        bh1 = movmatrix_trans(lo_cols ? pl1 : ph1);
    } else {
        bh0 = movmatrix_trans(ph0);
        bh1 = movmatrix_trans(ph1);
        bl0 = movmatrix_trans(pl0);
        bl1 = movmatrix_trans(pl1);
    }
    // V rows of ignored positions may hold anything (even NaN payloads): clear them, 0 * NaN would poison O.
    // The A fragment of V^T holds positions row0 + 2t, +1 (registers 0, 1) and row0 + 8 + 2t, +1 (registers 2, 3).
    const uint32_t t = lane & 3u;
    const uint32_t q0 = row0 + 2u * t;
    const bool partial = (lo > row0) || (hi < row0 + 16u);
    const uint32_t mlo = ((q0 >= lo && q0 < hi) ? 0x0000ffffu : 0u) | ((q0 + 1 >= lo && q0 + 1 < hi) ? 0xffff0000u : 0u);
    const uint32_t mhi = ((q0 + 8 >= lo && q0 + 8 < hi) ? 0x0000ffffu : 0u) | ((q0 + 9 >= lo && q0 + 9 < hi) ? 0xffff0000u : 0u);
    {
        const uint32_t r = row0 + (mi >> 1) * 8u + mr;
#pragma unroll
        for (int mt = 0; mt < NMT; ++mt) {
            uint32_t a[4];
            ldmatrix_x4_trans(a, vbase + swz_off(box_bytes, r, 2u * mt + (mi & 1u)));
            if (partial) {
                a[0] &= mlo;
                a[1] &= mlo;
                a[2] &= mhi;
                a[3] &= mhi;
            }
            mma_16816(st.o[mt], a, bh0, bh1);
            if (!PACK) mma_16816(st.o[mt], a, bl0, bl1);
        }
    }
}

}  // namespace kl
