// Device-side building blocks of the kernel-looped decoder: PTX wrappers (mbarrier, TMA bulk copy,
// acquire/release counters), the shared-memory weight ring, the GEMV stage consumer and the split-K
// attention stage.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kl {

constexpr int NCW = 10;                    // consumer warps per CTA; consumer warp w owns ring slot w
constexpr int NCT = NCW * 32;              // consumer threads
constexpr int NTHREADS = NCT + 32;         // + one producer warp (the last warp)
constexpr int SLOT_BYTES = 16384;          // one ring slot = one TMA bulk copy
constexpr int MAX_SLOTS = NCW;             // one owner warp per slot (see gemv_stage)
constexpr int MAX_PIECES = 8;              // chunks per unit when a unit spans several chunks
constexpr int UNIT_SLOTS = 32;             // in-flight multi-chunk units tracked per CTA
constexpr int MIN_POS_PER_CHUNK = 64;      // attention: fewest cached positions worth a CTA
constexpr int MAX_G = 8;                   // query heads per KV head
constexpr int SMEM_MISC_BYTES = 4096;

enum StageId { ST_QKV = 0, ST_ATTN = 1, ST_O = 2, ST_GU = 3, ST_D = 4, ST_LM = 5 };
enum EpilogueKind { EP_STORE = 0, EP_RESIDUAL = 1, EP_SWIGLU = 2 };
enum PlanId { PL_QKV = 0, PL_O = 1, PL_GU = 2, PL_D = 3, PL_LM = 4, PL_COUNT = 5 };

constexpr int ERR_SYNC_TIMEOUT = -5;
constexpr int ERR_OUT_OF_RANGE = -6;

// How one matrix [R, K] (bf16, row-major, rows contiguous) is cut into ring chunks and units.
//  rpc > 0 : a chunk holds rpc whole rows (the last chunk of the matrix may hold fewer); unit == chunk.
//  rpc == 0: a chunk is one piece (klen elements, the last piece of a row may be shorter) of one row; a unit is
//            rows_per_unit consecutive rows = rows_per_unit * ksplit consecutive chunks.
// Units are dealt to CTAs in contiguous ranges, so each CTA's share of a matrix is one linear byte range.
struct GemvPlan {
    uint32_t R, K;
    uint32_t rpc;
    uint32_t ksplit;
    uint32_t klen;
    uint32_t rows_per_unit;
    uint32_t nunits;
    uint32_t chunks_per_unit;
};

struct Params {
    uint32_t L, H, nq, nkv, hd, F, V, G, QD, KVD, max_ctx, B;
    uint32_t P;            // CTAs in the persistent grid
    uint32_t nslots;       // ring slots
    uint32_t vec_floats;   // capacity of the shared input-vector area
    uint32_t cps;          // attention: CTA slots per (sequence, kv head)
    float eps;
    int32_t skip_stage;    // test hook: stage of layer 0 whose end is not signalled (-1 = none)
    uint64_t wait_ns;
    uint64_t layer_stride; // elements between consecutive layers of any per-layer tensor
    GemvPlan plan[PL_COUNT];
    const __nv_bfloat16 *wqkv, *wo, *wgu, *wd, *g1, *g2, *gf, *wlm, *embed;
    __nv_bfloat16* kv;
    const int32_t* tokens;
    const int32_t* positions;
    float *x, *qkv, *o, *h, *part, *part_ml, *rope_cs, *logits;
    const double* inv_freq;
    uint32_t* counters;    // [L][8]
    uint32_t* tickets;     // [L][B*nkv]
    int32_t* status;
};

// ------------------------------------------------------------------------------------------------ PTX

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// 1-D TMA bulk copy global -> shared, completion counted in bytes on an mbarrier.  Both addresses and the size
// must be multiples of 16 bytes.
__device__ __forceinline__ void tma_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ void red_release_add(uint32_t* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t atom_add_acq_rel(uint32_t* p, uint32_t v) {
    uint32_t old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(NCT) : "memory"); }

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// ------------------------------------------------------------------------------------------------ shared state

struct Smem {
    uint8_t* ring;          // nslots * SLOT_BYTES
    float* vec;             // input vector of the current GEMV stage (lane-permuted), or attention workspace
    uint64_t* full;         // [MAX_SLOTS]
    uint64_t* empty;        // [MAX_SLOTS]
    float* red;             // [NCW]
    float* unit_part;       // [UNIT_SLOTS][MAX_PIECES]
    int* unit_cnt;          // [UNIT_SLOTS]
    volatile int* abort_flag;
    volatile int* bcast;
};

__device__ __forceinline__ Smem carve_smem(uint8_t* base, const Params& p) {
    Smem s;
    s.ring = base;
    s.vec = reinterpret_cast<float*>(base + (size_t)p.nslots * SLOT_BYTES);
    uint8_t* misc = reinterpret_cast<uint8_t*>(s.vec) + (size_t)p.vec_floats * 4;
    s.full = reinterpret_cast<uint64_t*>(misc);
    s.empty = s.full + MAX_SLOTS;
    s.red = reinterpret_cast<float*>(s.empty + MAX_SLOTS);
    s.unit_part = s.red + 32;
    s.unit_cnt = reinterpret_cast<int*>(s.unit_part + UNIT_SLOTS * MAX_PIECES);
    s.abort_flag = s.unit_cnt + UNIT_SLOTS;
    s.bcast = s.abort_flag + 1;
    return s;
}

// Records the first error and tells every waiter of this CTA to give up.  After an abort every wait returns at
// once but the control flow (stage order, CTA barriers) is unchanged, so no warp is left behind at a barrier; the
// step's outputs are then meaningless and the status word says so.
__device__ __forceinline__ void raise_abort(const Params& p, const Smem& s, int code) {
    atomicCAS(p.status, 0, code);
    *s.abort_flag = 1;
}

// Bounded mbarrier wait.  Returns false when the wait was abandoned (limit reached or abort raised elsewhere).
__device__ __forceinline__ bool mbar_wait(const Params& p, const Smem& s, uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*s.abort_flag) return false;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*s.abort_flag) return false;
            if (globaltimer_ns() - t0 > p.wait_ns) {
                raise_abort(p, s, ERR_SYNC_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// ------------------------------------------------------------------------------------------------ chunk geometry

struct CtaRange {
    uint32_t u0, u1;
};
__device__ __forceinline__ CtaRange cta_units(const GemvPlan& pl, uint32_t cta, uint32_t P) {
    CtaRange r;
    r.u0 = (uint32_t)(((uint64_t)cta * pl.nunits) / P);
    r.u1 = (uint32_t)(((uint64_t)(cta + 1) * pl.nunits) / P);
    return r;
}

struct ChunkGeom {
    uint64_t elem_off;  // offset of the chunk inside the matrix, elements
    uint32_t elems;     // elements in the chunk
    uint32_t row;       // first row
    uint32_t nrows;     // whole rows held (rpc > 0) or 1
    uint32_t kofs;      // first column (piece chunks)
    uint32_t piece;     // index of the chunk inside its unit
    uint32_t unit;      // unit index (matrix-wide)
};
__device__ __forceinline__ ChunkGeom chunk_geom(const GemvPlan& pl, uint32_t u0, uint32_t i) {
    ChunkGeom g;
    if (pl.rpc) {
        g.unit = u0 + i;
        g.piece = 0;
        g.row = g.unit * pl.rpc;
        g.nrows = min(pl.rpc, pl.R - g.row);
        g.kofs = 0;
        g.elem_off = (uint64_t)g.row * pl.K;
        g.elems = g.nrows * pl.K;
    } else {
        g.unit = u0 + i / pl.chunks_per_unit;
        g.piece = i % pl.chunks_per_unit;
        const uint32_t rr = g.piece / pl.ksplit, j = g.piece % pl.ksplit;
        g.row = g.unit * pl.rows_per_unit + rr;
        g.nrows = 1;
        g.kofs = j * pl.klen;
        g.elems = min(pl.klen, pl.K - g.kofs);
        g.elem_off = (uint64_t)g.row * pl.K + g.kofs;
    }
    return g;
}

// ------------------------------------------------------------------------------------------------ producer

struct RingPos {
    uint32_t slot, phase;   // phase = (use count of the slot) & 1
    uint64_t issued;
};

// Streams this CTA's share of one matrix into the ring, one bulk copy per chunk.
__device__ __forceinline__ bool produce_matrix(const Params& p, const Smem& s, const GemvPlan& pl,
                                               const __nv_bfloat16* base, uint32_t cta, RingPos& rp, uint64_t pol) {
    const CtaRange r = cta_units(pl, cta, p.P);
    const uint32_t nch = (r.u1 - r.u0) * pl.chunks_per_unit;
    for (uint32_t i = 0; i < nch; ++i) {
        const ChunkGeom g = chunk_geom(pl, r.u0, i);
        if (rp.issued >= p.nslots) {
            // wait until the consumer of the previous use of this slot has released it
            if (!mbar_wait(p, s, smem_u32(&s.empty[rp.slot]), rp.phase ^ 1u)) return false;
        }
        const uint32_t bar = smem_u32(&s.full[rp.slot]);
        const uint32_t bytes = g.elems * 2u;
        mbar_arrive_expect_tx(bar, bytes);
        tma_bulk_g2s(smem_u32(s.ring + (size_t)rp.slot * SLOT_BYTES), base + g.elem_off, bytes, bar, pol);
        ++rp.issued;
        if (++rp.slot == p.nslots) {
            rp.slot = 0;
            rp.phase ^= 1u;
        }
    }
    return true;
}

// After an abandoned run: wait (bounded) for the copies that were issued but never consumed, so that no bulk
// copy is still writing this CTA's shared memory when it exits.
__device__ __forceinline__ void drain_ring(const Params& p, const Smem& s, const RingPos& rp) {
    const uint64_t n = rp.issued < p.nslots ? rp.issued : p.nslots;
    uint32_t slot = rp.slot, phase = rp.phase;
    const uint64_t t0 = globaltimer_ns();
    for (uint64_t k = 0; k < n; ++k) {
        if (slot == 0) {
            slot = p.nslots;
            phase ^= 1u;
        }
        --slot;
        const uint32_t bar = smem_u32(&s.full[slot]);
        while (!mbar_try_wait(bar, phase)) {
            if (globaltimer_ns() - t0 > p.wait_ns) return;
        }
    }
}

// ------------------------------------------------------------------------------------------------ consumers

// Position of element e of the input vector in shared memory.  Within each block of 256 elements the eight
// elements a lane multiplies are split into two float4 groups stored 128 floats apart, so that both float4 loads
// of a warp are bank-conflict free.
__device__ __forceinline__ uint32_t vec_perm(uint32_t e) {
    return (e & ~255u) + (((e >> 2) & 1u) << 7) + (((e >> 3) & 31u) << 2) + (e & 3u);
}

// Loads src[0..n) (fp32, produced by other CTAs: read through L2) into the shared vector area, optionally
// applying RMSNorm with bf16 gains.  Every CTA recomputes the norm; the summation order is fixed.
__device__ __forceinline__ void load_vec(const Params& p, const Smem& s, const float* src, uint32_t n, bool norm,
                                         const __nv_bfloat16* gain, uint32_t ctid) {
    float ss = 0.f;
    for (uint32_t e = ctid * 4; e < n; e += NCT * 4) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(src + e));
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        *reinterpret_cast<float4*>(s.vec + vec_perm(e)) = v;
    }
    if (norm) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((ctid & 31) == 0) s.red[ctid >> 5] = ss;
        consumer_bar();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < NCW; ++w) tot += s.red[w];
        const float inv = rsqrtf(tot / (float)n + p.eps);
        for (uint32_t e = ctid * 4; e < n; e += NCT * 4) {
            float4* q = reinterpret_cast<float4*>(s.vec + vec_perm(e));
            const uint2 gb = *reinterpret_cast<const uint2*>(gain + e);
            float4 v = *q;
            v.x *= inv * bf_lo(gb.x);
            v.y *= inv * bf_hi(gb.x);
            v.z *= inv * bf_lo(gb.y);
            v.w *= inv * bf_hi(gb.y);
            *q = v;
        }
    }
    consumer_bar();
}

// acc[r] += sum over this lane's columns of W[r][k] * vec[k]; W rows in shared memory, row pitch rowbytes.
template <int NR>
__device__ __forceinline__ void dot_rows(const uint8_t* w, uint32_t rowbytes, const float* vec, uint32_t len,
                                         uint32_t lane, float (&acc)[NR]) {
    const float4* v4 = reinterpret_cast<const float4*>(vec);
#pragma unroll 4
    for (uint32_t k = lane * 8; k < len; k += 256) {
        const uint32_t blk = k >> 8;
        const float4 xa = v4[blk * 64 + lane];
        const float4 xb = v4[blk * 64 + 32 + lane];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const uint4 q = *reinterpret_cast<const uint4*>(w + (size_t)r * rowbytes + (size_t)k * 2);
            float a = acc[r];
            a = fmaf(bf_lo(q.x), xa.x, a);
            a = fmaf(bf_hi(q.x), xa.y, a);
            a = fmaf(bf_lo(q.y), xa.z, a);
            a = fmaf(bf_hi(q.y), xa.w, a);
            a = fmaf(bf_lo(q.z), xb.x, a);
            a = fmaf(bf_hi(q.z), xb.y, a);
            a = fmaf(bf_lo(q.w), xb.z, a);
            a = fmaf(bf_hi(q.w), xb.w, a);
            acc[r] = a;
        }
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float silu(float z) { return z / (1.0f + __expf(-z)); }

// Consumes this CTA's share of one matrix from the ring: y = W vec, followed by the stage's epilogue.
//   EP_STORE    out[row] = y
//   EP_RESIDUAL out[row] = out[row] + y            (out is the hidden state, owned row-wise by this CTA)
//   EP_SWIGLU   rows come in (gate, up) pairs: out[row/2] = silu(y_gate) * y_up
// nbase counts the chunks this CTA has consumed so far (identical to the producer's issue order).
// Chunk n lives in slot n % nslots and is consumed by warp n % nslots: every use of a slot is waited on by the
// same warp, in order, so a parity wait can never be satisfied by a phase two uses old.  (With free chunk-to-warp
// assignment a fast warp can test the barrier of use k while use k-1 is still in flight, and parity k&1 then
// reads as complete.)
__device__ __forceinline__ void gemv_stage(const Params& p, const Smem& s, const GemvPlan& pl, int ep, float* out,
                                           uint32_t cta, uint32_t warp, uint32_t lane, uint64_t& nbase) {
    const CtaRange r = cta_units(pl, cta, p.P);
    const uint32_t nch = (r.u1 - r.u0) * pl.chunks_per_unit;
    const uint32_t first = (warp + p.nslots - (uint32_t)(nbase % p.nslots)) % p.nslots;
    for (uint32_t i = (warp < p.nslots ? first : nch); i < nch; i += p.nslots) {
        const uint64_t n = nbase + i;
        const uint32_t slot = warp;
        const uint32_t phase = (uint32_t)((n / p.nslots) & 1u);
        mbar_wait(p, s, smem_u32(&s.full[slot]), phase);
        const uint8_t* sp = s.ring + (size_t)slot * SLOT_BYTES;
        const ChunkGeom g = chunk_geom(pl, r.u0, i);
        if (pl.rpc) {
            const uint32_t rowbytes = pl.K * 2u;
            for (uint32_t rr = 0; rr < g.nrows; rr += 2) {
                float y0, y1 = 0.f;
                if (rr + 1 < g.nrows) {
                    float acc[2] = {0.f, 0.f};
                    dot_rows<2>(sp + (size_t)rr * rowbytes, rowbytes, s.vec, pl.K, lane, acc);
                    y0 = warp_sum(acc[0]);
                    y1 = warp_sum(acc[1]);
                } else {
                    float acc[1] = {0.f};
                    dot_rows<1>(sp + (size_t)rr * rowbytes, rowbytes, s.vec, pl.K, lane, acc);
                    y0 = warp_sum(acc[0]);
                }
                if (lane == 0) {
                    const uint32_t row = g.row + rr;
                    if (ep == EP_STORE) {
                        out[row] = y0;
                        if (rr + 1 < g.nrows) out[row + 1] = y1;
                    } else if (ep == EP_RESIDUAL) {
                        out[row] = __ldcg(out + row) + y0;
                        if (rr + 1 < g.nrows) out[row + 1] = __ldcg(out + row + 1) + y1;
                    } else {
                        out[row >> 1] = silu(y0) * y1;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.empty[slot]));
        } else {
            float acc[1] = {0.f};
            dot_rows<1>(sp, 0, s.vec + g.kofs, g.elems, lane, acc);
            const float y = warp_sum(acc[0]);
            if (lane == 0) {
                const uint32_t us = (g.unit - r.u0) % UNIT_SLOTS;
                volatile float* part = s.unit_part + us * MAX_PIECES;
                part[g.piece] = y;
                __threadfence_block();
                const int old = atomicAdd(&s.unit_cnt[us], 1);
                if (old == (int)pl.chunks_per_unit - 1) {
                    __threadfence_block();
                    s.unit_cnt[us] = 0;
                    float row_y[2] = {0.f, 0.f};
                    for (uint32_t rr = 0; rr < pl.rows_per_unit; ++rr) {
                        float t = 0.f;
                        for (uint32_t j = 0; j < pl.ksplit; ++j) t += part[rr * pl.ksplit + j];
                        row_y[rr] = t;
                    }
                    const uint32_t row = g.unit * pl.rows_per_unit;
                    if (ep == EP_STORE) {
                        out[row] = row_y[0];
                        if (pl.rows_per_unit == 2) out[row + 1] = row_y[1];
                    } else if (ep == EP_RESIDUAL) {
                        out[row] = __ldcg(out + row) + row_y[0];
                        if (pl.rows_per_unit == 2) out[row + 1] = __ldcg(out + row + 1) + row_y[1];
                    } else {
                        out[row >> 1] = silu(row_y[0]) * row_y[1];
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&s.empty[slot]));
        }
    }
    nbase += nch;
}

// End of a stage: all consumer warps have written their outputs; one thread publishes the CTA's arrival.
__device__ __forceinline__ void stage_signal(uint32_t* ctr, uint32_t ctid, bool skip) {
    consumer_bar();
    if (ctid == 0 && !skip) {
        __threadfence();
        red_release_add(ctr, 1u);
    }
}

// Waits (bounded) until `target` CTAs have signalled.  Replaces the grid-wide barrier of a kernel boundary.
__device__ __forceinline__ void stage_wait(const Params& p, const Smem& s, const uint32_t* ctr, uint32_t target,
                                           uint32_t ctid) {
    if (ctid == 0) {
        if (*s.abort_flag == 0 && ld_acquire(ctr) < target) {
            const uint64_t t0 = globaltimer_ns();
            uint32_t it = 0;
            while (ld_acquire(ctr) < target) {
                if ((++it & 31u) == 0) {
                    if (*s.abort_flag) break;
                    if (__ldcg(p.status) != 0) {
                        *s.abort_flag = 1;
                        break;
                    }
                    if (globaltimer_ns() - t0 > p.wait_ns) {
                        raise_abort(p, s, ERR_SYNC_TIMEOUT);
                        break;
                    }
                }
            }
        }
    }
    consumer_bar();
}

// ------------------------------------------------------------------------------------------------ attention

__device__ __forceinline__ float ex2(float x) { return exp2f(x); }
__device__ __forceinline__ float rescale(float m, float M) { return m == -INFINITY ? 0.f : ex2(m - M); }

// Online-softmax state of one lane: G heads, the 8 value columns this lane owns.
template <int G>
struct AttnAcc {
    float m[G], l[G], a[G][8];
};

template <int G>
__device__ __forceinline__ void attn_update(AttnAcc<G>& st, const float (&q)[G][8], const uint4& kk, const uint4& vv,
                                            bool valid, uint32_t lpp) {
    const float kf[8] = {bf_lo(kk.x), bf_hi(kk.x), bf_lo(kk.y), bf_hi(kk.y),
                         bf_lo(kk.z), bf_hi(kk.z), bf_lo(kk.w), bf_hi(kk.w)};
    float sc[G];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float d = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) d = fmaf(q[h][j], kf[j], d);
        sc[h] = d;
    }
    for (uint32_t o = lpp >> 1; o > 0; o >>= 1) {
#pragma unroll
        for (int h = 0; h < G; ++h) sc[h] += __shfl_xor_sync(0xffffffffu, sc[h], o);
    }
    if (!valid) return;
    const float vf[8] = {bf_lo(vv.x), bf_hi(vv.x), bf_lo(vv.y), bf_hi(vv.y),
                         bf_lo(vv.z), bf_hi(vv.z), bf_lo(vv.w), bf_hi(vv.w)};
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (sc[h] > st.m[h]) {
            const float c = ex2(st.m[h] - sc[h]);  // exp2(-inf) = 0 on the first position
            st.l[h] *= c;
#pragma unroll
            for (int j = 0; j < 8; ++j) st.a[h][j] *= c;
            st.m[h] = sc[h];
        }
        const float pr = ex2(sc[h] - st.m[h]);
        st.l[h] += pr;
#pragma unroll
        for (int j = 0; j < 8; ++j) st.a[h][j] = fmaf(pr, vf[j], st.a[h][j]);
    }
}

// Split-K decode attention of one layer (flash-decoding): CTA `cta` owns at most one unit
// (sequence b, kv head g, chunk of cached positions); the last CTA to finish a (b, g) merges its chunks.
// Scores use q pre-multiplied by log2(e)/sqrt(hd), so the softmax runs in base 2.
template <int G>
__device__ __forceinline__ void attention_stage(const Params& p, const Smem& s, uint32_t layer, uint32_t cta,
                                                uint32_t ctid, uint32_t warp, uint32_t lane) {
    const uint32_t hd = p.hd, half = hd >> 1;
    const uint32_t bg = cta / p.cps, ch = cta % p.cps;
    if (bg >= p.B * p.nkv) return;
    const uint32_t b = bg / p.nkv, g = bg % p.nkv;
    const uint32_t pos = (uint32_t)p.positions[b];
    const uint32_t n = pos + 1;
    uint32_t nchunk = min(p.cps, (n + MIN_POS_PER_CHUNK - 1) / MIN_POS_PER_CHUNK);
    const uint32_t clen = (n + nchunk - 1) / nchunk;
    nchunk = (n + clen - 1) / clen;
    if (ch >= nchunk) return;
    const uint32_t c0 = ch * clen;
    const uint32_t c1 = min(n, c0 + clen);
    const bool has_new = (c1 == n);
    const uint32_t cend = has_new ? pos : c1;  // cached positions [c0, cend) come from the cache

    // shared workspace inside the vector area
    float* q_s = s.vec;                         // [G][hd]
    float* new_k = q_s + G * hd;                // [hd]
    float* new_v = new_k + hd;                  // [hd]
    float* comb = new_v + hd;                   // [NCW][G][hd + 2]

    const float* qkv = p.qkv + (size_t)b * (p.QD + 2 * p.KVD);
    const float* cs = p.rope_cs + (size_t)b * hd;  // [half][2]
    const size_t head_elems = (size_t)p.max_ctx * hd;
    __nv_bfloat16* Kc = p.kv + ((((size_t)layer * 2 + 0) * p.B + b) * p.nkv + g) * head_elems;
    __nv_bfloat16* Vc = p.kv + ((((size_t)layer * 2 + 1) * p.B + b) * p.nkv + g) * head_elems;

    const float qscale = 1.4426950408889634f * rsqrtf((float)hd);
    for (uint32_t idx = ctid; idx < G * half; idx += NCT) {
        const uint32_t h = idx / half, i = idx % half;
        const float* qr = qkv + (size_t)(g * G + h) * hd;
        const float a = __ldcg(qr + i), bb = __ldcg(qr + i + half);
        const float c = cs[2 * i], sn = cs[2 * i + 1];
        q_s[h * hd + i] = (a * c - bb * sn) * qscale;
        q_s[h * hd + i + half] = (bb * c + a * sn) * qscale;
    }
    if (has_new) {
        const float* kr = qkv + p.QD + (size_t)g * hd;
        const float* vr = qkv + p.QD + p.KVD + (size_t)g * hd;
        for (uint32_t i = ctid; i < half; i += NCT) {
            const float a = __ldcg(kr + i), bb = __ldcg(kr + i + half);
            const float c = cs[2 * i], sn = cs[2 * i + 1];
            const __nv_bfloat16 k0 = __float2bfloat16_rn(a * c - bb * sn);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(bb * c + a * sn);
            Kc[(size_t)pos * hd + i] = k0;
            Kc[(size_t)pos * hd + i + half] = k1;
            new_k[i] = __bfloat162float(k0);
            new_k[i + half] = __bfloat162float(k1);
        }
        for (uint32_t d = ctid; d < hd; d += NCT) {
            const __nv_bfloat16 v0 = __float2bfloat16_rn(__ldcg(vr + d));
            Vc[(size_t)pos * hd + d] = v0;
            new_v[d] = __bfloat162float(v0);
        }
    }
    consumer_bar();

    const uint32_t lpp = hd >> 3;           // lanes per position
    const uint32_t ppw = 32 / lpp;          // positions per warp step
    const uint32_t grp = lane / lpp, lig = lane % lpp;

    float q[G][8];
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
        for (int j = 0; j < 8; ++j) q[h][j] = q_s[h * hd + lig * 8 + j];

    AttnAcc<G> st;
#pragma unroll
    for (int h = 0; h < G; ++h) {
        st.m[h] = -INFINITY;
        st.l[h] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) st.a[h][j] = 0.f;
    }

    const uint32_t len = cend - c0;
    const uint32_t per_warp = (len + NCW - 1) / NCW;
    const uint32_t w0 = c0 + min(len, warp * per_warp);
    const uint32_t w1 = c0 + min(len, (warp + 1) * per_warp);
    constexpr int U = 4;
    for (uint32_t base = w0; base < w1; base += ppw * U) {
        uint4 kk[U], vv[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t t = base + u * ppw + grp;
            ok[u] = t < w1;
            kk[u] = make_uint4(0, 0, 0, 0);
            vv[u] = make_uint4(0, 0, 0, 0);
            if (ok[u]) {
                kk[u] = ldg_stream16(Kc + (size_t)t * hd + lig * 8);
                vv[u] = ldg_stream16(Vc + (size_t)t * hd + lig * 8);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) attn_update<G>(st, q, kk[u], vv[u], ok[u], lpp);
    }
    if (has_new && warp == 0) {
        // the position written by this step: its K/V come from shared memory (already rounded to bf16)
        uint4 kk, vv;
        const float* kp = new_k + lig * 8;
        const float* vp = new_v + lig * 8;
        kk.x = (__float_as_uint(kp[0]) >> 16) | (__float_as_uint(kp[1]) & 0xffff0000u);
        kk.y = (__float_as_uint(kp[2]) >> 16) | (__float_as_uint(kp[3]) & 0xffff0000u);
        kk.z = (__float_as_uint(kp[4]) >> 16) | (__float_as_uint(kp[5]) & 0xffff0000u);
        kk.w = (__float_as_uint(kp[6]) >> 16) | (__float_as_uint(kp[7]) & 0xffff0000u);
        vv.x = (__float_as_uint(vp[0]) >> 16) | (__float_as_uint(vp[1]) & 0xffff0000u);
        vv.y = (__float_as_uint(vp[2]) >> 16) | (__float_as_uint(vp[3]) & 0xffff0000u);
        vv.z = (__float_as_uint(vp[4]) >> 16) | (__float_as_uint(vp[5]) & 0xffff0000u);
        vv.w = (__float_as_uint(vp[6]) >> 16) | (__float_as_uint(vp[7]) & 0xffff0000u);
        attn_update<G>(st, q, kk, vv, grp == 0, lpp);
    }

    // merge the position groups of the warp (lanes with equal lig)
    for (uint32_t o = lpp; o < 32; o <<= 1) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float mo = __shfl_xor_sync(0xffffffffu, st.m[h], o);
            const float lo = __shfl_xor_sync(0xffffffffu, st.l[h], o);
            const float M = fmaxf(st.m[h], mo);
            const float cs_ = rescale(st.m[h], M), co = rescale(mo, M);
            st.l[h] = st.l[h] * cs_ + lo * co;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float ao = __shfl_xor_sync(0xffffffffu, st.a[h][j], o);
                st.a[h][j] = st.a[h][j] * cs_ + ao * co;
            }
            st.m[h] = M;
        }
    }
    if (grp == 0) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float* dst = comb + ((size_t)warp * G + h) * (hd + 2);
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[lig * 8 + j] = st.a[h][j];
            if (lig == 0) {
                dst[hd] = st.m[h];
                dst[hd + 1] = st.l[h];
            }
        }
    }
    consumer_bar();

    // merge the warps; thread t owns (head, column)
    const uint32_t unit = bg * p.cps + ch;
    for (uint32_t t = ctid; t < G * hd; t += NCT) {
        const uint32_t h = t / hd, d = t % hd;
        float M = -INFINITY;
        for (int w = 0; w < NCW; ++w) M = fmaxf(M, comb[((size_t)w * G + h) * (hd + 2) + hd]);
        float A = 0.f, Lsum = 0.f;
        for (int w = 0; w < NCW; ++w) {
            const float* src = comb + ((size_t)w * G + h) * (hd + 2);
            const float c = rescale(src[hd], M);
            A += src[d] * c;
            Lsum += src[hd + 1] * c;
        }
        if (nchunk == 1) {
            p.o[(size_t)b * p.QD + (size_t)(g * G + h) * hd + d] = A / Lsum;
        } else {
            p.part[((size_t)unit * G + h) * hd + d] = A;
            if (d == 0) {
                p.part_ml[((size_t)unit * G + h) * 2] = M;
                p.part_ml[((size_t)unit * G + h) * 2 + 1] = Lsum;
            }
        }
    }
    if (nchunk == 1) return;

    // ticket: the last unit of (b, g) to arrive merges all chunks
    consumer_bar();
    if (ctid == 0) {
        __threadfence();
        const uint32_t old = atom_add_acq_rel(p.tickets + (size_t)layer * p.B * p.nkv + bg, 1u);
        *s.bcast = (old == nchunk - 1) ? 1 : 0;
    }
    consumer_bar();
    if (*s.bcast == 0) return;
    const uint32_t unit0 = bg * p.cps;
    for (uint32_t t = ctid; t < G * hd; t += NCT) {
        const uint32_t h = t / hd, d = t % hd;
        float Mx = -INFINITY;
        for (uint32_t c = 0; c < nchunk; ++c) Mx = fmaxf(Mx, __ldcg(p.part_ml + ((size_t)(unit0 + c) * G + h) * 2));
        float Ax = 0.f, Lx = 0.f;
        for (uint32_t c = 0; c < nchunk; ++c) {
            const size_t u = (size_t)(unit0 + c) * G + h;
            const float sc = rescale(__ldcg(p.part_ml + u * 2), Mx);
            Ax += __ldcg(p.part + u * hd + d) * sc;
            Lx += __ldcg(p.part_ml + u * 2 + 1) * sc;
        }
        p.o[(size_t)b * p.QD + (size_t)(g * G + h) * hd + d] = Ax / Lx;
    }
}

}  // namespace kl
