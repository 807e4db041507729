// Device-side building blocks of the kernel-looped decoder: PTX wrappers (mbarrier, TMA bulk copy,
// acquire/release counters), the shared-memory weight ring, the GEMV stage consumer and the split-K
// attention stage.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kl {

constexpr int NCW = 8;                     // warps per CTA (two per scheduler, 255 registers each); warp w owns ring
                                           // slot w and keeps it filled itself
constexpr int NCT = NCW * 32;              // threads that take part in the CTA-wide steps (all of them)
constexpr int NTHREADS = NCT;
constexpr int SLOT_BYTES = 16384;          // one ring slot = one TMA bulk copy
constexpr int MAX_SLOTS = NCW;             // one owner warp per slot (see WarpRing)
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
    CUtensorMap kv_map;    // the whole KV cache as a 2-D tensor [rows, head_dim], 128-byte swizzle (64-byte aligned)
    uint32_t attn_tc;      // 1: tensor-core attention loop fed by kv_map boxes; 0: CUDA-core loop fed by linear copies
    uint32_t L, H, nq, nkv, hd, F, V, G, QD, KVD, max_ctx, B;
    uint32_t P;            // CTAs in the persistent grid
    uint32_t nslots;       // ring slots
    uint32_t vec_floats;   // capacity of the shared input-vector area
    uint32_t cps;          // attention: CTA slots per (sequence, kv head)
    uint32_t prefetch_chunks;  // L2 look-ahead of the producer beyond the ring, in chunks (0 = off)
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
    unsigned long long* trace;  // optional [P][L][TRACE_STAMPS] globaltimer stamps of consumer thread 0, or null
    unsigned long long* chunk_trace;  // optional [CHUNK_TRACE_ROWS][4] per-chunk stamps of CTA 0 (issue, wait, full, done)
};
constexpr uint32_t CHUNK_TRACE_ROWS = 8192;


// ------------------------------------------------------------------------------------------------ PTX

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

constexpr int TRACE_STAMPS = 16;
__device__ __forceinline__ void chunk_stamp(const Params& p, uint32_t cta, uint64_t n, int k) {
    if (p.chunk_trace != nullptr && cta == 0 && n < CHUNK_TRACE_ROWS) p.chunk_trace[n * 4 + k] = globaltimer_ns();
}
__device__ __forceinline__ void trace_stamp(const Params& p, uint32_t cta, uint32_t layer, int k, uint32_t ctid) {
    if (p.trace != nullptr && ctid == 0) p.trace[((size_t)cta * p.L + layer) * TRACE_STAMPS + k] = globaltimer_ns();
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
    struct SeqPlan* plan;   // this CTA's chunk sequence (written once by thread 0)
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
    s.plan = reinterpret_cast<struct SeqPlan*>(misc + 128);
    s.red = reinterpret_cast<float*>(misc + 1024);
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

// Geometry of the split-K attention unit of one CTA: (sequence b, kv head g, chunk ch of the cached positions).
// Producer and consumers derive it from the same device-resident positions, so they agree on the ring chunks.
struct AttnUnit {
    bool active;
    bool has_new;     // the chunk ends with the position written by this step
    uint32_t bg, b, g, ch, pos, nchunk;
    uint32_t c0, cend;  // cached positions [c0, cend) are streamed from the KV cache through the ring
    uint32_t nring;     // ring chunks of this unit
};
__device__ __forceinline__ uint32_t attn_positions_per_chunk(const Params& p) { return SLOT_BYTES / (4u * p.hd); }
__device__ __forceinline__ AttnUnit attn_unit(const Params& p, uint32_t cta) {
    AttnUnit u;
    u.active = false;
    u.nring = 0;
    u.bg = cta / p.cps;
    u.ch = cta % p.cps;
    if (u.bg >= p.B * p.nkv) return u;
    u.b = u.bg / p.nkv;
    u.g = u.bg % p.nkv;
    u.pos = (uint32_t)p.positions[u.b];
    const uint32_t n = u.pos + 1;
    uint32_t nchunk = min(p.cps, (n + MIN_POS_PER_CHUNK - 1) / MIN_POS_PER_CHUNK);
    const uint32_t clen = (n + nchunk - 1) / nchunk;
    u.nchunk = (n + clen - 1) / clen;
    if (u.ch >= u.nchunk) return u;
    u.active = true;
    u.c0 = u.ch * clen;
    const uint32_t c1 = min(n, u.c0 + clen);
    u.has_new = (c1 == n);
    u.cend = u.has_new ? u.pos : c1;
    const uint32_t pb = attn_positions_per_chunk(p);
    u.nring = (u.cend - u.c0 + pb - 1) / pb;
    return u;
}
__device__ __forceinline__ const __nv_bfloat16* kv_head(const Params& p, uint32_t layer, uint32_t kv, uint32_t b, uint32_t g) {
    return p.kv + ((((size_t)layer * 2 + kv) * p.B + b) * p.nkv + g) * ((size_t)p.max_ctx * p.hd);
}

// ------------------------------------------------------------------------------------------------ chunk streams

// This CTA's share of one matrix: a run of contiguous chunks.
struct StageStream {
    uint64_t byte_off;    // offset of the first chunk inside the matrix
    uint32_t nch;         // chunks
    uint32_t bytes_a;     // size of a regular chunk
    uint32_t bytes_b;     // size of every period-th chunk (the last piece of a row); == bytes_a for whole-row chunks
    uint32_t period;
    uint32_t bytes_last;  // size of the final chunk of the share (ragged tail of the matrix)
};
__device__ __forceinline__ StageStream make_stream(const GemvPlan& pl, uint32_t cta, uint32_t P) {
    const CtaRange r = cta_units(pl, cta, P);
    StageStream st;
    if (pl.rpc) {
        st.byte_off = (uint64_t)r.u0 * pl.rpc * pl.K * 2u;
        st.nch = r.u1 - r.u0;
        st.bytes_a = st.bytes_b = pl.rpc * pl.K * 2u;
        st.period = 1;
        st.bytes_last = (r.u1 == pl.nunits) ? (pl.R - (pl.nunits - 1) * pl.rpc) * pl.K * 2u : st.bytes_a;
    } else {
        st.byte_off = (uint64_t)r.u0 * pl.rows_per_unit * pl.K * 2u;
        st.nch = (r.u1 - r.u0) * pl.chunks_per_unit;
        st.bytes_a = pl.klen * 2u;
        st.bytes_b = (pl.K - (pl.ksplit - 1) * pl.klen) * 2u;
        st.period = pl.ksplit;
        st.bytes_last = st.bytes_b;
    }
    return st;
}

__device__ __forceinline__ void tma_tensor_2d_g2s(uint32_t dst, const void* tmap, int32_t x, int32_t y, uint32_t bar,
                                                  uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar), "l"(pol)
        : "memory");
}

// Window of cache rows a ring chunk of the tensor-core path holds.  Chunk i of a unit covers positions
// [c0 + i*pb, min(.. + pb, cend)); the box always has pb rows, so a short last chunk is slid back to end at cend
// (rows before the chunk's first position are valid cache rows that are simply ignored).
struct AttnWindow {
    uint32_t w0;      // cache position of box row 0
    uint32_t lo, hi;  // rows [lo, hi) of the box are this chunk's positions
};
__device__ __forceinline__ AttnWindow attn_window(uint32_t c0, uint32_t cend, uint32_t pb, uint32_t i) {
    AttnWindow w;
    const uint32_t t0 = c0 + i * pb;
    const uint32_t end = min(t0 + pb, cend);
    w.w0 = end >= pb ? end - pb : 0u;
    w.lo = t0 - w.w0;
    w.hi = end - w.w0;
    return w;
}

// ------------------------------------------------------------------------------------------------ chunk sequence
//
// The whole launch as one sequence of 16 KB chunks per CTA, in consumption order: for every layer the CTA's QKV
// rows, the K/V rows of its attention unit, its O rows, gate/up rows and down rows.  Every address is known when
// the kernel starts (weights are grouped per layer and linear in memory; cached K/V rows were written by earlier
// launches).  Chunk n lives in ring slot n % nslots, and warp (n % nslots) both consumes it and, the moment it has
// read the slot for the last time, starts the TMA copy of chunk n + nslots into the same slot.  So each warp runs
// its own pipeline through its own slot: there is no producer thread to serialise the issue, every parity wait is
// made by the one warp that armed the barrier, and the copies for the next stage -- or, in the looped kernel, the
// next layer -- are in flight while the warp sits in the counter wait that replaces a kernel boundary.
struct SeqPlan {
    StageStream st[4];         // QKV, O, GU, D  (for the classifier kernel: st[0] only)
    const uint8_t* base[4];    // layer-0 base of each matrix
    uint64_t layer_bytes;      // bytes between layers of a matrix
    uint32_t cnt[5];           // chunks per stage: QKV, attention, O, GU, D
    uint32_t per_layer;        // sum of cnt
    // attention unit (one slot holds K rows in its first half, V rows of the same positions in its second half)
    uint32_t attn_len, pb, row_bytes;
    const uint8_t* k0;         // layer-0 K rows of the unit's first position
    const uint8_t* v0;
    uint64_t kv_layer_bytes;
    // tensor-core attention: the same rows addressed as rows of the 2-D cache tensor
    uint32_t tc, c0, cend;
    uint32_t k_row0;           // tensor row of position 0 of the unit's (sequence, kv head), K half, layer 0
    uint32_t v_row_delta;      // rows from a K row to the matching V row
    uint32_t rows_per_layer;
    uint32_t l1;
};

__device__ __forceinline__ void make_decoder_plan(SeqPlan& q, const Params& p, uint32_t cta, uint32_t l1) {
    q.st[0] = make_stream(p.plan[PL_QKV], cta, p.P);
    q.st[1] = make_stream(p.plan[PL_O], cta, p.P);
    q.st[2] = make_stream(p.plan[PL_GU], cta, p.P);
    q.st[3] = make_stream(p.plan[PL_D], cta, p.P);
    q.base[0] = reinterpret_cast<const uint8_t*>(p.wqkv);
    q.base[1] = reinterpret_cast<const uint8_t*>(p.wo);
    q.base[2] = reinterpret_cast<const uint8_t*>(p.wgu);
    q.base[3] = reinterpret_cast<const uint8_t*>(p.wd);
    q.layer_bytes = p.layer_stride * 2ull;
    const AttnUnit u = attn_unit(p, cta);
    q.attn_len = u.active ? u.cend - u.c0 : 0u;
    q.pb = attn_positions_per_chunk(p);
    q.row_bytes = p.hd * 2u;
    q.k0 = q.v0 = nullptr;
    if (u.active) {
        q.k0 = reinterpret_cast<const uint8_t*>(kv_head(p, 0, 0, u.b, u.g)) + (size_t)u.c0 * q.row_bytes;
        q.v0 = reinterpret_cast<const uint8_t*>(kv_head(p, 0, 1, u.b, u.g)) + (size_t)u.c0 * q.row_bytes;
    }
    q.kv_layer_bytes = 2ull * p.B * p.nkv * p.max_ctx * p.hd * 2ull;
    q.tc = p.attn_tc;
    q.c0 = u.active ? u.c0 : 0u;
    q.cend = u.active ? u.cend : 0u;
    q.k_row0 = u.active ? (u.b * p.nkv + u.g) * p.max_ctx : 0u;
    q.v_row_delta = p.B * p.nkv * p.max_ctx;
    q.rows_per_layer = 2u * q.v_row_delta;
    q.cnt[0] = q.st[0].nch;
    q.cnt[1] = u.nring;
    q.cnt[2] = q.st[1].nch;
    q.cnt[3] = q.st[2].nch;
    q.cnt[4] = q.st[3].nch;
    q.per_layer = q.cnt[0] + q.cnt[1] + q.cnt[2] + q.cnt[3] + q.cnt[4];
    q.l1 = l1;
}
__device__ __forceinline__ void make_classifier_plan(SeqPlan& q, const Params& p, uint32_t cta) {
    q.st[0] = make_stream(p.plan[PL_LM], cta, p.P);
    q.st[1] = q.st[2] = q.st[3] = q.st[0];
    q.base[0] = q.base[1] = q.base[2] = q.base[3] = reinterpret_cast<const uint8_t*>(p.wlm);
    q.layer_bytes = 0;
    q.attn_len = 0;
    q.pb = 1;
    q.row_bytes = 0;
    q.k0 = q.v0 = nullptr;
    q.kv_layer_bytes = 0;
    q.tc = q.c0 = q.cend = q.k_row0 = q.v_row_delta = q.rows_per_layer = 0;
    q.cnt[0] = q.st[0].nch;
    q.cnt[1] = q.cnt[2] = q.cnt[3] = q.cnt[4] = 0;
    q.per_layer = q.cnt[0];
    q.l1 = 1;
}

struct SeqPos {
    uint32_t l, stage, i;   // stage: 0 QKV, 1 attention, 2 O, 3 GU, 4 D; i = chunk index inside the stage
    bool done;
};
__device__ __forceinline__ void seq_normalize(const SeqPlan& q, SeqPos& r) {
    if (q.per_layer == 0) {
        r.done = true;
        return;
    }
    while (r.i >= q.cnt[r.stage]) {
        r.i -= q.cnt[r.stage];
        if (++r.stage == 5) {
            r.stage = 0;
            if (++r.l >= q.l1) {
                r.done = true;
                return;
            }
        }
    }
}
struct ChunkSrc {
    const uint8_t* src0;
    const uint8_t* src1;
    uint32_t bytes0, bytes1;
};
__device__ __forceinline__ ChunkSrc seq_chunk(const SeqPlan& q, const SeqPos& r) {
    ChunkSrc c;
    c.src1 = nullptr;
    c.bytes1 = 0;
    if (r.stage == 1) {
        const uint32_t t = r.i * q.pb;
        const uint32_t np = min(q.pb, q.attn_len - t);
        c.bytes0 = c.bytes1 = np * q.row_bytes;
        c.src0 = q.k0 + (size_t)r.l * q.kv_layer_bytes + (size_t)t * q.row_bytes;
        c.src1 = q.v0 + (size_t)r.l * q.kv_layer_bytes + (size_t)t * q.row_bytes;
    } else {
        const uint32_t m = r.stage == 0 ? 0u : r.stage - 1u;
        const StageStream& st = q.st[m];
        uint64_t off;
        if (st.period == 1) {
            off = (uint64_t)r.i * st.bytes_a;
            c.bytes0 = (r.i == st.nch - 1) ? st.bytes_last : st.bytes_a;
        } else {
            const uint32_t row = r.i / st.period, j = r.i % st.period;
            off = (uint64_t)row * ((st.period - 1) * st.bytes_a + st.bytes_b) + (uint64_t)j * st.bytes_a;
            c.bytes0 = (j == st.period - 1) ? st.bytes_b : st.bytes_a;
        }
        c.src0 = q.base[m] + (size_t)r.l * q.layer_bytes + st.byte_off + off;
    }
    return c;
}

__device__ __forceinline__ void l2_prefetch(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// Everything lane 0 needs to start the copies of a chunk, worked out ahead of time.
struct ChunkIssue {
    const uint8_t* src0;   // linear copies: sources; tensor boxes: unused
    const uint8_t* src1;
    uint32_t bytes0, bytes1;
    int32_t yk, yv;        // tensor boxes: first cache row of the K and of the V boxes
    bool boxes;
};
__device__ __forceinline__ ChunkIssue seq_issue_info(const SeqPlan& q, const SeqPos& r) {
    ChunkIssue c;
    c.boxes = (r.stage == 1 && q.tc != 0);
    c.yk = c.yv = 0;
    if (c.boxes) {
        const AttnWindow w = attn_window(q.c0, q.cend, q.pb, r.i);
        c.yk = (int32_t)(q.k_row0 + r.l * q.rows_per_layer + w.w0);
        c.yv = c.yk + (int32_t)q.v_row_delta;
        c.src0 = c.src1 = nullptr;
        c.bytes0 = c.bytes1 = SLOT_BYTES / 2;
    } else {
        const ChunkSrc l = seq_chunk(q, r);
        c.src0 = l.src0;
        c.src1 = l.src1;
        c.bytes0 = l.bytes0;
        c.bytes1 = l.bytes1;
    }
    return c;
}

// State of a warp's slot: the next chunk it will issue, the chunk it will prefetch into L2, and the use counts.
struct WarpRing {
    SeqPos pos;             // next chunk to issue
    ChunkIssue nx;          // how to issue pos (precomputed)
    SeqPos ahead;           // chunk to prefetch into L2 at the next issue (pos + prefetch_chunks turns)
    uint32_t n;             // global index of pos (for the optional chunk log)
    uint32_t issued;        // copies armed on this warp's barrier so far
    uint32_t uses;          // chunks taken from the slot so far; (uses & 1) is the phase to wait for
};

// Arms the warp's barrier and starts the copies of its next chunk (lane 0) from the precomputed description, then
// steps nslots chunks ahead and works out the following chunk -- that arithmetic overlaps with the copy just
// started.  Called once the whole warp has finished reading the slot (after __syncwarp).
// With Params::prefetch_chunks = k > 0 the warp also asks L2 to fetch the chunk it will issue k turns later.
__device__ __forceinline__ void ring_issue_next(const Params& p, const Smem& s, WarpRing& r, uint32_t warp, uint32_t lane,
                                                uint64_t pol) {
    if (r.pos.done || *s.abort_flag) return;
    if (lane == 0) {
        const ChunkIssue& c = r.nx;
        const uint32_t bar = smem_u32(&s.full[warp]);
        const uint32_t dst = smem_u32(s.ring) + warp * SLOT_BYTES;
        // the slot was read through the generic proxy; the copies write it through the async proxy
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        chunk_stamp(p, blockIdx.x, r.n, 0);
        mbar_arrive_expect_tx(bar, c.bytes0 + c.bytes1);
        if (c.boxes) {
            // K/V rows as swizzled boxes of the cache tensor: [pb rows] x [64 columns] per box, K boxes in the first
            // half of the slot, V boxes in the second; a box is always written whole (rows outside the chunk's own
            // positions are ignored by the consumer)
            const uint32_t box_bytes = SLOT_BYTES / 2 / (p.hd / 64u);
            for (uint32_t bx = 0; bx < p.hd / 64u; ++bx) {
                tma_tensor_2d_g2s(dst + bx * box_bytes, &p.kv_map, (int32_t)(bx * 64u), c.yk, bar, pol);
                tma_tensor_2d_g2s(dst + SLOT_BYTES / 2 + bx * box_bytes, &p.kv_map, (int32_t)(bx * 64u), c.yv, bar, pol);
            }
        } else {
            tma_bulk_g2s(dst, c.src0, c.bytes0, bar, pol);
            if (c.bytes1) tma_bulk_g2s(dst + SLOT_BYTES / 2, c.src1, c.bytes1, bar, pol);
        }
    }
    ++r.issued;
    const SeqPlan& q = *s.plan;
    r.pos.i += p.nslots;
    r.n += p.nslots;
    seq_normalize(q, r.pos);
    if (!r.pos.done) r.nx = seq_issue_info(q, r.pos);
    if (p.prefetch_chunks && !r.ahead.done && !(r.ahead.stage == 1 && q.tc)) {
        const ChunkSrc f = seq_chunk(q, r.ahead);
        for (uint32_t o = lane * 128u; o < f.bytes0; o += 32u * 128u)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(f.src0 + o));
        for (uint32_t o = lane * 128u; o < f.bytes1; o += 32u * 128u)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(f.src1 + o));
        r.ahead.i += p.nslots;
        seq_normalize(q, r.ahead);
    }
}

__device__ __forceinline__ WarpRing ring_begin(const Params& p, const Smem& s, uint32_t warp, uint32_t l0) {
    WarpRing r;
    r.pos.l = l0;
    r.pos.stage = 0;
    r.pos.i = warp;
    r.pos.done = warp >= p.nslots || l0 >= s.plan->l1;
    r.n = warp;
    r.issued = 0;
    r.uses = 0;
    if (!r.pos.done) seq_normalize(*s.plan, r.pos);
    if (!r.pos.done) r.nx = seq_issue_info(*s.plan, r.pos);
    r.ahead = r.pos;
    if (!r.ahead.done) {
        r.ahead.i += p.prefetch_chunks * p.nslots;
        seq_normalize(*s.plan, r.ahead);
    }
    return r;
}

// Before the CTA exits no bulk copy may still be writing its shared memory: wait (bounded) for the last copy this
// warp armed.  On the normal path that copy was consumed long ago and the wait returns at once.
__device__ __forceinline__ void ring_finish(const Params& p, const Smem& s, const WarpRing& r, uint32_t warp) {
    if (r.issued == 0) return;
    const uint32_t bar = smem_u32(&s.full[warp]);
    const uint32_t parity = (r.issued - 1u) & 1u;
    const uint64_t t0 = globaltimer_ns();
    while (!mbar_try_wait(bar, parity)) {
        if (globaltimer_ns() - t0 > p.wait_ns) return;
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
    constexpr int NB = 8;  // float4 loads kept in flight per thread: one L2 round trip per NB * NCT * 4 elements
    if (norm && n <= (uint32_t)(NB * NCT * 4)) {
        // whole vector in registers: x and gains are fetched together, one round trip before the reduction
        float4 v[NB];
        uint2 gb[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = (ctid + i * NCT) * 4;
            v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            gb[i] = make_uint2(0u, 0u);
            if (e < n) {
                v[i] = __ldcg(reinterpret_cast<const float4*>(src + e));
                gb[i] = __ldg(reinterpret_cast<const uint2*>(gain + e));
            }
        }
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < NB; ++i) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((ctid & 31) == 0) s.red[ctid >> 5] = ss;
        consumer_bar();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < NCW; ++w) tot += s.red[w];
        const float inv = rsqrtf(tot / (float)n + p.eps);
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = (ctid + i * NCT) * 4;
            if (e < n) {
                float4 o;
                o.x = v[i].x * inv * bf_lo(gb[i].x);
                o.y = v[i].y * inv * bf_hi(gb[i].x);
                o.z = v[i].z * inv * bf_lo(gb[i].y);
                o.w = v[i].w * inv * bf_hi(gb[i].y);
                *reinterpret_cast<float4*>(s.vec + vec_perm(e)) = o;
            }
        }
        consumer_bar();
        return;
    }
    float ss = 0.f;
    for (uint32_t base = 0; base < n; base += NB * NCT * 4) {
        float4 v[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * NCT) * 4;
            v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e < n) v[i] = __ldcg(reinterpret_cast<const float4*>(src + e));
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * NCT) * 4;
            ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
            if (e < n) *reinterpret_cast<float4*>(s.vec + vec_perm(e)) = v[i];
        }
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
            const uint2 gb = __ldg(reinterpret_cast<const uint2*>(gain + e));
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
// One 256-column block of the dot products: this lane's 8 columns of NR rows against its 8 vector elements,
// into two accumulators per row (even and odd columns) so that the FMA chains stay short.
template <int NR>
__device__ __forceinline__ void dot_block(const uint4 (&q)[NR], const float4& xa, const float4& xb, float (&e)[NR],
                                          float (&o)[NR]) {
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        e[r] = fmaf(bf_lo(q[r].x), xa.x, e[r]);
        o[r] = fmaf(bf_hi(q[r].x), xa.y, o[r]);
        e[r] = fmaf(bf_lo(q[r].y), xa.z, e[r]);
        o[r] = fmaf(bf_hi(q[r].y), xa.w, o[r]);
        e[r] = fmaf(bf_lo(q[r].z), xb.x, e[r]);
        o[r] = fmaf(bf_hi(q[r].z), xb.y, o[r]);
        e[r] = fmaf(bf_lo(q[r].w), xb.z, e[r]);
        o[r] = fmaf(bf_hi(q[r].w), xb.w, o[r]);
    }
}

// acc[r] += sum over this lane's columns of W[r][k] * vec[k]; W rows in shared memory, row pitch rowbytes.
// Four blocks are loaded before any is used, so the shared-memory latency overlaps with the arithmetic.
template <int NR>
__device__ __forceinline__ void dot_rows(const uint8_t* w, uint32_t rowbytes, const float* vec, uint32_t len,
                                         uint32_t lane, float (&acc)[NR]) {
    const float4* v4 = reinterpret_cast<const float4*>(vec);
    float e[NR], o[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) e[r] = o[r] = 0.f;
    const uint32_t nblk = len >> 8;  // full 256-column blocks
    uint32_t blk = 0;
    for (; blk + 4 <= nblk; blk += 4) {
        float4 xa[4], xb[4];
        uint4 q[4][NR];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            xa[u] = v4[(blk + u) * 64 + lane];
            xb[u] = v4[(blk + u) * 64 + 32 + lane];
#pragma unroll
            for (int r = 0; r < NR; ++r)
                q[u][r] = *reinterpret_cast<const uint4*>(w + (size_t)r * rowbytes + (size_t)((blk + u) * 256 + lane * 8) * 2);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) dot_block<NR>(q[u], xa[u], xb[u], e, o);
    }
    for (uint32_t k = blk * 256 + lane * 8; k < len; k += 256) {  // remaining blocks, the last possibly partial
        const uint32_t bk = k >> 8;
        const float4 xa = v4[bk * 64 + lane];
        const float4 xb = v4[bk * 64 + 32 + lane];
        uint4 q[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) q[r] = *reinterpret_cast<const uint4*>(w + (size_t)r * rowbytes + (size_t)k * 2);
        dot_block<NR>(q, xa, xb, e, o);
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] += e[r] + o[r];
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float silu(float z) { return z / (1.0f + __expf(-z)); }

// Where the CTA stands in its chunk sequence: `start` is the slot of the next stage's first chunk (chunks so far
// modulo the slot count, identical for every warp).
struct RingCursor {
    uint32_t start;
    uint32_t n0;  // chunks before the current stage (for the optional chunk log)
    __device__ __forceinline__ uint32_t first_chunk(uint32_t warp, uint32_t nslots) const {
        return warp < nslots ? (warp + nslots - start) % nslots : warp;
    }
    __device__ __forceinline__ void advance(uint32_t nch, uint32_t nslots) {
        start = (start + nch) % nslots;
        n0 += nch;
    }
};

// Consumes this CTA's share of one matrix from the ring: y = W vec, followed by the stage's epilogue.
//   EP_STORE    out[row] = y
//   EP_RESIDUAL out[row] = out[row] + y            (out is the hidden state, owned row-wise by this CTA)
//   EP_SWIGLU   rows come in (gate, up) pairs: out[row/2] = silu(y_gate) * y_up
// The cursor follows the producer's issue order.
// Chunk n lives in slot n % nslots and is consumed by warp n % nslots: every use of a slot is waited on by the
// same warp, in order, so a parity wait can never be satisfied by a phase two uses old.  (With free chunk-to-warp
// assignment a fast warp can test the barrier of use k while use k-1 is still in flight, and parity k&1 then
// reads as complete.)
__device__ __forceinline__ void gemv_stage(const Params& p, const Smem& s, const GemvPlan& pl, int ep, float* out,
                                           uint32_t cta, uint32_t warp, uint32_t lane, RingCursor& rc, WarpRing& wr,
                                           uint64_t pol) {
    const CtaRange r = cta_units(pl, cta, p.P);
    const uint32_t nch = (r.u1 - r.u0) * pl.chunks_per_unit;
    const uint32_t first = rc.first_chunk(warp, p.nslots);
    for (uint32_t i = (warp < p.nslots ? first : nch); i < nch; i += p.nslots) {
        const uint32_t slot = warp;
        if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 1);
        mbar_wait(p, s, smem_u32(&s.full[slot]), wr.uses & 1u);
        if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 2);
        ++wr.uses;
        const uint8_t* sp = s.ring + (size_t)slot * SLOT_BYTES;
        const ChunkGeom g = chunk_geom(pl, r.u0, i);
        if (pl.rpc) {
            const uint32_t rowbytes = pl.K * 2u;
            for (uint32_t rr = 0; rr < g.nrows; rr += 2) {
                float y0, y1 = 0.f;
                float res0 = 0.f, res1 = 0.f;  // residual inputs, fetched before the dot products hide their latency
                if (ep == EP_RESIDUAL && lane == 0) {
                    res0 = __ldcg(out + g.row + rr);
                    if (rr + 1 < g.nrows) res1 = __ldcg(out + g.row + rr + 1);
                }
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
                        out[row] = res0 + y0;
                        if (rr + 1 < g.nrows) out[row + 1] = res1 + y1;
                    } else {
                        out[row >> 1] = silu(y0) * y1;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 1);
            ring_issue_next(p, s, wr, warp, lane, pol);
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 3);
        } else {
            float resb[2] = {0.f, 0.f};
            if (ep == EP_RESIDUAL && lane == 0) {
                resb[0] = __ldcg(out + g.unit * pl.rows_per_unit);
                if (pl.rows_per_unit == 2) resb[1] = __ldcg(out + g.unit * pl.rows_per_unit + 1);
            }
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
                        out[row] = resb[0] + row_y[0];
                        if (pl.rows_per_unit == 2) out[row + 1] = resb[1] + row_y[1];
                    } else {
                        out[row >> 1] = silu(row_y[0]) * row_y[1];
                    }
                }
            }
            __syncwarp();
            ring_issue_next(p, s, wr, warp, lane, pol);
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 3);
        }
    }
    rc.advance(nch, p.nslots);
}

// End of a stage: all consumer warps have written their outputs; one thread publishes the CTA's arrival.
__device__ __forceinline__ void stage_signal(uint32_t* ctr, uint32_t ctid, bool skip) {
    consumer_bar();
    if (ctid == 0 && !skip) red_release_add(ctr, 1u);  // release: cumulative over the CTA barrier above
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

}  // namespace kl
#include "kl_attention_tc.cuh"
namespace kl {

// Online-softmax state of one lane: G heads, the 8 value columns this lane owns.
template <int G>
struct AttnAcc {
    float m[G], l[G], a[G][8];
};

// One batch of U warp steps (U * 32/lpp positions): all scores first (independent dot products and butterfly
// reductions, so the instruction streams of the positions interleave), then ONE running-max update per head for the
// whole batch, then the value accumulation.  kk/vv hold this lane's 8 columns of each position's K/V row.
template <int G, int U>
__device__ __forceinline__ void attn_batch(AttnAcc<G>& st, const float (&q)[G][8], const uint4 (&kk)[U],
                                           const uint4 (&vv)[U], const bool (&valid)[U], uint32_t lpp) {
    float sc[U][G];
#pragma unroll
    for (int x = 0; x < U; ++x) {
        const float kf[8] = {bf_lo(kk[x].x), bf_hi(kk[x].x), bf_lo(kk[x].y), bf_hi(kk[x].y),
                             bf_lo(kk[x].z), bf_hi(kk[x].z), bf_lo(kk[x].w), bf_hi(kk[x].w)};
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float d = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) d = fmaf(q[h][j], kf[j], d);
            sc[x][h] = d;
        }
    }
    for (uint32_t o = lpp >> 1; o > 0; o >>= 1) {
#pragma unroll
        for (int x = 0; x < U; ++x)
#pragma unroll
            for (int h = 0; h < G; ++h) sc[x][h] += __shfl_xor_sync(0xffffffffu, sc[x][h], o);
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float mb = -INFINITY;
#pragma unroll
        for (int x = 0; x < U; ++x) mb = fmaxf(mb, valid[x] ? sc[x][h] : -INFINITY);
        const float mn = fmaxf(st.m[h], mb);
        const float c = rescale(st.m[h], mn);
        float pr[U];
        float ls = 0.f;
#pragma unroll
        for (int x = 0; x < U; ++x) {
            pr[x] = valid[x] ? ex2(sc[x][h] - mn) : 0.f;
            ls += pr[x];
        }
        st.l[h] = st.l[h] * c + ls;
        st.m[h] = mn;
#pragma unroll
        for (int j = 0; j < 8; ++j) st.a[h][j] *= c;
#pragma unroll
        for (int x = 0; x < U; ++x) {
            const float vf[8] = {bf_lo(vv[x].x), bf_hi(vv[x].x), bf_lo(vv[x].y), bf_hi(vv[x].y),
                                 bf_lo(vv[x].z), bf_hi(vv[x].z), bf_lo(vv[x].w), bf_hi(vv[x].w)};
#pragma unroll
            for (int j = 0; j < 8; ++j) st.a[h][j] = fmaf(pr[x], vf[j], st.a[h][j]);
        }
    }
}

// Ring chunks of the unit through the tensor-core loop; leaves this warp's partial result in comb[first].
template <int HD>
__device__ __forceinline__ void attn_chunks_tc(const Params& p, const Smem& s, const AttnUnit& u, uint32_t cta,
                                               uint32_t warp, uint32_t lane, uint32_t first, const RingCursor& rc,
                                               WarpRing& wr, uint64_t pol, const float* q_s, float* comb,
                                               const uint8_t* stage_k, const uint8_t* stage_v) {
    constexpr int NKB = HD / 16, NNT = HD / 8;
    const uint32_t G = p.G, g = lane >> 2, t = lane & 3u;
    AttnTcState<HD> st;
#pragma unroll
    for (int kb = 0; kb < NKB; ++kb) {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const uint32_t k = kb * 16 + hf * 8 + 2 * t;
            const float x0 = g < G ? q_s[g * HD + k] : 0.f, x1 = g < G ? q_s[g * HD + k + 1] : 0.f;
            const uint32_t hi = pack_bf16(x0, x1);
            st.qh[kb][hf] = hi;
            st.ql[kb][hf] = pack_bf16(x0 - bf_lo(hi), x1 - bf_hi(hi));
        }
    }
#pragma unroll
    for (int n = 0; n < NNT; ++n) st.o[n][0] = st.o[n][1] = st.o[n][2] = st.o[n][3] = 0.f;
    st.m = -INFINITY;
    st.l = 0.f;

    const uint32_t pb = attn_positions_per_chunk(p);
    const uint32_t box_bytes = pb * 128u;
    for (uint32_t i = (warp < p.nslots ? first : u.nring); i < u.nring; i += p.nslots) {
        if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 1);
        mbar_wait(p, s, smem_u32(&s.full[warp]), wr.uses & 1u);
        if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 2);
        ++wr.uses;
        const uint32_t kbase = smem_u32(s.ring) + warp * SLOT_BYTES;
        const AttnWindow w = attn_window(u.c0, u.cend, pb, i);
        for (uint32_t row0 = 0; row0 < pb; row0 += 16)
            if (row0 + 16 > w.lo && row0 < w.hi) attn_tc_tile<HD>(st, kbase, kbase + SLOT_BYTES / 2, box_bytes, row0, w.lo, w.hi, lane);
        __syncwarp();
        ring_issue_next(p, s, wr, warp, lane, pol);
        if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 3);
    }
    if (u.has_new && first == 0)  // the position written by this step sits in row 0 of the staging tile
        attn_tc_tile<HD>(st, smem_u32(stage_k), smem_u32(stage_v), 16u * 128u, 0u, 0u, 1u, lane);

    float l = st.l;
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (g < G) {
        float* dst = comb + ((size_t)first * G + g) * (HD + 2);
#pragma unroll
        for (int n = 0; n < NNT; ++n) {
            dst[n * 8 + 2 * t] = st.o[n][0];
            dst[n * 8 + 2 * t + 1] = st.o[n][1];
        }
        if (t == 0) {
            dst[HD] = st.m;
            dst[HD + 1] = l;
        }
    }
}

// Split-K decode attention of one layer (flash-decoding): CTA `cta` owns at most one unit; its cached K/V rows
// arrive through the ring (in flight while the QKV stage and its counter wait were still running); the last CTA
// to finish a (b, g) merges its chunks.  Scores use q pre-multiplied by log2(e)/sqrt(hd): the softmax runs in
// base 2.  GT > 0 selects the CUDA-core inner loop for GT query heads per KV head; GT == 0 the tensor-core loop.
template <int GT>
__device__ __noinline__ void attention_stage(const Params& p, const Smem& s, uint32_t layer, uint32_t cta,
                                                uint32_t ctid, uint32_t warp, uint32_t lane, RingCursor& rc, WarpRing& wr,
                                                uint64_t pol) {
    const AttnUnit u = attn_unit(p, cta);
    if (!u.active) return;
    const uint32_t G = GT > 0 ? (uint32_t)GT : p.G;
    const uint32_t hd = p.hd, half = hd >> 1;
    const uint32_t b = u.b, g = u.g, pos = u.pos, nchunk = u.nchunk;

    // shared workspace inside the vector area
    float* q_s = s.vec;                         // [G][hd]
    float* new_k = q_s + G * hd;                // [hd]
    float* new_v = new_k + hd;                  // [hd]
    float* comb = new_v + hd;                   // [NCW][G][hd + 2]
    uint8_t* stage_k = reinterpret_cast<uint8_t*>(comb + (size_t)NCW * G * (hd + 2));  // [hd/64][16 rows][128 B]
    uint8_t* stage_v = stage_k + hd * 32u;

    const float* qkv = p.qkv + (size_t)b * (p.QD + 2 * p.KVD);
    const float* cs = p.rope_cs + (size_t)b * hd;  // [half][2]
    __nv_bfloat16* Kc = const_cast<__nv_bfloat16*>(kv_head(p, layer, 0, b, g));
    __nv_bfloat16* Vc = const_cast<__nv_bfloat16*>(kv_head(p, layer, 1, b, g));

    const float qscale = 1.4426950408889634f * rsqrtf((float)hd);
    for (uint32_t idx = ctid; idx < G * half; idx += NCT) {
        const uint32_t h = idx / half, i = idx % half;
        const float* qr = qkv + (size_t)(g * G + h) * hd;
        const float a = __ldcg(qr + i), bb = __ldcg(qr + i + half);
        const float c = cs[2 * i], sn = cs[2 * i + 1];
        q_s[h * hd + i] = (a * c - bb * sn) * qscale;
        q_s[h * hd + i + half] = (bb * c + a * sn) * qscale;
    }
    if (u.has_new) {
        const float* kr = qkv + p.QD + (size_t)g * hd;
        const float* vr = qkv + p.QD + p.KVD + (size_t)g * hd;
        // row 0 of a swizzled box is stored unswizzled: column k of box k/64 sits at byte (k % 64) * 2
        for (uint32_t i = ctid; i < half; i += NCT) {
            const float a = __ldcg(kr + i), bb = __ldcg(kr + i + half);
            const float c = cs[2 * i], sn = cs[2 * i + 1];
            const __nv_bfloat16 k0 = __float2bfloat16_rn(a * c - bb * sn);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(bb * c + a * sn);
            Kc[(size_t)pos * hd + i] = k0;
            Kc[(size_t)pos * hd + i + half] = k1;
            new_k[i] = __bfloat162float(k0);
            new_k[i + half] = __bfloat162float(k1);
            if (GT == 0) {
                const uint32_t j = i + half;
                *reinterpret_cast<__nv_bfloat16*>(stage_k + (i >> 6) * 2048u + (i & 63u) * 2u) = k0;
                *reinterpret_cast<__nv_bfloat16*>(stage_k + (j >> 6) * 2048u + (j & 63u) * 2u) = k1;
            }
        }
        for (uint32_t d = ctid; d < hd; d += NCT) {
            const __nv_bfloat16 v0 = __float2bfloat16_rn(__ldcg(vr + d));
            Vc[(size_t)pos * hd + d] = v0;
            new_v[d] = __bfloat162float(v0);
            if (GT == 0) *reinterpret_cast<__nv_bfloat16*>(stage_v + (d >> 6) * 2048u + (d & 63u) * 2u) = v0;
        }
    }
    consumer_bar();
    trace_stamp(p, cta, layer, 14, ctid);

    const uint32_t first = rc.first_chunk(warp, p.nslots);
    if constexpr (GT == 0) {
        if (hd == 128)
            attn_chunks_tc<128>(p, s, u, cta, warp, lane, first, rc, wr, pol, q_s, comb, stage_k, stage_v);
        else
            attn_chunks_tc<64>(p, s, u, cta, warp, lane, first, rc, wr, pol, q_s, comb, stage_k, stage_v);
    } else {
        constexpr int G_ = GT > 0 ? GT : 1;
        const uint32_t lpp = hd >> 3;           // lanes per position
        const uint32_t ppw = 32 / lpp;          // positions per warp step
        const uint32_t grp = lane / lpp, lig = lane % lpp;

        float q[G_][8];
    #pragma unroll
        for (int h = 0; h < G_; ++h)
    #pragma unroll
            for (int j = 0; j < 8; ++j) q[h][j] = q_s[h * hd + lig * 8 + j];

        AttnAcc<G_> st;
    #pragma unroll
        for (int h = 0; h < G_; ++h) {
            st.m[h] = -INFINITY;
            st.l[h] = 0.f;
    #pragma unroll
            for (int j = 0; j < 8; ++j) st.a[h][j] = 0.f;
        }

        // ring chunks owned by this warp's slot.  `first` is the index (within the unit) of the first chunk this warp
        // consumes; the warp then takes every nslots-th chunk.  The partial results are merged in the order of `first`,
        // not of the physical warp, so the arithmetic does not depend on where in the ring the unit happens to start
        // (looped and per-layer launches then agree bit for bit).
        const uint32_t pb = attn_positions_per_chunk(p);
        for (uint32_t i = (warp < p.nslots ? first : u.nring); i < u.nring; i += p.nslots) {
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 1);
            mbar_wait(p, s, smem_u32(&s.full[warp]), wr.uses & 1u);
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 2);
            ++wr.uses;
            const uint8_t* kp = s.ring + (size_t)warp * SLOT_BYTES;
            const uint8_t* vp = kp + SLOT_BYTES / 2;
            const uint32_t np = min(pb, u.cend - (u.c0 + i * pb));
            constexpr int U = (G_ <= 4) ? 4 : 2;
            for (uint32_t base = 0; base < np; base += ppw * U) {
                uint4 kk[U], vv[U];
                bool ok[U];
    #pragma unroll
                for (int x = 0; x < U; ++x) {
                    const uint32_t t = base + x * ppw + grp;
                    ok[x] = t < np;
                    const uint32_t tt = ok[x] ? t : 0u;
                    kk[x] = *reinterpret_cast<const uint4*>(kp + ((size_t)tt * hd + lig * 8) * 2);
                    vv[x] = *reinterpret_cast<const uint4*>(vp + ((size_t)tt * hd + lig * 8) * 2);
                }
                attn_batch<G_, U>(st, q, kk, vv, ok, lpp);
            }
            __syncwarp();
            ring_issue_next(p, s, wr, warp, lane, pol);
            if (lane == 0) chunk_stamp(p, cta, rc.n0 + i, 3);
        }
        if (u.has_new && first == 0) {
            // the position written by this step: its K/V come from shared memory (already rounded to bf16)
            uint4 kk1[1], vv1[1];
            uint4& kk = kk1[0];
            uint4& vv = vv1[0];
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
            const bool ok1[1] = {grp == 0};
            attn_batch<G_, 1>(st, q, kk1, vv1, ok1, lpp);
        }

        // merge the position groups of the warp (lanes with equal lig)
        for (uint32_t o = lpp; o < 32; o <<= 1) {
    #pragma unroll
            for (int h = 0; h < G_; ++h) {
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
            for (int h = 0; h < G_; ++h) {
                float* dst = comb + ((size_t)first * G + h) * (hd + 2);
    #pragma unroll
                for (int j = 0; j < 8; ++j) dst[lig * 8 + j] = st.a[h][j];
                if (lig == 0) {
                    dst[hd] = st.m[h];
                    dst[hd + 1] = st.l[h];
                }
            }
        }
    }
    trace_stamp(p, cta, layer, 15, ctid);
    consumer_bar();

    // merge the warps; thread t owns (head, column)
    const uint32_t unit = u.bg * p.cps + u.ch;
    for (uint32_t t = ctid; t < G * hd; t += NCT) {
        const uint32_t h = t / hd, d = t % hd;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NCW; ++w) M = fmaxf(M, comb[((size_t)w * G + h) * (hd + 2) + hd]);
        float A = 0.f, Lsum = 0.f;
#pragma unroll
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
        const uint32_t old = atom_add_acq_rel(p.tickets + (size_t)layer * p.B * p.nkv + u.bg, 1u);
        *s.bcast = (old == nchunk - 1) ? 1 : 0;
    }
    consumer_bar();
    if (*s.bcast == 0) return;
    const uint32_t unit0 = u.bg * p.cps;
    for (uint32_t t = ctid; t < G * hd; t += NCT) {
        const uint32_t h = t / hd, d = t % hd;
        float Mx = -INFINITY;
#pragma unroll 8
        for (uint32_t c = 0; c < nchunk; ++c) Mx = fmaxf(Mx, __ldcg(p.part_ml + ((size_t)(unit0 + c) * G + h) * 2));
        float Ax = 0.f, Lx = 0.f;
#pragma unroll 8
        for (uint32_t c = 0; c < nchunk; ++c) {
            const size_t uu = (size_t)(unit0 + c) * G + h;
            const float sc = rescale(__ldcg(p.part_ml + uu * 2), Mx);
            Ax += __ldcg(p.part + uu * hd + d) * sc;
            Lx += __ldcg(p.part_ml + uu * 2 + 1) * sc;
        }
        p.o[(size_t)b * p.QD + (size_t)(g * G + h) * hd + d] = Ax / Lx;
    }
}

// Runs the attention stage and moves the ring cursor past the unit's chunks (also for CTAs without a unit).
template <int GT>
__device__ __forceinline__ void attention_stage_and_advance(const Params& p, const Smem& s, uint32_t layer, uint32_t cta,
                                                            uint32_t ctid, uint32_t warp, uint32_t lane, RingCursor& rc,
                                                            WarpRing& wr, uint64_t pol) {
    attention_stage<GT>(p, s, layer, cta, ctid, warp, lane, rc, wr, pol);
    rc.advance(attn_unit(p, cta).nring, p.nslots);
}

}  // namespace kl
