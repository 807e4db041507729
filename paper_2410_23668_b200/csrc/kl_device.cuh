// Device-side building blocks of the kernel-looped decoder: PTX wrappers (mbarrier, TMA bulk and tensor copies,
// tagged 64-bit words, one acquire/release counter), the shared-memory weight ring, the GEMV stage consumer and
// the split-K attention stage.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#ifndef KL_POLL_NS
#define KL_POLL_NS 64
#endif
#ifndef KL_T_OHEAD
#define KL_T_OHEAD 1   // stash mode: stream the head of W_o ahead of the K/V chunks (see t_o_head)
#endif
#ifndef KL_T_OHEAD_REGIONS
#define KL_T_OHEAD_REGIONS 8   // ... as many chunks per pipeline as it has TMEM regions (fewer measured slower: 6 -> +0.4 %, 4 -> +1 %)
#endif
#ifndef KL_ST_TW
#define KL_ST_TW "st.relaxed.gpu.global.b64"
#endif

namespace kl {

#ifndef KL_NCW
#define KL_NCW 10
#endif

constexpr int NCW = KL_NCW;                     // consumer warps per CTA; consumer c takes chunks c, c + NCW, ... and so
                                           // always meets the same nsw ring slots, in order
constexpr int NCT = NCW * 32;              // consumer threads (they take part in the CTA-wide steps)
constexpr int NTHREADS = NCT + 32;         // + the producer warp (the last warp; 7 warps leave 255 registers each)
constexpr int SLOT_BYTES = 16384;          // one ring slot = one chunk (one or two TMA copies)
constexpr int MAX_NSW = 24 / NCW;          // ring slots per consumer warp (the barrier arrays hold 24 slots)
constexpr int MAX_SLOTS = NCW * MAX_NSW;
constexpr int MAX_PIECES = 2 * NCW;            // chunks per unit when a unit spans several chunks
constexpr int UNIT_SLOTS = 8;             // in-flight multi-chunk units tracked per CTA
constexpr int MAX_RPC_SPLIT = 4;           // rows per unit when units are split into column pieces
constexpr int MIN_POS_PER_CHUNK = 64;      // attention: fewest cached positions worth a CTA
constexpr int MAX_G = 8;                   // query heads per KV head
constexpr int T_NCW = 8;                   // stash mode: consumer warps (two teams of four, one per TMEM lane quarter)
constexpr int T_NSP = 4;                   // stash mode: ring slots per pipeline (two pipelines, one per team)
constexpr int T_NREG = 8;                  // stash mode: TMEM regions (16 KB, 32 columns) per pipeline
constexpr int T_USLOTS = 16;               // stash mode: units of a team whose quarter sums may be in flight
constexpr int MAX_EXPERTS = 16;            // experts of a mixture-of-experts layer
constexpr int MAX_TOP_K = 4;               // experts per token
constexpr int SMEM_MISC_BYTES = 7168;  // barriers, reduction scratch, unit table, step context (see SmemT); a multiple of 1024

enum StageId { ST_QKV = 0, ST_ATTN = 1, ST_O = 2, ST_GU = 3, ST_D = 4, ST_LM = 5 };
enum EpilogueKind { EP_STORE = 0, EP_RESIDUAL = 1, EP_SWIGLU = 2 };
enum PlanId { PL_QKV = 0, PL_O = 1, PL_GU = 2, PL_D = 3, PL_LM = 4, PL_COUNT = 5 };

constexpr int ERR_SYNC_TIMEOUT = -5;
constexpr int ERR_OUT_OF_RANGE = -6;

// How one matrix [R, K] (bf16) is cut into ring chunks.  Rows are grouped into units of `rpc` consecutive rows,
// dealt to the CTAs in contiguous ranges.  A unit is streamed as `npieces` chunks; chunk j holds columns
// [j*kp, min(K, (j+1)*kp)) of the unit's rows, row after row.  kp <= MAX_KP so that a lane keeps its share of the
// matching slice of the input vector in registers for the whole stage, and rpc * kp * 2 <= SLOT_BYTES.
// The library's copy of the matrix is stored in exactly this order -- unit, then piece, then row, then column --
// so every chunk, and in fact the whole share of a CTA, is one linear run of bytes ("grouped tensors laid out
// linearly in memory", Section 3.2).  With npieces == 1 this is plain row-major.
struct GemvPlan {
    uint32_t R, K;
    uint32_t rpc;
    uint32_t kp;
    uint32_t npieces;
    uint32_t nunits;
    uint32_t nseg;      // mixture-of-experts down projection: the chosen experts' matrices side by side, K columns and
                        // npieces pieces EACH (1 everywhere else)
};
#ifndef KL_MAX_KP
#define KL_MAX_KP 1536
#endif
constexpr uint32_t MAX_KP = KL_MAX_KP;      // columns per chunk piece: blocks of 256, 8 per lane and block
constexpr int MAX_XB = MAX_KP / 256;

struct Params {
    CUtensorMap kv_map;    // the whole KV cache as a 2-D tensor [rows, head_dim], 128-byte swizzle (64-byte aligned)
    uint32_t attn_tc;      // 1: tensor-core attention loop fed by kv_map boxes; 0: CUDA-core loop fed by linear copies
    uint32_t L, H, nq, nkv, hd, F, V, G, QD, KVD, max_ctx, B;   // B: sequences in the KV cache of this step
    uint32_t b0;           // the sequence this launch decodes (batches run one sequence after another)
    uint32_t P;            // CTAs in the persistent grid
    uint32_t nslots;       // ways of the ring = consumer warps (chunk n belongs to consumer n % nslots)
    uint32_t nsw;          // slots per consumer (chunk n sits in slot (n % nslots) * nsw + (n / nslots) % nsw)
    uint32_t vec_floats;   // capacity of the shared input-vector area
    uint32_t cps;          // attention: CTA slots per (sequence, kv head)
    float eps;
    int32_t skip_stage;    // test hook: stage of layer 0 whose end is not signalled (-1 = none)
    uint32_t jitter_seed;  // test hook: != 0 makes every CTA sleep a pseudo-random time (below jitter_ns) when it enters a stage
    uint32_t jitter_ns;
    uint64_t wait_ns;
    uint64_t layer_stride; // elements between consecutive layers of any per-layer tensor
    const __nv_bfloat16* bqkv;   // biases of the q, k, v projections [L][QD + 2 KVD] (layer_stride apart), or null
    // mixture-of-experts layers (n_experts > 0): wgu / wd point at expert 0 of layer 0, the experts of a layer lie
    // expert_stride elements apart; wrouter [L][n_experts][H] (layer_stride apart)
    uint32_t n_experts, top_k;
    uint64_t expert_stride;
    const __nv_bfloat16* wrouter;
    GemvPlan plan[PL_COUNT];
    const __nv_bfloat16 *wqkv, *wo, *wgu, *wd, *g1, *g2, *gf, *wlm, *embed;
    __nv_bfloat16* kv;
    const int32_t* tokens;
    const int32_t* positions;
    // activations that cross CTAs.  xa, xb, qkv, o and the split-K partials are arrays of tagged words (see TW):
    // xa = hidden state entering a layer, xb = hidden state after the attention half.  h (the MLP's inner vector) is
    // plain fp32 guarded by a counter.
    struct TW *xa, *xb, *qkv, *o, *part, *part_ml;
    float *h, *rope_cs, *logits;
    uint32_t* step_dev;    // device word: sequences decoded on this handle so far (makes the tags of every launch
                           // distinct).  The embedding kernel increments it, so a captured step can be replayed.
    const double* inv_freq;
    uint32_t* counters;    // [L]: CTAs that have finished the gate/up stage of each layer
    int32_t* status;
    unsigned long long* trace;  // optional [P][L][TRACE_STAMPS] globaltimer stamps of consumer thread 0, or null
    unsigned long long* chunk_trace;  // optional [CHUNK_TRACE_ROWS][4] per-chunk stamps of CTA 0 (issue, wait, full, done)
    // the KV cache once more, as a 4-D tensor [64 columns][rows][head_dim / 64 column halves][K | V of the same (layer, sequence, head)]:
    // ONE copy brings the K and the V rows of a chunk, every 64-column half as a box of its own.  The producer thread
    // pays per instruction, and a unit at a long context is hundreds of chunks: units of more chunks than the ring has
    // slots take this form (context 65536: 236 against 221 tok/s), shorter ones -- whose chunks are all in flight at
    // once and whose last arrival is what the attention block waits for -- the four separate boxes, which land sooner.
    CUtensorMap kv_map4;
};
constexpr uint32_t CHUNK_TRACE_ROWS = 8192;

// What changes from one decoded token to the next: the step number the tags are built from, the position written by
// the step, and the rotary table of that position.  One copy per CTA in shared memory, written by one thread at the
// start of the launch (and behind every token of a launch that decodes several) and read between the stages.
struct StepCtx {
    uint32_t step;
    uint32_t pos;
    const float* rope_cs;
    uint64_t wait_ns;    // copies of the launch's wait limit and status word, for code that runs as a call
    int32_t* status;
};


// ------------------------------------------------------------------------------------------------ PTX

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

constexpr int TRACE_STAMPS = 16;
template <class SM>
__device__ __forceinline__ void chunk_stamp(const Params& p, const SM&, uint32_t cta, uint64_t n, int k) {
    if constexpr (SM::kTrace)
        if (p.chunk_trace != nullptr && cta == 0 && n < CHUNK_TRACE_ROWS) p.chunk_trace[n * 4 + k] = globaltimer_ns();
}
// Test hook of the synchronisation protocol (instantiations with the debug hooks only): every consumer thread of the
// CTA sleeps the same pseudo-random time, a function of (seed, CTA, step, layer, stage), before it enters a stage, so
// that the CTAs reach every exchange in a different order on every step.  Bounded: at most jitter_ns, in naps.
template <class SM>
__device__ __forceinline__ void stage_jitter(const Params& p, const SM&, uint32_t cta, uint32_t step, uint32_t layer, uint32_t st) {
    if constexpr (SM::kTrace) {
        if (p.jitter_seed != 0u) {
            uint32_t h = p.jitter_seed ^ (cta * 0x9E3779B1u) ^ (step * 0x85EBCA77u) ^ ((layer * 8u + st) * 0xC2B2AE3Du);
            h ^= h >> 15; h *= 0x2C1B3C6Du; h ^= h >> 12; h *= 0x297A2D39u; h ^= h >> 15;
            uint32_t ns = (uint32_t)(((uint64_t)h * p.jitter_ns) >> 32);
            while (ns > 0u) {
                const uint32_t nap = ns < 1000u ? ns : 1000u;
                __nanosleep(nap);
                ns -= nap;
            }
        }
    }
}
template <class SM>
__device__ __forceinline__ void trace_stamp(const Params& p, const SM&, uint32_t cta, uint32_t layer, int k, uint32_t ctid) {
    if constexpr (SM::kTrace)
        if (p.trace != nullptr && ctid == 0 && layer < p.L) p.trace[((size_t)cta * p.L + layer) * TRACE_STAMPS + k] = globaltimer_ns();
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
// A value that crosses CTAs travels with its own flag: one aligned 8-byte word {fp32 value, 32-bit tag}, written
// with a single 64-bit store and read with 64-bit (or 2 x 64-bit) loads that bypass L1.  A reader that sees the
// tag it expects has the value -- no fence on the writer's side, no counter to poll, one L2 round trip on the
// reader's side.  Tags are odd numbers built from (decode step, layer, stage), so a word left over from an earlier
// layer or step never matches, and neither does zero-initialised memory.
// ---- stash mode: tensor memory as a second stage of the weight ring (tcgen05.cp from shared memory, tcgen05.ld into
// registers).  One allocation of all 512 columns per CTA, made and released by one warp.
__device__ __forceinline__ void tm_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tm_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tm_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tm_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tm_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 128 lanes x 32 bytes: lane r takes the two 16-byte granules at start + 16 r and start + 16 r + 2048 (descriptor
// without swizzle: 16 bytes between consecutive rows of a group of eight, 128 bytes between groups, 2048 bytes
// between the two granules of a row), i.e. a linear run of 4 KB lands as granule (r + 128 k) in lane r, columns 4 k .. 4 k + 3
__device__ __forceinline__ void tm_cp_4k(uint32_t taddr, uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(2048u >> 4) << 16;
    d |= (uint64_t)(128u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(d) : "memory");
}
__device__ __forceinline__ void tm_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, "
        "%25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tm_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tm_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

struct __align__(8) TW {
    float v;
    uint32_t tag;
};
// Every tagged word is moved by one 64-bit access (value in the low half, tag in the high half): a single aligned
// 64-bit access is never torn, so the tag cannot be seen without its value.  The accesses are strong (relaxed at gpu
// scope): a weak load inside a polling loop may legally be hoisted out of it by the assembler.
__device__ __forceinline__ void st_tw(TW* p, float v, uint32_t tag) {
    const uint64_t w = ((uint64_t)tag << 32) | __float_as_uint(v);
    asm volatile(KL_ST_TW " [%0], %1;" ::"l"(p), "l"(w) : "memory");
}
__device__ __forceinline__ TW ld_tw(const TW* p) {
    uint64_t r;
    asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(r) : "l"(p) : "memory");
    TW w;
    w.v = __uint_as_float((uint32_t)r);
    w.tag = (uint32_t)(r >> 32);
    return w;
}
// two consecutive words (16-byte aligned): x, y = value and tag of the first, z, w of the second
__device__ __forceinline__ uint4 ld_tw2(const TW* p) {
    uint64_t a, b;
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
    return make_uint4((uint32_t)a, (uint32_t)(a >> 32), (uint32_t)b, (uint32_t)(b >> 32));
}
enum TagSlot { TG_XA = 0, TG_QKV = 1, TG_PART = 2, TG_O = 3, TG_XB = 4 };
__device__ __forceinline__ uint32_t tag_from(uint32_t step, uint32_t L, uint32_t layer, uint32_t slot) {
    return ((((step * L + layer) << 3) + slot) << 1) | 1u;
}
__device__ __forceinline__ uint32_t tag_of(const Params& p, const StepCtx& cx, uint32_t layer, uint32_t slot) {
    return tag_from(cx.step, p.L, layer, slot);
}
// The step word as a launch finds it.  The launch that writes it (the last CTA of a sampling kernel, behind every
// reader's last stage) may still have readers of this load in flight when a bounded wait gave up, so the load is a
// strong one, not a read-only one.
__device__ __forceinline__ uint32_t ld_step(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ StepCtx step_ctx(const Params& p) {
    StepCtx cx;
    cx.step = ld_step(p.step_dev);
    cx.pos = (uint32_t)p.positions[p.b0];
    cx.rope_cs = p.rope_cs;
    return cx;
}

template <class SM>
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(SM::NCT) : "memory"); }

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
// d0 += a0 * b0, d1 += a1 * b1 as ONE instruction (packed fp32 multiply-add of sm_100): the even and the odd columns
// of a weight register are the two halves of the pair, so the multiply-adds of a chunk take half the issue slots.
__device__ __forceinline__ void ffma2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb, rc;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rc;\n\t}"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

// ------------------------------------------------------------------------------------------------ shared state

// Dynamic shared memory of the persistent kernels, at fixed offsets from its start, so that no thread holds a pointer
// to any part of it in a register: barriers and small tables first (SMEM_MISC_BYTES, a multiple of 1024), then the
// ring (slots on 1024-byte boundaries, as the swizzled K/V boxes need), then the vector area.
//   full  [MAX_SLOTS] copy landed                       empty [MAX_SLOTS] consumer has finished reading
//   red   [NCW] reduction scratch                       unit_part [UNIT_SLOTS][MAX_PIECES][MAX_RPC_SPLIT]
//   unit_cnt [UNIT_SLOTS], abort flag                   ctx  step number, position and rotary table (see StepCtx)
//   ring  nslots * nsw * SLOT_BYTES                     vec  input vector of the current GEMV stage (lane-permuted),
//                                                            or the attention workspace
// TR selects the instantiation with the trace stamps compiled in (kl_set_trace); the production kernels carry none.
extern __shared__ __align__(1024) uint8_t kl_smem[];
// What the router of a mixture-of-experts layer chose, for the producer thread and the consumer warps of this CTA.
struct MoeSel {
    volatile uint32_t seq;          // layers routed so far in this launch (written last)
    uint32_t e[MAX_TOP_K];          // the chosen experts, in descending order of their logits
    float w[MAX_TOP_K];             // and their gate weights
};
template <bool TR, bool MOE = false, int TM = 0, bool CC = true>
struct SmemT {
    static constexpr bool kTrace = TR;
    static constexpr bool kMoe = MOE;
    // CC: the CUDA-core attention loops are compiled in.  Launches that run the tensor-core loop take kernels without
    // them: code a launch never runs costs time by being there (3.5 % of a token on the 8B shape).  The stash-mode
    // kernels never carry them.
    static constexpr bool kCudaCoreAttn = CC && TM == 0;
    static constexpr bool kTmem = TM != 0;       // stash mode: weights go ring -> TMEM -> registers (see the stash section)
    // TM == 1: the stage exists for chunks of 2048 and 4096 columns only; TM == 2: for 1024 and 3072 as well.  Two kernels,
    // because the code the common shapes never run costs them time by lying between the code they do run
    // (measured: 3.04 against 2.97 ms per token on the 8B shape).
    static constexpr bool kAllWidths = TM == 2;
    static constexpr int NCW = TM ? T_NCW : kl::NCW;   // consumer warps
    static constexpr int NCT = NCW * 32;               // consumer threads (they take part in the CTA-wide steps)
    __device__ __forceinline__ static MoeSel* moe() { return reinterpret_cast<MoeSel*>(kl_smem + 6240); }
    __device__ __forceinline__ static uint64_t* full() { return reinterpret_cast<uint64_t*>(kl_smem); }
    __device__ __forceinline__ static uint64_t* empty() { return reinterpret_cast<uint64_t*>(kl_smem + 256); }
    // stash mode: per TMEM region "copy complete" / "all four warps have read it", the drain barriers of the two stash
    // threads, the TMEM base address, the arrival counters of the units whose quarter sums meet in unit_part()
    __device__ __forceinline__ static uint64_t* tfull() { return reinterpret_cast<uint64_t*>(kl_smem + 512); }
    __device__ __forceinline__ static uint64_t* tfree() { return reinterpret_cast<uint64_t*>(kl_smem + 640); }
    __device__ __forceinline__ static uint64_t* tdone() { return reinterpret_cast<uint64_t*>(kl_smem + 768); }
    __device__ __forceinline__ static uint32_t* tbase() { return reinterpret_cast<uint32_t*>(kl_smem + 784); }
    // stash mode: "the K/V chunk in this slot has landed", signalled by the stash thread, which sees every use of a slot
    // land in order (a reader that tested the slot's own barrier could be two phases behind: the uses before its chunk
    // are weight chunks it never waits for)
    __device__ __forceinline__ static uint64_t* kvready() { return reinterpret_cast<uint64_t*>(kl_smem + 800); }
    // the barrier a reader of K/V chunks in ring slot `slot` waits on
    __device__ __forceinline__ static uint64_t* kv_bar(uint32_t slot) { return ((TM != 0 && KL_T_OHEAD) ? kvready() : full()) + slot; }
    __device__ __forceinline__ static int* t_ucnt() { return reinterpret_cast<int*>(kl_smem + 1024); }
    __device__ __forceinline__ static float* red() { return reinterpret_cast<float*>(kl_smem + 1536); }
    __device__ __forceinline__ static float* unit_part() { return reinterpret_cast<float*>(kl_smem + 2048); }
    __device__ __forceinline__ static int* unit_cnt() { return reinterpret_cast<int*>(kl_smem + 6144); }
    __device__ __forceinline__ static volatile int* abort_flag() { return reinterpret_cast<volatile int*>(kl_smem + 6144 + 4 * UNIT_SLOTS); }
    __device__ __forceinline__ static StepCtx* ctx() { return reinterpret_cast<StepCtx*>(kl_smem + 6208); }
    __device__ __forceinline__ static uint8_t* ring() { return kl_smem + SMEM_MISC_BYTES; }
    // stash mode: the ring is always 2 * T_NSP slots
    __device__ __forceinline__ static float* vec_t() {
        return reinterpret_cast<float*>(kl_smem + SMEM_MISC_BYTES + (size_t)2 * T_NSP * SLOT_BYTES);
    }
    __device__ __forceinline__ static float* vec(const Params& p) {
        return reinterpret_cast<float*>(kl_smem + SMEM_MISC_BYTES + (size_t)p.nslots * p.nsw * SLOT_BYTES);
    }
};

// Records the first error and tells every waiter of this CTA to give up.  After an abort every wait returns at
// once but the control flow (stage order, CTA barriers) is unchanged, so no warp is left behind at a barrier; the
// step's outputs are then meaningless and the status word says so.
template <class SM>
__device__ __noinline__ bool raise_abort(const Params& p, const SM& s, int code, int where = 0) {
    bool first = false;
    if (atomicCAS(p.status, 0, code) == 0) {   // following words: which wait gave up, where (diagnostics)
        p.status[1] = where;
        p.status[2] = (int)blockIdx.x;
        p.status[3] = (int)threadIdx.x;
        first = true;
    }
    *s.abort_flag() = 1;
    return first;
}

// Bounded mbarrier wait.  Returns false when the wait was abandoned (limit reached or abort raised elsewhere).
template <class SM>
__device__ __forceinline__ bool mbar_wait(const Params& p, const SM& s, uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*s.abort_flag()) return false;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*s.abort_flag()) return false;
            if (globaltimer_ns() - t0 > p.wait_ns) {
                raise_abort(p, s, ERR_SYNC_TIMEOUT, 500);   // out of line: it runs once, if ever
                return false;
            }
        }
    }
    return true;
}

// Bookkeeping of a bounded polling loop on tagged words or counters.  poll_continue() returns false when the loop
// must be abandoned: another waiter of the CTA gave up, a kernel of this step flagged an error, or the limit ran out.
struct PollGuard {
    uint64_t t0;
    uint32_t it;
    int where;
};
template <class SM>
__device__ __forceinline__ bool poll_continue(const Params& p, const SM& s, PollGuard& g) {
    if (g.it == 0) g.t0 = globaltimer_ns();
    // a nap keeps the polling traffic of a waiting CTA off the L2 ports the late CTAs still need; in stash mode, where the
    // weight stream runs through every exchange anyway, it only delays the waiter (2.833 against 2.845 ms per token)
    if (KL_POLL_NS && !SM::kTmem) __nanosleep(KL_POLL_NS);
    if ((++g.it & 7u) == 0) {
        if (*s.abort_flag()) return false;
        if (__ldcg(p.status) != 0) {
            *s.abort_flag() = 1;
            return false;
        }
        if (globaltimer_ns() - g.t0 > p.wait_ns) {
            raise_abort(p, s, ERR_SYNC_TIMEOUT, g.where);
            return false;
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

// Stash mode streams the first units of the output projection BEFORE the K/V chunks of the attention unit: K/V chunks
// stay in their ring slots until the attention stage reads them, and whatever is queued behind them waits; the head of
// W_o moves on into tensor memory while the QKV stage still runs, so the copies do not stop there.  At most eight
// chunks per pipeline -- what its TMEM regions hold -- or the K/V chunks behind them could never be requested.
__device__ __forceinline__ uint32_t t_o_head(const GemvPlan& pl, uint32_t nu) {
    if (!KL_T_OHEAD) return 0u;
    const uint32_t h = 2u * ((uint32_t)(KL_T_OHEAD_REGIONS) / pl.npieces);
    return nu < h ? nu : h;
}
struct ChunkGeom {
    uint32_t unit;      // unit index (matrix-wide)
    uint32_t piece;     // column piece
    uint32_t row;       // first row of the unit
    uint32_t nrows;     // rows in the chunk
    uint32_t kofs;      // first column
    uint32_t klen;      // columns (row pitch inside the slot = klen * 2 bytes)
};
template <bool MOE = false>
__device__ __forceinline__ ChunkGeom chunk_geom(const GemvPlan& pl, uint32_t u0, uint32_t i) {
    ChunkGeom g;
    const uint32_t tp = MOE ? pl.npieces * pl.nseg : pl.npieces;
    if (tp == 1) {
        g.unit = u0 + i;
        g.piece = 0;
    } else {
        g.unit = u0 + i / tp;
        g.piece = i % tp;
    }
    g.row = g.unit * pl.rpc;
    g.nrows = min(pl.rpc, pl.R - g.row);
    if (MOE && pl.nseg > 1) {   // piece j of segment sg: columns sg * K + j * kp ... of the concatenated input vector
        const uint32_t sg = g.piece / pl.npieces, j = g.piece % pl.npieces;
        g.kofs = sg * pl.K + j * pl.kp;
        g.klen = min(pl.kp, pl.K - j * pl.kp);
    } else {
        g.kofs = g.piece * pl.kp;
        g.klen = min(pl.kp, pl.K - g.kofs);
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
__device__ __forceinline__ AttnUnit attn_unit(const Params& p, uint32_t cta, uint32_t pos) {
    AttnUnit u;
    u.active = false;
    u.nring = 0;
    u.bg = cta / p.cps;
    u.ch = cta % p.cps;
    if (u.bg >= p.nkv) return u;
    u.b = p.b0;
    u.g = u.bg;
    u.pos = pos;
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

__device__ __forceinline__ void tma_tensor_2d_g2s(uint32_t dst, const void* tmap, int32_t x, int32_t y, uint32_t bar,
                                                  uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ void tma_tensor_4d_g2s(uint32_t dst, const void* tmap, int32_t x, int32_t y, int32_t z, int32_t w,
                                                  uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar), "l"(pol)
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

// ------------------------------------------------------------------------------------------------ the ring
//
// The whole launch is one sequence of chunks per CTA, in consumption order: for every layer the CTA's QKV rows, the
// K/V rows of its attention unit, its O rows, gate/up rows and down rows.  Every address is known when the kernel
// starts (weights are grouped per layer and linear in memory; cached K/V rows were written by earlier launches),
// so the producer thread runs ahead of the consumers across stage boundaries and, in the looped kernel, across
// layer boundaries: while the consumers sit in the counter wait that replaces a kernel boundary, the copies of the
// next stage's (next layer's) chunks are already in flight.
//
// Chunk n goes to consumer n % nslots, into that consumer's slot (n / nslots) % nsw.  Each slot therefore sees its
// uses in order on both sides, and every parity wait is made by the one warp that will read the data (a fast warp
// can never test a barrier two phases behind).

// Consumer side of the ring: which of its nsw slots the warp reads next and with which barrier phase.
struct WarpRing {
    uint32_t cslot;         // slot (0..nsw-1) the next chunk is consumed from
    uint32_t cphase;        // barrier phase of that slot to wait for
    uint32_t rslot;         // slot consumed last (the one to release)
};
// The warp takes a chunk from its current slot and moves to the next one (call after the wait).
__device__ __forceinline__ void ring_advance_consume(const Params& p, WarpRing& r) {
    r.rslot = r.cslot;
    if (++r.cslot == p.nsw) {
        r.cslot = 0;
        r.cphase ^= 1u;
    }
}
// The whole warp has finished reading the slot it consumed last (call after __syncwarp): hand it back.
template <class SM>
__device__ __forceinline__ void ring_release(const Params& p, const SM& s, const WarpRing& r, uint32_t warp, uint32_t lane) {
    if (lane == 0) mbar_arrive(smem_u32(&s.empty()[warp * p.nsw + r.rslot]));
}
__device__ __forceinline__ WarpRing ring_begin() {
    WarpRing r;
    r.cslot = 0;
    r.cphase = 0;
    r.rslot = 0;
    return r;
}

// Producer state: where the next chunk goes.
struct RingProd {
    uint32_t c, k, use, n;   // consumer, slot of that consumer, use count of that slot, chunk index (for the log)
    uint64_t pol;
    bool aborted;
    // stash mode: the chunk sequence is dealt to two pipelines (team 0 / team 1 of the consumer warps), each with
    // T_NSP ring slots and T_NREG TMEM regions of its own.  The producer thread and the two stash threads walk the same
    // sequence: role 0 issues the copies, role 1 + t moves the chunks of pipeline t from the ring into TMEM.
    uint32_t role, pi;       // role of this thread; pipeline of the next chunk
    uint32_t uc;             // units of all stages so far (unit k of a stage goes to pipeline (uc + k) & 1)
    uint32_t tc[2];          // chunks so far per pipeline
    uint32_t tg;             // stash thread: weight chunks of its pipeline so far
};
__device__ __forceinline__ RingProd ring_prod_begin(uint32_t role) {
    RingProd r;
    r.c = r.k = r.use = r.n = 0u;
    r.pol = l2_policy_evict_first();
    r.aborted = false;
    r.role = role;
    r.pi = r.uc = r.tg = 0u;
    r.tc[0] = r.tc[1] = 0u;
    return r;
}
// Stash mode, the stash thread's part in a chunk of its pipeline.  A weight chunk: wait for the copy, wait for the
// TMEM region, move the slot's 16 KB into it (four copies of 4 KB), let the completion of the copies signal the region
// full and the slot empty.  A chunk of K/V rows is read from the ring by a consumer warp: the stash thread only sees it
// land.  Every slot's barrier completes a phase on two arrivals -- the stash thread's and the reader's (for a weight
// chunk both are the stash thread's) -- so neither side can fall two phases behind on a parity wait.
template <class SM>
__device__ __forceinline__ void stash_chunk(const Params& p, const SM& s, RingProd& r, bool weights) {
    const uint32_t pi = r.role - 1u, seq = r.tc[0]++;   // a stash thread only counts the chunks of its own pipeline
    if (r.aborted) return;
    const uint32_t slot = pi * T_NSP + seq % T_NSP;
    if (!mbar_wait(p, s, smem_u32(&s.full()[slot]), (seq / T_NSP) & 1u)) {
        r.aborted = true;
        return;
    }
    const uint32_t ebar = smem_u32(&s.empty()[slot]);
    if (weights) {
        const uint32_t g = r.tg++, reg = pi * T_NREG + g % T_NREG;
        if (g >= (uint32_t)T_NREG && !mbar_wait(p, s, smem_u32(&s.tfree()[reg]), ((g / T_NREG) - 1u) & 1u)) {
            r.aborted = true;
            return;
        }
        tm_fence_after();
        const uint32_t src = smem_u32(s.ring()) + slot * SLOT_BYTES, dst = *s.tbase() + reg * 32u;
#pragma unroll
        for (uint32_t i = 0; i < 4; ++i) tm_cp_4k(dst + i * 8u, src + i * 4096u);
        tm_commit(smem_u32(&s.tfull()[reg]));
        tm_commit(ebar);
    } else {
        mbar_arrive(smem_u32(&s.kvready()[slot]));
    }
    mbar_arrive(ebar);
}
// The stash thread is done: no copy into TMEM may be in flight when the allocation is released.
template <class SM>
__device__ __forceinline__ void stash_drain(const Params& p, const SM& s, const RingProd& r) {
    const uint32_t bar = smem_u32(&s.tdone()[r.role - 1u]);
    tm_commit(bar);
    const uint64_t t0 = globaltimer_ns();
    while (!mbar_try_wait(bar, 0u)) {
        if (globaltimer_ns() - t0 > p.wait_ns) return;
    }
}
// Slot and use count of the next chunk, and the step to the one after it.
template <class SM>
__device__ __forceinline__ void prod_slot(const Params& p, const RingProd& r, uint32_t& slot, uint32_t& use) {
    if constexpr (SM::kTmem) {
        slot = r.pi * T_NSP + r.tc[r.pi] % T_NSP;
        use = r.tc[r.pi] / T_NSP;
    } else {
        slot = r.c * p.nsw + r.k;
        use = r.use;
    }
}
template <class SM>
__device__ __forceinline__ void prod_advance(const Params& p, RingProd& r) {
    ++r.n;
    if constexpr (SM::kTmem) {
        ++r.tc[r.pi];
    } else {
        if (++r.c == p.nslots) {
            r.c = 0;
            if (++r.k == p.nsw) {
                r.k = 0;
                ++r.use;
            }
        }
    }
}

// Waits for the slot of the next chunk, arms its barrier and starts one or two linear copies into it.
template <class SM>
__device__ __forceinline__ void prod_issue(const Params& p, const SM& s, RingProd& r, const uint8_t* src0, uint32_t bytes0,
                                           const uint8_t* src1, uint32_t bytes1, uint32_t dst1) {
    if (r.aborted) return;
    uint32_t slot, use;
    prod_slot<SM>(p, r, slot, use);
    if (use > 0 && !mbar_wait(p, s, smem_u32(&s.empty()[slot]), (use - 1u) & 1u)) {
        r.aborted = true;
        return;
    }
    const uint32_t bar = smem_u32(&s.full()[slot]);
    const uint32_t dst = smem_u32(s.ring()) + slot * SLOT_BYTES;
    chunk_stamp(p, s, blockIdx.x, r.n, 0);
    mbar_arrive_expect_tx(bar, bytes0 + bytes1);
    tma_bulk_g2s(dst, src0, bytes0, bar, r.pol);
    if (bytes1) tma_bulk_g2s(dst + dst1, src1, bytes1, bar, r.pol);
    prod_advance<SM>(p, r);
}
// Same for a chunk of K/V rows as swizzled boxes of the cache tensor: [pb rows] x [64 columns] per box, K boxes in
// the first half of the slot, V boxes in the second, written by one copy each or all of them by one copy (the boxes
// are the outer dimensions of the 4-D tensor map); a box is always written whole (rows outside the chunk's own
// positions are ignored by the consumer).  yk, yv: cache rows of the first row of the K and of the V boxes.
template <class SM>
__device__ __forceinline__ void prod_issue_boxes(const Params& p, const SM& s, RingProd& r, int32_t yk, int32_t yv, bool one_copy) {
    if (r.aborted) return;
    uint32_t slot, use;
    prod_slot<SM>(p, r, slot, use);
    if (use > 0 && !mbar_wait(p, s, smem_u32(&s.empty()[slot]), (use - 1u) & 1u)) {
        r.aborted = true;
        return;
    }
    const uint32_t bar = smem_u32(&s.full()[slot]);
    const uint32_t dst = smem_u32(s.ring()) + slot * SLOT_BYTES;
    chunk_stamp(p, s, blockIdx.x, r.n, 0);
    mbar_arrive_expect_tx(bar, (uint32_t)SLOT_BYTES);
    if (one_copy) {
        tma_tensor_4d_g2s(dst, &p.kv_map4, 0, yk, 0, 0, bar, r.pol);
    } else {
        const uint32_t box_bytes = SLOT_BYTES / 2 / (p.hd / 64u);
        for (uint32_t bx = 0; bx < p.hd / 64u; ++bx) {
            tma_tensor_2d_g2s(dst + bx * box_bytes, &p.kv_map, (int32_t)(bx * 64u), yk, bar, r.pol);
            tma_tensor_2d_g2s(dst + SLOT_BYTES / 2 + bx * box_bytes, &p.kv_map, (int32_t)(bx * 64u), yv, bar, r.pol);
        }
    }
    prod_advance<SM>(p, r);
}

// Streams this CTA's share of one matrix (units [u0, u1) of the plan): one linear run of bytes cut into chunks,
// per chunk only pointer increments.
template <class SM>
__device__ __forceinline__ void produce_matrix(const Params& p, const SM& s, RingProd& r, const GemvPlan& pl,
                                               const __nv_bfloat16* base, uint32_t cta, uint32_t kb = 0u, uint32_t ke = 0xffffffffu) {
    // units [kb, ke) of the CTA's share (stash mode streams a matrix in two parts where it pays)
    CtaRange cr = cta_units(pl, cta, p.P);
    const uint32_t nu = cr.u1 - cr.u0;
    const bool last = ke == 0xffffffffu;   // the call that ends the matrix moves the unit count on
    if (ke > nu) ke = nu;
    if (kb > ke) kb = ke;
    if constexpr (SM::kTmem) {
        if (r.role) {   // stash thread: the chunks of the units of its pipeline, nothing else
            for (uint32_t k = kb + ((((r.uc + kb) & 1u) == r.role - 1u) ? 0u : 1u); k < ke; k += 2)
                for (uint32_t j = 0; j < pl.npieces; ++j) stash_chunk(p, s, r, true);
            if (last) r.uc += nu;
            return;
        }
    }
    const uint32_t ubase = cr.u0;
    cr.u1 = cr.u0 + ke;
    cr.u0 += kb;
    const uint8_t* ptr = reinterpret_cast<const uint8_t*>(base) + (size_t)cr.u0 * pl.rpc * pl.K * 2u;
    const uint32_t last_len = pl.K - (pl.npieces - 1) * pl.kp;
    for (uint32_t u = cr.u0; u < cr.u1; ++u) {
        const uint32_t rows = min(pl.rpc, pl.R - u * pl.rpc);   // only the matrix's last unit can be short
        if constexpr (SM::kTmem) r.pi = (r.uc + (u - ubase)) & 1u;
        for (uint32_t j = 0; j < pl.npieces; ++j) {
            const uint32_t bytes = rows * ((j == pl.npieces - 1) ? last_len : pl.kp) * 2u;
            prod_issue(p, s, r, ptr, bytes, nullptr, 0u, 0u);
            ptr += bytes;
        }
    }
    if constexpr (SM::kTmem) {
        if (last) r.uc += nu;
    }
}

// Streams the cached K/V rows of this CTA's attention unit for one layer.
template <class SM>
__device__ __forceinline__ void produce_attention(const Params& p, const SM& s, RingProd& r, const AttnUnit& u,
                                                  uint32_t layer) {
    if (!u.active) return;
    if constexpr (SM::kTmem) {
        if (r.role) {   // stash thread: chunk i of the unit belongs to pipeline i & 1
            for (uint32_t i = r.role - 1u; i < u.nring; i += 2) stash_chunk(p, s, r, false);
            return;
        }
    }
    const uint32_t pb = attn_positions_per_chunk(p);
    if (p.attn_tc) {
        const uint32_t vdelta = p.B * p.nkv * p.max_ctx;
        const uint32_t row0 = layer * 2u * vdelta + (u.b * p.nkv + u.g) * p.max_ctx;
        for (uint32_t i = 0; i < u.nring; ++i) {
            const AttnWindow w = attn_window(u.c0, u.cend, pb, i);
            if constexpr (SM::kTmem) r.pi = i & 1u;
            prod_issue_boxes(p, s, r, (int32_t)(row0 + w.w0), (int32_t)(row0 + w.w0 + vdelta), u.nring > p.nslots);
        }
    } else {
        const uint32_t row_bytes = p.hd * 2u;
        const uint8_t* ks = reinterpret_cast<const uint8_t*>(kv_head(p, layer, 0, u.b, u.g)) + (size_t)u.c0 * row_bytes;
        const uint8_t* vs = reinterpret_cast<const uint8_t*>(kv_head(p, layer, 1, u.b, u.g)) + (size_t)u.c0 * row_bytes;
        uint32_t left = u.cend - u.c0;
        for (uint32_t i = 0; i < u.nring; ++i) {
            const uint32_t np = left < pb ? left : pb;
            if constexpr (SM::kTmem) r.pi = i & 1u;
            prod_issue(p, s, r, ks, np * row_bytes, vs, np * row_bytes, SLOT_BYTES / 2);
            ks += np * row_bytes;
            vs += np * row_bytes;
            left -= np;
        }
    }
}

// After an abandoned run no bulk copy may still be writing this CTA's shared memory when it exits: wait (bounded)
// for the last copy armed on every slot.
template <class SM>
__device__ __forceinline__ void produce_drain(const Params& p, const SM& s, const RingProd& r) {
    if constexpr (SM::kTmem) {
        if (r.role) {
            stash_drain(p, s, r);
            return;
        }
    }
    if (!r.aborted) return;
    const uint64_t t0 = globaltimer_ns();
    if constexpr (SM::kTmem) {
        for (uint32_t pi = 0; pi < 2; ++pi)
            for (uint32_t kk = 0; kk < (uint32_t)T_NSP; ++kk) {
                const uint32_t cnt = (r.tc[pi] + T_NSP - 1u - kk) / T_NSP;   // uses of this slot so far
                if (cnt == 0) continue;
                const uint32_t bar = smem_u32(&s.full()[pi * T_NSP + kk]);
                while (!mbar_try_wait(bar, (cnt - 1u) & 1u)) {
                    if (globaltimer_ns() - t0 > p.wait_ns) return;
                }
            }
    } else {
        for (uint32_t cc = 0; cc < p.nslots; ++cc) {
            for (uint32_t kk = 0; kk < p.nsw; ++kk) {
                const uint32_t cnt = r.use + ((kk < r.k || (kk == r.k && cc < r.c)) ? 1u : 0u);  // uses of this slot so far
                if (cnt == 0) continue;
                const uint32_t bar = smem_u32(&s.full()[cc * p.nsw + kk]);
                while (!mbar_try_wait(bar, (cnt - 1u) & 1u)) {
                    if (globaltimer_ns() - t0 > p.wait_ns) return;
                }
            }
        }
    }
}

// The producer thread of the decoder kernel: layers [l0, l1).
template <class SM>
__device__ __forceinline__ void produce_decoder(const Params& p, const SM& s, uint32_t cta, uint32_t l0, uint32_t l1,
                                                uint32_t sbeg, uint32_t send, uint32_t role = 0u) {
    RingProd r = ring_prod_begin(role);
    const AttnUnit u = attn_unit(p, cta, (uint32_t)p.positions[p.b0]);
    uint32_t routed = 0, ex[MAX_TOP_K] = {0u, 0u, 0u, 0u};   // mixture of experts: layers routed so far, the chosen experts
    // stash mode, launches that hold both the attention and the O stage: the head of W_o goes ahead of the K/V chunks
    uint32_t ohead = 0u;
    if constexpr (SM::kTmem) {
        if (sbeg <= ST_ATTN && send > ST_O) {
            const CtaRange co = cta_units(p.plan[PL_O], cta, p.P);
            ohead = t_o_head(p.plan[PL_O], co.u1 - co.u0);
        }
    }
    for (uint32_t l = l0; l < l1 && !r.aborted; ++l) {
        const size_t lo = (size_t)l * p.layer_stride;
        for (uint32_t st = sbeg; st < send; ++st) {
            if (st == ST_QKV) produce_matrix(p, s, r, p.plan[PL_QKV], p.wqkv + lo, cta);
            else if (st == ST_ATTN) {
                if (ohead) produce_matrix(p, s, r, p.plan[PL_O], p.wo + lo, cta, 0u, ohead);
                produce_attention(p, s, r, u, l);
            } else if (st == ST_O) produce_matrix(p, s, r, p.plan[PL_O], p.wo + lo, cta, ohead);
            else if (SM::kMoe) {
                if (st == ST_GU && !moe_wait_route(p, s, ++routed, ex)) r.aborted = true;   // the experts of this layer are known now
                if (!r.aborted) produce_matrix_moe(p, s, r, p.plan[st == ST_GU ? PL_GU : PL_D], (st == ST_GU ? p.wgu : p.wd) + lo, cta, ex, st != ST_GU);
            }
            else if (st == ST_GU) produce_matrix(p, s, r, p.plan[PL_GU], p.wgu + lo, cta);
            else produce_matrix(p, s, r, p.plan[PL_D], p.wd + lo, cta);
        }
    }
    produce_drain(p, s, r);
}
// ... and of the classifier kernel.
template <class SM>
__device__ __forceinline__ void produce_classifier(const Params& p, const SM& s, uint32_t cta, uint32_t role = 0u) {
    RingProd r = ring_prod_begin(role);
    produce_matrix(p, s, r, p.plan[PL_LM], p.wlm, cta);
    produce_drain(p, s, r);
}

// ------------------------------------------------------------------------------------------------ consumers

// Position of element e of the input vector in shared memory.  Within each block of 256 elements the eight
// elements a lane multiplies are split into two float4 groups stored 128 floats apart, so that both float4 loads
// of a warp are bank-conflict free.
__device__ __forceinline__ uint32_t vec_perm(uint32_t e) {
    return (e & ~255u) + (((e >> 2) & 1u) << 7) + (((e >> 3) & 31u) << 2) + (e & 3u);
}

// Loads the tagged vector src[0..n) (produced by other CTAs) into the shared vector area, polling until every word
// carries `tag`.  With `norm` the values are multiplied by the bf16 gains on the way in and the function returns
// rsqrt(mean(x^2) + eps): RMSNorm's normaliser is one number for the whole vector, so the stage applies it to its
// outputs instead of to its 4096 inputs (one pass and one barrier less).  Every CTA recomputes it; the summation
// order is fixed.  Without `norm` the function returns 1.  This poll is what replaces the grid-wide barrier of a kernel boundary: the first read that finds
// all tags in place already holds the data.
template <class SM>
__device__ __noinline__ float load_vec(const Params& p, const SM& s, const TW* src, uint32_t n, uint32_t tag, bool norm,
                                          const __nv_bfloat16* gain, uint32_t ctid) {
    constexpr int NB = 4;  // groups of four values kept in flight per thread (two 16-byte loads each)
    // The vector area is about to be overwritten: every warp of the CTA must be done with what the previous stage
    // kept there (the stage's input vector, read block by block until a warp's last chunk; the attention workspace).
    consumer_bar<SM>();
    float ss = 0.f;
    for (uint32_t base = 0; base < n; base += NB * SM::NCT * 4) {
        float4 v[NB];
        uint2 gk[NB];
        // Only the groups whose tags are not all in place yet are read again: the words that are late come from the
        // few CTAs that finish the previous stage last, and re-reading the whole vector from every waiting CTA
        // floods the L2 slices those late CTAs stream their weights through.
        uint32_t pend = 0u;
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * SM::NCT) * 4;
            v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            gk[i] = make_uint2(0x3f803f80u, 0x3f803f80u);   // bf16 ones
            if (e < n) {
                pend |= 1u << i;
                if (norm) gk[i] = __ldg(reinterpret_cast<const uint2*>(gain + e));
            }
        }
        PollGuard pg = {0ull, 0u, (int)(tag & 15u) + 100};
        for (;;) {
#pragma unroll
            for (int i = 0; i < NB; ++i) {
                if ((pend >> i) & 1u) {
                    const uint32_t e = base + (ctid + i * SM::NCT) * 4;
                    const uint4 a = ld_tw2(src + e), b = ld_tw2(src + e + 2);
                    if (a.y == tag && a.w == tag && b.y == tag && b.w == tag) {
                        v[i] = make_float4(__uint_as_float(a.x), __uint_as_float(a.z), __uint_as_float(b.x), __uint_as_float(b.z));
                        pend &= ~(1u << i);
                    }
                }
            }
            if (pend == 0u || !poll_continue(p, s, pg)) break;
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * SM::NCT) * 4;
            ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
            if (e < n) {
                // the gains go in now, the normaliser (one number for the whole vector) is applied to the stage's outputs
                const float4 o = make_float4(v[i].x * bf_lo(gk[i].x), v[i].y * bf_hi(gk[i].x), v[i].z * bf_lo(gk[i].y),
                                             v[i].w * bf_hi(gk[i].y));
                *reinterpret_cast<float4*>(s.vec(p) + vec_perm(e)) = o;
            }
        }
    }
    if (SM::kTrace && norm && p.trace != nullptr && ctid == 0) {   // stamps 8 / 11: thread 0 holds valid data (diagnostic)
        const uint32_t layer = (tag >> 4) % p.L;
        p.trace[((size_t)blockIdx.x * p.L + layer) * TRACE_STAMPS + (((tag >> 1) & 7u) == TG_XA ? 8 : 11)] = globaltimer_ns();
    }
    float inv = 1.f;
    if (norm) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((ctid & 31) == 0) s.red()[ctid >> 5] = ss;
    }
    consumer_bar<SM>();
    if (norm) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < SM::NCW; ++w) tot += s.red()[w];
        inv = rsqrtf(tot / (float)n + p.eps);
    }
    return inv;
}

// This lane's share of a slice of the input vector: for block b of 256 columns the 8 columns b*256 + lane*8 .. +7.
struct XRegs {
    float v[MAX_XB][8];
};
// Loads columns [kofs, kofs + klen) of the shared input vector (lane-permuted layout, see vec_perm) into registers;
// columns beyond klen read as zero.  kofs is a multiple of 256.
__device__ __forceinline__ void load_xregs(XRegs& x, const float* vec, uint32_t kofs, uint32_t klen, uint32_t lane) {
    const float4* v4 = reinterpret_cast<const float4*>(vec) + (kofs >> 8) * 64;
#pragma unroll
    for (int b = 0; b < MAX_XB; ++b) {
        float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
        if ((uint32_t)b * 256u + lane * 8u < klen) {
            lo = v4[b * 64 + lane];
            hi = v4[b * 64 + 32 + lane];
        }
        x.v[b][0] = lo.x; x.v[b][1] = lo.y; x.v[b][2] = lo.z; x.v[b][3] = lo.w;
        x.v[b][4] = hi.x; x.v[b][5] = hi.y; x.v[b][6] = hi.z; x.v[b][7] = hi.w;
    }
}

// Same slice taken straight from global memory (a vector written by other CTAs: read through L2), for input
// vectors that are not staged in shared memory.  src points at column 0 of the whole vector.
__device__ __forceinline__ void load_xregs_global(XRegs& x, const float* src, uint32_t kofs, uint32_t klen, uint32_t lane) {
    float4 lo[MAX_XB], hi[MAX_XB];
#pragma unroll
    for (int b = 0; b < MAX_XB; ++b) {
        lo[b] = make_float4(0.f, 0.f, 0.f, 0.f);
        hi[b] = lo[b];
        const uint32_t k = (uint32_t)b * 256u + lane * 8u;
        if (k < klen) {
            lo[b] = __ldcg(reinterpret_cast<const float4*>(src + kofs + k));
            hi[b] = __ldcg(reinterpret_cast<const float4*>(src + kofs + k + 4));
        }
    }
#pragma unroll
    for (int b = 0; b < MAX_XB; ++b) {
        x.v[b][0] = lo[b].x; x.v[b][1] = lo[b].y; x.v[b][2] = lo[b].z; x.v[b][3] = lo[b].w;
        x.v[b][4] = hi[b].x; x.v[b][5] = hi[b].y; x.v[b][6] = hi[b].z; x.v[b][7] = hi[b].w;
    }
}

// acc[r] = sum over this lane's columns of W[r][k] * x[k] for NR rows held in shared memory (row pitch `pitch`
// bytes, klen columns each).  The vector comes from registers, so the only shared-memory traffic is the weights.
// Two accumulators per row (even and odd columns) keep the FMA chains short; the order of the sums is fixed.
template <int NR>
__device__ __forceinline__ void dot_rows(const uint8_t* w, uint32_t pitch, uint32_t klen, uint32_t lane, const XRegs& x,
                                         float (&acc)[NR]) {
    float e[NR], o[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) e[r] = o[r] = 0.f;
    // blocks in groups of four: the (predicated) loads of a group are all issued before its arithmetic, so the
    // shared-memory latency is paid once per group, not once per block
#pragma unroll
    for (int b0 = 0; b0 < MAX_XB; b0 += 4) {
        if ((uint32_t)b0 * 256u < klen) {                   // uniform over the warp
            uint4 q[4][NR];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t k = (uint32_t)(b0 + u) * 256u + lane * 8u;
                const bool in = b0 + u < MAX_XB && k < klen;   // false only in or after the last, partial block
                const uint32_t kk = in ? k : 0u;
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    q[u][r] = *reinterpret_cast<const uint4*>(w + (size_t)r * pitch + (size_t)kk * 2);
                    if (!in) q[u][r] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int b = b0 + u < MAX_XB ? b0 + u : MAX_XB - 1;   // blocks past the end hold zero weights
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    ffma2(e[r], o[r], bf_lo(q[u][r].x), bf_hi(q[u][r].x), x.v[b][0], x.v[b][1]);
                    ffma2(e[r], o[r], bf_lo(q[u][r].y), bf_hi(q[u][r].y), x.v[b][2], x.v[b][3]);
                    ffma2(e[r], o[r], bf_lo(q[u][r].z), bf_hi(q[u][r].z), x.v[b][4], x.v[b][5]);
                    ffma2(e[r], o[r], bf_lo(q[u][r].w), bf_hi(q[u][r].w), x.v[b][6], x.v[b][7]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] = e[r] + o[r];
}

// Variant for pieces of NB full blocks plus, possibly, one partial block: no predicates on the full blocks, so the
// compiler is free to software-pipeline the shared-memory loads against the arithmetic.  Same order of operations as
// dot_rows.
template <int NR, int NB>
__device__ __forceinline__ void dot_rows_full(const uint8_t* w, uint32_t pitch, uint32_t klen, uint32_t lane, const XRegs& x,
                                              float (&acc)[NR]) {
    float e[NR], o[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) e[r] = o[r] = 0.f;
    const uint8_t* wl = w + (size_t)lane * 16;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const uint4 q = *reinterpret_cast<const uint4*>(wl + (size_t)r * pitch + (size_t)b * 512);
            ffma2(e[r], o[r], bf_lo(q.x), bf_hi(q.x), x.v[b][0], x.v[b][1]);
            ffma2(e[r], o[r], bf_lo(q.y), bf_hi(q.y), x.v[b][2], x.v[b][3]);
            ffma2(e[r], o[r], bf_lo(q.z), bf_hi(q.z), x.v[b][4], x.v[b][5]);
            ffma2(e[r], o[r], bf_lo(q.w), bf_hi(q.w), x.v[b][6], x.v[b][7]);
        }
    }
    if constexpr (NB < MAX_XB) {
        if ((uint32_t)NB * 256u + lane * 8u < klen) {   // the partial block (klen is a multiple of 8)
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                const uint4 q = *reinterpret_cast<const uint4*>(wl + (size_t)r * pitch + (size_t)NB * 512);
                ffma2(e[r], o[r], bf_lo(q.x), bf_hi(q.x), x.v[NB][0], x.v[NB][1]);
                ffma2(e[r], o[r], bf_lo(q.y), bf_hi(q.y), x.v[NB][2], x.v[NB][3]);
                ffma2(e[r], o[r], bf_lo(q.z), bf_hi(q.z), x.v[NB][4], x.v[NB][5]);
                ffma2(e[r], o[r], bf_lo(q.w), bf_hi(q.w), x.v[NB][6], x.v[NB][7]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] = e[r] + o[r];
}
// NR rows: picks the variant by the number of full blocks of the piece.
template <int NR>
__device__ __forceinline__ void dot_n(const uint8_t* w, uint32_t pitch, uint32_t klen, uint32_t lane, const XRegs& x,
                                      float (&acc)[NR]) {
    switch (klen >> 8) {
        case 5: dot_rows_full<NR, (MAX_XB >= 5 ? 5 : MAX_XB)>(w, pitch, klen, lane, x, acc); break;
        case 6: dot_rows_full<NR, (MAX_XB >= 6 ? 6 : MAX_XB)>(w, pitch, klen, lane, x, acc); break;
        default: dot_rows<NR>(w, pitch, klen, lane, x, acc); break;
    }
}

// Whole rows with the input vector read from shared memory block by block (lane-permuted layout, see vec_perm):
// for rows too long for a register-resident slice.  Per block of 256 columns a lane loads its 8 vector elements
// (two conflict-free 16-byte loads) and one 16-byte piece of every row.  klen is a multiple of 8.
template <int NR>
__device__ __forceinline__ void dot_rows_smemx(const uint8_t* w, uint32_t pitch, uint32_t klen, uint32_t lane,
                                               const float* vec, float (&acc)[NR]) {
    float e[NR], o[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) e[r] = o[r] = 0.f;
    const float4* v4 = reinterpret_cast<const float4*>(vec) + lane;
    const uint8_t* wl = w + (size_t)lane * 16;
    const uint32_t nb = klen >> 8;
#pragma unroll 4
    for (uint32_t b = 0; b < nb; ++b) {
        const float4 lo = v4[b * 64], hi = v4[b * 64 + 32];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const uint4 q = *reinterpret_cast<const uint4*>(wl + (size_t)r * pitch + (size_t)b * 512);
            ffma2(e[r], o[r], bf_lo(q.x), bf_hi(q.x), lo.x, lo.y);
            ffma2(e[r], o[r], bf_lo(q.y), bf_hi(q.y), lo.z, lo.w);
            ffma2(e[r], o[r], bf_lo(q.z), bf_hi(q.z), hi.x, hi.y);
            ffma2(e[r], o[r], bf_lo(q.w), bf_hi(q.w), hi.z, hi.w);
        }
    }
    if ((klen & 255u) && nb * 256u + lane * 8u < klen) {   // last, partial block
        const float4 lo = v4[nb * 64], hi = v4[nb * 64 + 32];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const uint4 q = *reinterpret_cast<const uint4*>(wl + (size_t)r * pitch + (size_t)nb * 512);
            ffma2(e[r], o[r], bf_lo(q.x), bf_hi(q.x), lo.x, lo.y);
            ffma2(e[r], o[r], bf_lo(q.y), bf_hi(q.y), lo.z, lo.w);
            ffma2(e[r], o[r], bf_lo(q.z), bf_hi(q.z), hi.x, hi.y);
            ffma2(e[r], o[r], bf_lo(q.w), bf_hi(q.w), hi.z, hi.w);
        }
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) acc[r] = e[r] + o[r];
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
// Where a stage's results go.  Tagged outputs (`tw`) are read by other CTAs of the running kernel; `plain` outputs are
// only read after the kernel (logits) or are guarded by a counter (h).  `res` is the tagged vector the residual is
// taken from: this CTA validated all of its tags when it loaded the vector at the start of an earlier stage.
struct GemvOut {
    TW* tw;
    float* plain;
    const TW* res;
    uint32_t tag;
};
__device__ __forceinline__ void emit_value(const GemvOut& o, uint32_t idx, float v) {
    if (o.tw) st_tw(o.tw + idx, v, o.tag);
    else o.plain[idx] = v;
}

// Partial sums of a unit's column pieces meet in shared memory; the last piece to arrive adds them in piece order.
// Called by one lane per chunk.  Returns true for that last piece, with the unit's complete sums in y.
template <class SM>
__device__ __forceinline__ bool unit_combine(const SM& s, const GemvPlan& pl, const ChunkGeom& g, uint32_t u0,
                                             float (&y)[MAX_RPC_SPLIT]) {
    const uint32_t us = (g.unit - u0) % UNIT_SLOTS;
    volatile float* part = s.unit_part() + us * (MAX_PIECES * MAX_RPC_SPLIT);
#pragma unroll
    for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr) part[g.piece * MAX_RPC_SPLIT + rr] = y[rr];
    __threadfence_block();
    const int old = atomicAdd(&s.unit_cnt()[us], 1);
    const uint32_t tp = SM::kMoe ? pl.npieces * pl.nseg : pl.npieces;
    if (old != (int)tp - 1) return false;
    __threadfence_block();
    s.unit_cnt()[us] = 0;
#pragma unroll
    for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr) y[rr] = 0.f;
    for (uint32_t j = 0; j < tp; ++j) {
#pragma unroll
        for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr) y[rr] += part[j * MAX_RPC_SPLIT + rr];
    }
    return true;
}

// Router of a mixture-of-experts layer, computed by EVERY CTA for itself from the normalised hidden state in the vector
// area (g2 * x; xscale is RMSNorm's normaliser): logits r_e = xscale * W_r[e] . vec, the top_k largest in descending
// order (the lower index first among equals), their softmax as gate weights.  The result goes to shared memory for the
// consumer warps (gate weights) and the producer thread, which cannot request an expert's tiles before it knows which
// expert it is -- the one place where the weight stream of the looped kernel depends on an activation.
template <class SM>
__device__ __noinline__ void moe_router(const Params& p, const SM& s, uint32_t layer, float xscale, uint32_t ctid) {
    const uint32_t warp = ctid >> 5, lane = ctid & 31u, E = p.n_experts;
    float* logits = s.unit_part();   // the unit table is idle between the stages
    const __nv_bfloat16* wr = p.wrouter + (size_t)layer * p.layer_stride;
    const float4* v4 = reinterpret_cast<const float4*>(s.vec(p)) + lane;
    for (uint32_t e = warp; e < E; e += SM::NCW) {
        const uint8_t* row = reinterpret_cast<const uint8_t*>(wr + (size_t)e * p.H) + (size_t)lane * 16;
        float acc = 0.f;
        for (uint32_t b = 0; b * 256u < p.H; ++b) {
            if (b * 256u + lane * 8u < p.H) {   // H is a multiple of 8
                const uint4 q = __ldg(reinterpret_cast<const uint4*>(row + (size_t)b * 512));
                const float4 lo = v4[b * 64], hi = v4[b * 64 + 32];
                acc = fmaf(bf_lo(q.x), lo.x, acc); acc = fmaf(bf_hi(q.x), lo.y, acc);
                acc = fmaf(bf_lo(q.y), lo.z, acc); acc = fmaf(bf_hi(q.y), lo.w, acc);
                acc = fmaf(bf_lo(q.z), hi.x, acc); acc = fmaf(bf_hi(q.z), hi.y, acc);
                acc = fmaf(bf_lo(q.w), hi.z, acc); acc = fmaf(bf_hi(q.w), hi.w, acc);
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) logits[e] = acc * xscale;
    }
    consumer_bar<SM>();
    if (ctid == 0) {
        MoeSel* m = s.moe();
        uint32_t taken = 0u;
        float top[MAX_TOP_K];
        for (uint32_t k = 0; k < p.top_k; ++k) {
            uint32_t best = 0xffffffffu;
            for (uint32_t e = 0; e < E; ++e)
                if (!((taken >> e) & 1u) && (best == 0xffffffffu || logits[e] > logits[best])) best = e;
            taken |= 1u << best;
            m->e[k] = best;
            top[k] = logits[best];
        }
        float sum = 0.f;
        const float mx = top[0];   // chosen in descending order: the first is the maximum
        for (uint32_t k = 0; k < p.top_k; ++k) {
            top[k] = expf(top[k] - mx);
            sum += top[k];
        }
        for (uint32_t k = 0; k < p.top_k; ++k) m->w[k] = top[k] / sum;
        __threadfence_block();
        m->seq = m->seq + 1u;   // the producer thread waits for this
    }
    consumer_bar<SM>();
}

// Producer side of a mixture-of-experts layer: waits (bounded) until the consumers have routed the n-th layer of the
// launch, then streams this CTA's share of the chosen experts' gate/up matrices and down matrices.
template <class SM>
__device__ __forceinline__ bool moe_wait_route(const Params& p, const SM& s, uint32_t n, uint32_t (&ex)[MAX_TOP_K]) {
    const MoeSel* m = s.moe();
    if (m->seq < n) {
        const uint64_t t0 = globaltimer_ns();
        uint32_t it = 0;
        while (m->seq < n) {
            if ((++it & 63u) == 0) {
                if (*s.abort_flag()) return false;
                if (globaltimer_ns() - t0 > p.wait_ns) {
                    raise_abort(p, s, ERR_SYNC_TIMEOUT, 800);
                    return false;
                }
            }
        }
    }
    __threadfence_block();
    for (uint32_t k = 0; k < (uint32_t)MAX_TOP_K; ++k) ex[k] = k < p.top_k ? m->e[k] : 0u;
    return true;
}
// gate/up: the chosen experts' row units one expert after the other (unit u of the stage = unit u % nunits of chosen
// expert u / nunits); down: every row unit has the pieces of all chosen experts, expert after expert.
template <class SM>
__device__ __forceinline__ void produce_matrix_moe(const Params& p, const SM& s, RingProd& r, const GemvPlan& pl,
                                                   const __nv_bfloat16* base, uint32_t cta, const uint32_t (&ex)[MAX_TOP_K], bool down) {
    const uint32_t k = p.top_k;
    const uint32_t last_len = pl.K - (pl.npieces - 1) * pl.kp;
    if (!down) {
        GemvPlan all = pl;
        all.nunits = pl.nunits * k;
        const CtaRange cr = cta_units(all, cta, p.P);
        for (uint32_t u = cr.u0; u < cr.u1; ++u) {
            const uint32_t sl = u / pl.nunits, ue = u - sl * pl.nunits;
            const uint8_t* ptr = reinterpret_cast<const uint8_t*>(base + (size_t)ex[sl] * p.expert_stride) + (size_t)ue * pl.rpc * pl.K * 2u;
            const uint32_t rows = min(pl.rpc, pl.R - ue * pl.rpc);
            for (uint32_t j = 0; j < pl.npieces; ++j) {
                const uint32_t bytes = rows * ((j == pl.npieces - 1) ? last_len : pl.kp) * 2u;
                prod_issue(p, s, r, ptr, bytes, nullptr, 0u, 0u);
                ptr += bytes;
            }
        }
    } else {
        const CtaRange cr = cta_units(pl, cta, p.P);
        for (uint32_t u = cr.u0; u < cr.u1; ++u) {
            const uint32_t rows = min(pl.rpc, pl.R - u * pl.rpc);
            for (uint32_t sl = 0; sl < k; ++sl) {
                const uint8_t* ptr = reinterpret_cast<const uint8_t*>(base + (size_t)ex[sl] * p.expert_stride) + (size_t)u * pl.rpc * pl.K * 2u;
                for (uint32_t j = 0; j < pl.npieces; ++j) {
                    const uint32_t bytes = rows * ((j == pl.npieces - 1) ? last_len : pl.kp) * 2u;
                    prod_issue(p, s, r, ptr, bytes, nullptr, 0u, 0u);
                    ptr += bytes;
                }
            }
        }
    }
}

template <class SM>
__device__ __forceinline__ void gemv_stage(const Params& p, const SM& s, const GemvPlan& pl, int ep, const GemvOut& out,
                                        uint32_t cta, uint32_t warp, uint32_t lane, RingCursor& rc, WarpRing& wr,
                                        const float* xsrc, float xscale) {
    // xsrc == nullptr: the input vector is staged in s.vec(p); otherwise it is read from global memory per piece
    const CtaRange r = cta_units(pl, cta, p.P);
    const uint32_t tp = SM::kMoe ? pl.npieces * pl.nseg : pl.npieces;   // chunks per unit
    const uint32_t nch = (r.u1 - r.u0) * tp;
    const uint32_t first = rc.first_chunk(warp, p.nslots);
    XRegs x;
    uint32_t x_piece = 0xffffffffu;
    // rows that come whole and find their vector in shared memory are multiplied against it block by block
    const bool smemx = xsrc == nullptr && pl.rpc <= (uint32_t)MAX_RPC_SPLIT;
    for (uint32_t i = first; i < nch; i += p.nslots) {
        const ChunkGeom g = chunk_geom<SM::kMoe>(pl, r.u0, i);
        // mixture of experts: the gate weight of the expert whose (gate, up) rows these are goes into the SwiGLU output
        const float gw = (SM::kMoe && ep == EP_SWIGLU) ? s.moe()->w[g.row / (2u * p.F)] : 1.f;
        if (!smemx && g.piece != x_piece) {  // same piece on every turn when the piece count divides the consumer count
            if (xsrc) load_xregs_global(x, xsrc, g.kofs, g.klen, lane);
            else load_xregs(x, s.vec(p), g.kofs, g.klen, lane);
            x_piece = g.piece;
        }
        const uint32_t slot = warp * p.nsw + wr.cslot;
        const uint8_t* sp = s.ring() + (size_t)slot * SLOT_BYTES;
        const uint32_t pitch = g.klen * 2u;
        if (smemx) {
            // Rows (or, for rows longer than a slot, column pieces starting at a block of 256) multiplied against the
            // vector in shared memory block by block.  Whole rows need no cross-warp combine: the warp that
            // multiplied them emits them.
            float res = 0.f;
            if (ep == EP_RESIDUAL && lane < g.nrows) res = ld_tw(out.res + g.row + lane).v;
            mbar_wait(p, s, smem_u32(&s.full()[slot]), wr.cphase);
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 2);
            ring_advance_consume(p, wr);
            float y[MAX_RPC_SPLIT] = {0.f, 0.f, 0.f, 0.f};
            if (g.nrows == 2) {
                float acc[2];
                dot_rows_smemx<2>(sp, pitch, g.klen, lane, s.vec(p) + g.kofs, acc);
                y[0] = acc[0]; y[1] = acc[1];
            } else if (g.nrows == 4) {
                float acc[4];
                dot_rows_smemx<4>(sp, pitch, g.klen, lane, s.vec(p) + g.kofs, acc);
                y[0] = acc[0]; y[1] = acc[1]; y[2] = acc[2]; y[3] = acc[3];
            } else if (g.nrows == 3) {
                float acc[3];
                dot_rows_smemx<3>(sp, pitch, g.klen, lane, s.vec(p) + g.kofs, acc);
                y[0] = acc[0]; y[1] = acc[1]; y[2] = acc[2];
            } else {
                float acc[1];
                dot_rows_smemx<1>(sp, pitch, g.klen, lane, s.vec(p) + g.kofs, acc);
                y[0] = acc[0];
            }
            __syncwarp();
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 1);
            ring_release(p, s, wr, warp, lane);
            y[0] = warp_sum(y[0]);
            y[1] = warp_sum(y[1]);
            if (g.nrows > 2) {   // uniform over the warp
                y[2] = warp_sum(y[2]);
                y[3] = warp_sum(y[3]);
            }
            if (tp > 1) {
                if (lane == 0 && unit_combine(s, pl, g, r.u0, y)) {
                    if (ep == EP_SWIGLU) {
                        emit_value(out, g.row >> 1, gw * silu(y[0] * xscale) * (y[1] * xscale));
                        if (g.nrows == 4) emit_value(out, (g.row >> 1) + 1, gw * silu(y[2] * xscale) * (y[3] * xscale));
                    } else {
#pragma unroll
                        for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr)
                            if ((uint32_t)rr < g.nrows)
                                emit_value(out, g.row + rr, (ep == EP_RESIDUAL ? ld_tw(out.res + g.row + rr).v : 0.f) + y[rr] * xscale);
                    }
                }
            } else if (ep == EP_SWIGLU) {
                if (lane == 0) emit_value(out, g.row >> 1, gw * silu(y[0] * xscale) * (y[1] * xscale));
                if (lane == 1 && g.nrows == 4) emit_value(out, (g.row >> 1) + 1, gw * silu(y[2] * xscale) * (y[3] * xscale));
            } else if (lane < g.nrows) {
                // lane rr emits row rr (every lane holds all sums after the butterfly)
                const float v = lane == 0 ? y[0] : lane == 1 ? y[1] : lane == 2 ? y[2] : y[3];
                emit_value(out, g.row + lane, (ep == EP_RESIDUAL ? res : 0.f) + v * xscale);
            }
        } else if (pl.rpc <= MAX_RPC_SPLIT) {
            // one unit piece of up to four rows: the common case.  Residual inputs are fetched before the wait, their
            // L2 latency hides behind it.
            float res = 0.f;
            if (ep == EP_RESIDUAL && lane < g.nrows) res = ld_tw(out.res + g.row + lane).v;
            mbar_wait(p, s, smem_u32(&s.full()[slot]), wr.cphase);
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 2);
            ring_advance_consume(p, wr);
            float y[MAX_RPC_SPLIT] = {0.f, 0.f, 0.f, 0.f};
            if (g.nrows == 2) {
                float acc[2];
                dot_n<2>(sp, pitch, g.klen, lane, x, acc);
                y[0] = acc[0]; y[1] = acc[1];
            } else if (g.nrows == 3) {
                float acc[3];
                dot_n<3>(sp, pitch, g.klen, lane, x, acc);
                y[0] = acc[0]; y[1] = acc[1]; y[2] = acc[2];
            } else if (g.nrows == 4) {
                float acc[4];
                dot_n<4>(sp, pitch, g.klen, lane, x, acc);
                y[0] = acc[0]; y[1] = acc[1]; y[2] = acc[2]; y[3] = acc[3];
            } else {
                float acc[1];
                dot_n<1>(sp, pitch, g.klen, lane, x, acc);
                y[0] = acc[0];
            }
            __syncwarp();
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 1);
            ring_release(p, s, wr, warp, lane);   // the slot has been read for the last time
#pragma unroll
            for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr) y[rr] = warp_sum(y[rr]);
            float rs[MAX_RPC_SPLIT];
#pragma unroll
            for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr) rs[rr] = __shfl_sync(0xffffffffu, res, rr);
            if (lane == 0) {
                bool emit = true;
                if (tp > 1) emit = unit_combine(s, pl, g, r.u0, y);
                if (emit) {
                    if (ep == EP_SWIGLU) {
                        emit_value(out, g.row >> 1, gw * silu(y[0] * xscale) * (y[1] * xscale));
                        if (g.nrows == 4) emit_value(out, (g.row >> 1) + 1, gw * silu(y[2] * xscale) * (y[3] * xscale));
                    } else {
#pragma unroll
                        for (int rr = 0; rr < MAX_RPC_SPLIT; ++rr)
                            if ((uint32_t)rr < g.nrows) emit_value(out, g.row + rr, (ep == EP_RESIDUAL ? rs[rr] : 0.f) + y[rr] * xscale);
                    }
                }
            }
        } else {
            // many short rows in one chunk (small hidden sizes): pair after pair, whole rows (npieces == 1)
            mbar_wait(p, s, smem_u32(&s.full()[slot]), wr.cphase);
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 2);
            ring_advance_consume(p, wr);
            for (uint32_t rr = 0; rr < g.nrows; rr += 2) {
                const bool two = rr + 1 < g.nrows;
                float rs0 = 0.f, rs1 = 0.f;
                if (ep == EP_RESIDUAL && lane == 0) {
                    rs0 = ld_tw(out.res + g.row + rr).v;
                    if (two) rs1 = ld_tw(out.res + g.row + rr + 1).v;
                }
                float y0, y1 = 0.f;
                if (two) {
                    float acc[2];
                    dot_rows<2>(sp + (size_t)rr * pitch, pitch, g.klen, lane, x, acc);
                    y0 = warp_sum(acc[0]);
                    y1 = warp_sum(acc[1]);
                } else {
                    float acc[1];
                    dot_rows<1>(sp + (size_t)rr * pitch, pitch, g.klen, lane, x, acc);
                    y0 = warp_sum(acc[0]);
                }
                if (lane == 0) {
                    const uint32_t row = g.row + rr;
                    if (ep == EP_STORE) {
                        emit_value(out, row, y0 * xscale);
                        if (two) emit_value(out, row + 1, y1 * xscale);
                    } else if (ep == EP_RESIDUAL) {
                        emit_value(out, row, rs0 + y0 * xscale);
                        if (two) emit_value(out, row + 1, rs1 + y1 * xscale);
                    } else {
                        emit_value(out, row >> 1, gw * silu(y0 * xscale) * (y1 * xscale));
                    }
                }
            }
            __syncwarp();
            ring_release(p, s, wr, warp, lane);
        }
        if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 3);
    }
    rc.advance(nch, p.nslots);
}

// ------------------------------------------------------------------------------------------------ stash mode
// The ring alone holds nslots * 16 KB per SM -- about 3.6 us of HBM time over the whole GPU -- and every exchange between
// dependent stages that lasts longer stops the weight stream.  Tensor memory is otherwise idle in this kernel: in stash
// mode each weight chunk is moved on from its ring slot into one of 16 TMEM regions of 16 KB by an asynchronous copy
// (tcgen05.cp, issued by two stash threads, one per pipeline), which frees the slot for the next bulk copy at once; the
// consumer warps read the regions into registers (tcgen05.ld).  Ring + TMEM hold 24 chunks = 384 KB per SM.
//   * A TMEM lane quarter is readable by the warps w with w % 4 == quarter only, and the copy spreads a chunk over all
//     128 lanes: lane r receives the 16-byte granules r, r + 128, ... of the chunk.  A chunk is therefore multiplied by
//     a TEAM of four warps (warps 0..3: team 0, warps 4..7: team 1); quarter q holds, of every row, the columns
//     1024 j + 256 q + 8 lane .. + 7 (j = 0 .. kp / 1024 - 1), which is block 4 j + q, lane `lane` of the staged vector.
//   * Plans of this mode have kp a multiple of 1024 that divides K, so every row of a chunk meets the same columns.
//   * All chunks of a unit go to the same team; its four warps add up their quarters over the unit's pieces in registers
//     and meet in shared memory, where the last warp to arrive adds the quarters in order and emits the rows.
//   * K/V chunks of the attention units stay in the ring and are read there, as in the plain mode.
struct TCur {
    uint32_t uc;   // units of all stages so far
    uint32_t c;    // chunks so far in this warp's pipeline
    uint32_t g;    // weight chunks so far in this warp's pipeline
    uint32_t tu;   // units so far of this warp's team
    uint32_t ohead;   // 1: the first units of the O projection are streamed ahead of the K/V chunks (see t_o_head)
    uint32_t kv;      // K/V chunks this warp has read from its ring slot so far
};
// how many k in [0, n) have ((uc + k) & 1) == t
__device__ __forceinline__ uint32_t t_count(uint32_t uc, uint32_t n, uint32_t t) { return (n + (((uc & 1u) == t) ? 1u : 0u)) >> 1; }

// Half a chunk (16 registers = four 16-byte granules per lane) times the lane's slice of the vector.  Granule m of a
// chunk (m = 0 .. 7) belongs to row m / NJ and to column block 4 (m % NJ) + q of the piece; rows beyond 8 / NJ do not
// exist (NJ = 3 leaves two granules unused).  acc[row][0] takes the even columns, acc[row][1] the odd ones.
template <int NJ, int HALF>
__device__ __forceinline__ void t_dot(const uint32_t (&w)[16], const float4* v4, uint32_t blk0, uint32_t q, uint32_t lane,
                                      float (&acc)[8 / NJ][2]) {
    constexpr int NR = 8 / NJ;
#pragma unroll
    for (int jj = 0; jj < NJ; ++jj) {
        // the vector block of column group jj is loaded once for all rows of this half that meet it
        bool used = false;
#pragma unroll
        for (int row = 0; row < NR; ++row) used = used || (row * NJ + jj) / 4 == HALF;
        if (used) {
            const float4 lo = v4[(blk0 + 4u * jj + q) * 64u + lane], hi = v4[(blk0 + 4u * jj + q) * 64u + 32u + lane];
#pragma unroll
            for (int row = 0; row < NR; ++row) {
                const int m = row * NJ + jj;
                if (m / 4 == HALF) {
                    const int gi = (m % 4) * 4;
                    ffma2(acc[row][0], acc[row][1], bf_lo(w[gi]), bf_hi(w[gi]), lo.x, lo.y);
                    ffma2(acc[row][0], acc[row][1], bf_lo(w[gi + 1]), bf_hi(w[gi + 1]), lo.z, lo.w);
                    ffma2(acc[row][0], acc[row][1], bf_lo(w[gi + 2]), bf_hi(w[gi + 2]), hi.x, hi.y);
                    ffma2(acc[row][0], acc[row][1], bf_lo(w[gi + 3]), bf_hi(w[gi + 3]), hi.z, hi.w);
                }
            }
        }
    }
}
// The same with the lane's slice of the vector in registers (whole rows: x[jj] is column block 4 jj + q).
template <int NJ, int HALF>
__device__ __forceinline__ void t_dot_xr(const uint32_t (&w)[16], const float (&x)[NJ][8], float (&acc)[8 / NJ][2]) {
#pragma unroll
    for (int gi = 0; gi < 4; ++gi) {
        constexpr int NR = 8 / NJ;
        const int m = HALF * 4 + gi, row = m / NJ, jj = m % NJ;
        if (row < NR) {
            ffma2(acc[row][0], acc[row][1], bf_lo(w[gi * 4]), bf_hi(w[gi * 4]), x[jj][0], x[jj][1]);
            ffma2(acc[row][0], acc[row][1], bf_lo(w[gi * 4 + 1]), bf_hi(w[gi * 4 + 1]), x[jj][2], x[jj][3]);
            ffma2(acc[row][0], acc[row][1], bf_lo(w[gi * 4 + 2]), bf_hi(w[gi * 4 + 2]), x[jj][4], x[jj][5]);
            ffma2(acc[row][0], acc[row][1], bf_lo(w[gi * 4 + 3]), bf_hi(w[gi * 4 + 3]), x[jj][6], x[jj][7]);
        }
    }
}

// Sums N values per lane over the 32 lanes with N - 1 + log2(32 / N) shuffles: every step halves the values a lane still
// carries (the lane keeps the half named by one of its bits and adds the partner's copy of it), then the single value
// left is summed over the remaining lanes.  Afterwards v[0] of lane l is the total of value (l >> log2(32 / N)) % N --
// a fixed order of additions, the same in every launch.
template <int N>
__device__ __forceinline__ void lanes_reduce(float (&v)[N], uint32_t lane) {
    int o = 16;
#pragma unroll
    for (int n = N; n > 1; n >>= 1, o >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float send = up ? v[i] : v[i + n / 2], keep = up ? v[i + n / 2] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    for (; o > 0; o >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
}

// What the stash-mode stage needs, by value: the stage is a real call (its registers are allocated on their own, whatever
// the calling kernel keeps live), and a callee that reached into the kernel's parameter block would pay a generic load
// for every field.
struct TStageArgs {
    uint32_t R, rpc, kp, tp;      // the plan: rows, rows per unit, columns per chunk, chunks per unit
    uint32_t u0, nu;              // this CTA's units
    int ep;
    GemvOut out;
    float xscale;
    uint32_t warp, lane;
    uint32_t uc, g, tu;           // cursor on entry (see TCur)
};
struct TStageRet {
    uint32_t g, tu;
};
// Bounded mbarrier wait of the stash-mode stage: limit and status word come from the CTA's shared-memory record.
template <class SM>
__device__ __forceinline__ bool mbar_wait_c(const SM& s, uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*s.abort_flag()) return false;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*s.abort_flag()) return false;
            if (globaltimer_ns() - t0 > s.ctx()->wait_ns) {
                int32_t* st = s.ctx()->status;
                if (atomicCAS(st, 0, ERR_SYNC_TIMEOUT) == 0) {
                    st[1] = 510;
                    st[2] = (int)blockIdx.x;
                    st[3] = (int)threadIdx.x;
                }
                *s.abort_flag() = 1;
                return false;
            }
        }
    }
    return true;
}

// One GROUP of units of this warp's team: GU = 8 / NR units of one chunk each (WHOLE rows), or one unit of tp chunks.
// The warp adds up its quarter of every row in registers -- the tensor-memory load of the next half chunk in flight
// under the multiplications of the current one -- and the group's (up to) eight row sums are reduced over the lanes
// together; the four quarters meet in shared memory, where the last warp to arrive adds them in quarter order and emits
// the rows.  Value v of a group is row v % NR of its unit v / NR.
//   wa: the first half of the group's first chunk, its load already in flight; on return, if `more`, that of the next
//       group's first chunk (so that the reduction runs under a load, too)
//   xr: whole rows keep the lane's slice of the vector in registers
template <int NJ, bool WHOLE, class SM>
__device__ __forceinline__ void gemv_group_t(const SM& s, const TStageArgs& a, uint32_t unit0, uint32_t nun, uint32_t T, uint32_t q,
                                             uint32_t& g, uint32_t tu, uint32_t (&wa)[16], bool more, const float (&xr)[NJ][8]) {
    constexpr int NR = 8 / NJ, GU = WHOLE ? 8 / NR : 1;
    const uint32_t lane = a.lane;
    const float4* v4 = reinterpret_cast<const float4*>(s.vec_t());
    const uint32_t tbase = *s.tbase() + ((32u * q) << 16) + T * T_NREG * 32u;
    const uint32_t bars = smem_u32(&s.tfull()[T * T_NREG]), barf = smem_u32(&s.tfree()[T * T_NREG]);
    const uint32_t vrow = (unit0 + 2u * (lane / NR)) * a.rpc + lane % NR;   // units of a team are two apart
    const bool vok = lane < (uint32_t)(GU * NR) && lane / NR < nun && lane % NR < a.rpc && vrow < a.R;
    float res = 0.f;   // fetched before the waits: the L2 latency hides behind them
    if (a.ep == EP_RESIDUAL && vok) res = ld_tw(a.out.res + vrow).v;
    float y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = 0.f;
    float acc[NR][2];
#pragma unroll
    for (int rr = 0; rr < NR; ++rr) acc[rr][0] = acc[rr][1] = 0.f;
    // Half chunks of 16 registers: while one half is multiplied the load of the next one is in flight.
    uint32_t wb[16];
    auto fetch0 = [&]() {   // first half of chunk g
        mbar_wait_c(s, bars + (g % T_NREG) * 8u, (g / T_NREG) & 1u);
        tm_fence_after();
        tm_ld16(tbase + (g % T_NREG) * 32u, wa);
    };
    auto second = [&]() { tm_ld16(tbase + (g % T_NREG) * 32u + 16u, wb); };
    auto landed = [&]() {   // both halves of chunk g are in registers: its region may be overwritten
        tm_fence_before();
        if (lane == 0) mbar_arrive(barf + (g % T_NREG) * 8u);
        ++g;
    };
    if constexpr (WHOLE) {
        // whole rows: chunk c is unit c of the group
#pragma unroll
        for (int c = 0; c < GU; ++c) {
            if ((uint32_t)c < nun) {
                tm_ld_wait();
                second();
                t_dot_xr<NJ, 0>(wa, xr, acc);
                tm_ld_wait();
                landed();
                if ((uint32_t)c + 1u < nun || more) fetch0();
                t_dot_xr<NJ, 1>(wb, xr, acc);
#pragma unroll
                for (int rr = 0; rr < NR; ++rr) {
                    y[c * NR + rr] = acc[rr][0] + acc[rr][1];
                    acc[rr][0] = acc[rr][1] = 0.f;
                }
            }
        }
    } else {
        // one unit of tp column pieces
        for (uint32_t j = 0; j < a.tp; ++j) {
            const uint32_t blk0 = (j * a.kp) >> 8;
            tm_ld_wait();
            second();
            t_dot<NJ, 0>(wa, v4, blk0, q, lane, acc);
            tm_ld_wait();
            landed();
            if (j + 1u < a.tp || more) fetch0();
            t_dot<NJ, 1>(wb, v4, blk0, q, lane, acc);
        }
#pragma unroll
        for (int rr = 0; rr < NR; ++rr) y[rr] = acc[rr][0] + acc[rr][1];
    }
    lanes_reduce<8>(y, lane);
    const uint32_t us = T * T_USLOTS + tu % T_USLOTS;
    volatile float* part = s.unit_part() + us * 32u;
    if ((lane & 3u) == 0u) part[q * 8u + (lane >> 2)] = y[0];
    __syncwarp();
    int old = 0;
    if (lane == 0) {
        // release the quarter sums written above (ordered before this by __syncwarp), acquire the other warps'
        asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(smem_u32(&s.t_ucnt()[us])) : "memory");
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old == 3) {
        if (lane == 0) s.t_ucnt()[us] = 0;
        if (a.ep == EP_SWIGLU) {
            // rows come in (gate, up) pairs: values 2 i and 2 i + 1
            const uint32_t v = 2u * lane;
            const uint32_t prow = (unit0 + 2u * (v / NR)) * a.rpc + v % NR;
            if (v < (uint32_t)(GU * NR) && v / NR < nun && v % NR < a.rpc && prow < a.R) {
                const float ga = part[v] + part[8u + v] + part[16u + v] + part[24u + v];
                const float up = part[v + 1u] + part[8u + v + 1u] + part[16u + v + 1u] + part[24u + v + 1u];
                emit_value(a.out, prow >> 1, silu(ga * a.xscale) * (up * a.xscale));
            }
        } else if (vok) {
            const float sum = part[lane] + part[8u + lane] + part[16u + lane] + part[24u + lane];
            emit_value(a.out, vrow, (a.ep == EP_RESIDUAL ? res : 0.f) + sum * a.xscale);
        }
    }
}

// The units of this warp's team in one stage (see the stash section above).
template <int NJ, class SM>
__device__ __noinline__ TStageRet gemv_units_t(const TStageArgs a) {
    const SM s;
    constexpr int NR = 8 / NJ, GU = 8 / NR;
    const uint32_t T = a.warp >> 2, q = a.warp & 3u, lane = a.lane;
    const uint32_t mine = t_count(a.uc, a.nu, T);
    const uint32_t k0 = ((a.uc & 1u) == T) ? 0u : 1u;
    uint32_t g = a.g, tu = a.tu;
    uint32_t wa[16];
    if (mine) {   // first half of the warp's first chunk of the stage
        mbar_wait_c(s, smem_u32(&s.tfull()[T * T_NREG + g % T_NREG]), (g / T_NREG) & 1u);
        tm_fence_after();
        tm_ld16(*s.tbase() + ((32u * q) << 16) + (T * T_NREG + g % T_NREG) * 32u, wa);
    }
    float xr[NJ][8];   // whole rows: the lane's slice of the vector stays in registers for the stage
    if (a.tp == 1) {
        const float4* v4 = reinterpret_cast<const float4*>(s.vec_t());
#pragma unroll
        for (int jj = 0; jj < NJ; ++jj) {
            const float4 lo = v4[(4u * jj + q) * 64u + lane], hi = v4[(4u * jj + q) * 64u + 32u + lane];
            xr[jj][0] = lo.x; xr[jj][1] = lo.y; xr[jj][2] = lo.z; xr[jj][3] = lo.w;
            xr[jj][4] = hi.x; xr[jj][5] = hi.y; xr[jj][6] = hi.z; xr[jj][7] = hi.w;
        }
    }
    if (a.tp == 1) {
        for (uint32_t m = 0; m < mine; m += GU, ++tu)
            gemv_group_t<NJ, true>(s, a, a.u0 + k0 + 2u * m, min((uint32_t)GU, mine - m), T, q, g, tu, wa, m + GU < mine, xr);
    } else {
        for (uint32_t m = 0; m < mine; ++m, ++tu)
            gemv_group_t<NJ, false>(s, a, a.u0 + k0 + 2u * m, 1u, T, q, g, tu, wa, m + 1u < mine, xr);
    }
    TStageRet r;
    r.g = g;
    r.tu = tu;
    return r;
}

// Consumes this CTA's share of one matrix in stash mode: y = W vec and the stage's epilogue (see gemv_stage).  The input
// vector is staged in the vector area in the lane-permuted layout.
template <class SM>
__device__ __forceinline__ void gemv_stage_t(const Params& p, const SM& s, const GemvPlan& pl, int ep, const GemvOut& out,
                                             uint32_t cta, uint32_t warp, uint32_t lane, TCur& tc, float xscale) {
    const CtaRange r = cta_units(pl, cta, p.P);
    TStageArgs a;
    a.R = pl.R; a.rpc = pl.rpc; a.kp = pl.kp; a.tp = pl.npieces;
    a.u0 = r.u0; a.nu = r.u1 - r.u0;
    a.ep = ep; a.out = out; a.xscale = xscale;
    a.warp = warp; a.lane = lane;
    a.uc = tc.uc; a.g = tc.g; a.tu = tc.tu;
    const uint32_t nj = pl.kp >> 10;
    TStageRet ret;
    if constexpr (SM::kAllWidths) {
        ret = nj == 4u ? gemv_units_t<4, SM>(a) : nj == 2u ? gemv_units_t<2, SM>(a)
            : nj == 3u ? gemv_units_t<3, SM>(a) : gemv_units_t<1, SM>(a);
    } else {
        ret = nj == 4u ? gemv_units_t<4, SM>(a) : gemv_units_t<2, SM>(a);
    }
    const uint32_t mine = t_count(tc.uc, a.nu, warp >> 2);
    tc.uc += a.nu;
    tc.c += mine * a.tp;
    tc.g = ret.g;
    tc.tu = ret.tu;
}

// Stages a plain fp32 vector written by other CTAs (guarded by a counter the caller has waited on) in the vector area.
template <class SM>
__device__ __forceinline__ void load_plain_vec(const Params& p, const SM& s, const float* src, uint32_t n, uint32_t ctid) {
    constexpr int NB = 7;
    for (uint32_t base = 0; base < n; base += NB * SM::NCT * 4) {
        float4 v[NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * SM::NCT) * 4;
            if (e < n) v[i] = __ldcg(reinterpret_cast<const float4*>(src + e));
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const uint32_t e = base + (ctid + i * SM::NCT) * 4;
            if (e < n) *reinterpret_cast<float4*>(s.vec(p) + vec_perm(e)) = v[i];
        }
    }
    consumer_bar<SM>();
}

// End of a stage: all consumer warps have written their outputs; one thread publishes the CTA's arrival.
template <class SM>
__device__ __forceinline__ void stage_signal(uint32_t* ctr, uint32_t ctid, bool skip) {
    consumer_bar<SM>();
    if (ctid == 0 && !skip) red_release_add(ctr, 1u);  // release: cumulative over the CTA barrier above
}

// Waits (bounded) until `target` CTAs have signalled.  Replaces the grid-wide barrier of a kernel boundary.
template <class SM>
__device__ __forceinline__ void stage_wait(const Params& p, const SM& s, const uint32_t* ctr, uint32_t target,
                                           uint32_t ctid) {
    if (ctid == 0) {
        if (*s.abort_flag() == 0 && ld_acquire(ctr) < target) {
            const uint64_t t0 = globaltimer_ns();
            uint32_t it = 0;
            while (ld_acquire(ctr) < target) {
                if ((++it & 31u) == 0) {
                    if (*s.abort_flag()) break;
                    if (__ldcg(p.status) != 0) {
                        *s.abort_flag() = 1;
                        break;
                    }
                    if (globaltimer_ns() - t0 > p.wait_ns) {
                        raise_abort(p, s, ERR_SYNC_TIMEOUT, 600);
                        break;
                    }
                }
            }
        }
    }
    consumer_bar<SM>();
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
template <int HD, bool PACK, class SM>
__device__ __forceinline__ void attn_chunks_tc(const Params& p, const SM& s, const AttnUnit& u, uint32_t cta,
                                               uint32_t warp, uint32_t lane, uint32_t first, const RingCursor& rc,
                                               WarpRing& wr, const float* q_s, float* comb,
                                               const uint8_t* stage_k, const uint8_t* stage_v) {
    constexpr int NKB = HD / 16, NMT = HD / 16;
    const uint32_t G = p.G, g = lane >> 2, t = lane & 3u;
    AttnTcState<HD> st;
#pragma unroll
    for (int kb = 0; kb < NKB; ++kb) {
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const uint32_t k = kb * 16 + hf * 8 + 2 * t;
            const uint32_t head = PACK ? (g & 3u) : g;   // PACK: column g = hi (g < 4) or lo (g >= 4) half of head g % 4
            float2 xx = make_float2(0.f, 0.f);
            if (head < G) xx = *reinterpret_cast<const float2*>(q_s + head * HD + k);   // k is even: 8-byte aligned
            const float x0 = xx.x, x1 = xx.y;
            const uint32_t hi = pack_bf16(x0, x1);
            const uint32_t lo = pack_bf16(x0 - bf_lo(hi), x1 - bf_hi(hi));
            st.qh[kb][hf] = (PACK && g >= 4u) ? lo : hi;
            st.ql[kb][hf] = lo;
        }
    }
#pragma unroll
    for (int n = 0; n < NMT; ++n) st.o[n][0] = st.o[n][1] = st.o[n][2] = st.o[n][3] = 0.f;
    st.m[0] = st.m[1] = -INFINITY;
    st.l[0] = st.l[1] = 0.f;

    const uint32_t pb = attn_positions_per_chunk(p);
    const uint32_t box_bytes = pb * 128u;
    for (uint32_t i = first; i < u.nring; i += p.nslots) {
        const uint32_t slot = warp * p.nsw + wr.cslot;
        mbar_wait(p, s, smem_u32(s.kv_bar(slot)), wr.cphase);
        if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 2);
        ring_advance_consume(p, wr);
        const uint32_t kbase = smem_u32(s.ring()) + slot * SLOT_BYTES;
        const AttnWindow w = attn_window(u.c0, u.cend, pb, i);
        for (uint32_t row0 = 0; row0 < pb; row0 += 16)
            if (row0 + 16 > w.lo && row0 < w.hi) attn_tc_tile<HD, PACK>(st, kbase, kbase + SLOT_BYTES / 2, box_bytes, row0, w.lo, w.hi, lane);
        __syncwarp();
        if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 1);
        ring_release(p, s, wr, warp, lane);
        if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 3);
    }
    if (u.has_new && first == 0)  // the position written by this step sits in row 0 of the staging tile
        attn_tc_tile<HD, PACK>(st, smem_u32(stage_k), smem_u32(stage_v), 128u, 0u, 0u, 1u, lane);

    // row sums: add the parts held by the lanes that share the heads (same lane % 4)
    float l0 = st.l[0], l1 = st.l[1];
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, o);
        l1 += __shfl_xor_sync(0xffffffffu, l1, o);
    }
    if (PACK) {   // columns 0..3 hold the hi parts of O^T, columns 4..7 the lo parts: lanes t and t ^ 2 of a quad
#pragma unroll
        for (int n = 0; n < NMT; ++n)
#pragma unroll
            for (int j = 0; j < 4; ++j) st.o[n][j] += __shfl_xor_sync(0xffffffffu, st.o[n][j], 2);
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const uint32_t h = 2 * t + hh;
        if (h < G && (!PACK || t < 2u)) {
            float* dst = comb + ((size_t)first * G + h) * (HD + 2);
#pragma unroll
            for (int n = 0; n < NMT; ++n) {
                dst[n * 16 + g] = st.o[n][hh];
                dst[n * 16 + g + 8] = st.o[n][2 + hh];
            }
            if (g == 0) {
                dst[HD] = st.m[hh];
                dst[HD + 1] = hh ? l1 : l0;
            }
        }
    }
}

// Two tagged words that may lie apart, polled until both carry `tag` (bounded).
template <class SM>
__device__ __forceinline__ void poll_pair(const Params& p, const SM& s, const TW* a, const TW* b, uint32_t tag, float& va,
                                          float& vb) {
    PollGuard pg = {0ull, 0u, 200 + (int)(tag >> 4) * 1000};
    for (;;) {
        const TW x = ld_tw(a), y = ld_tw(b);
        va = x.v;
        vb = y.v;
        if ((x.tag == tag && y.tag == tag) || !poll_continue(p, s, pg)) return;
    }
}

// Merges the split-K partial results of one (sequence, kv head) into the attention output o.  Every unit of the
// group merges its own slice of the G * hd outputs (unit c takes outputs [c*S, (c+1)*S), S = ceil(G*hd / nchunk)), so
// the merge costs each unit a handful of loads that are all in flight at once -- one L2 round trip after the last
// unit of the group has published its partial result -- instead of one unit reading everything in several passes.
// The partial results are tagged words, polled until they are there.  Steps: the (max, sum) pairs of every
// (head, chunk) and the unit's slice of every chunk's partial output go to shared memory; the pairs become weights
// w[h][c] = exp2(m_c - M_h) / L_h; thread j adds its output's nchunk terms in chunk order.  The orders of all sums
// are fixed.
template <class SM>
__device__ __noinline__ void attn_merge(const Params& p, const SM& s, const StepCtx& cx, const AttnUnit& u, uint32_t layer,
                                        uint32_t G, uint32_t ctid, float* comb) {
    const uint32_t hd = p.hd, b = 0u, g = u.g, nchunk = u.nchunk;   // b: slot of the sequence in the scratch vectors
    const uint32_t unit0 = u.bg * p.cps;
    const uint32_t tag = tag_of(p, cx, layer, TG_PART), otag = tag_of(p, cx, layer, TG_O);
    const uint32_t total = G * hd;
    const uint32_t S = (total + nchunk - 1) / nchunk;
    const uint32_t t_lo = min(total, u.ch * S), t_hi = min(total, t_lo + S);
    const uint32_t ns = t_hi - t_lo;
    // the tables sit behind the per-warp partials, which other threads of the CTA may still be reading
    float* wtab = comb + (size_t)SM::NCW * G * (hd + 2);   // [2][G][nchunk]: maxima, sums; then weights in the first half
    float* pv = wtab + 2 * G * nchunk;                 // [ns][nchunk] partial outputs of this unit's slice
    // all loads of a thread are issued before it waits on any of them; only those that are late are repeated
    constexpr int NL = 2;
    const uint32_t nml = G * nchunk, npv = ns * nchunk;
    for (uint32_t i0 = 0; i0 < max(nml, (npv + NL - 1) / NL); i0 += SM::NCT) {
        const uint32_t i = i0 + ctid;
        bool ml_pend = i < nml;
        uint32_t pend = 0u;
#pragma unroll
        for (int k = 0; k < NL; ++k)
            if (i * NL + k < npv) pend |= 1u << k;
        PollGuard pg = {0ull, 0u, 300};
        while (ml_pend || pend) {
            if (ml_pend) {
                const uint32_t h = i / nchunk, c = i % nchunk;
                const uint4 ml = ld_tw2(p.part_ml + ((size_t)(unit0 + c) * G + h) * 2);
                if (ml.y == tag && ml.w == tag) {
                    wtab[i] = __uint_as_float(ml.x);
                    wtab[nml + i] = __uint_as_float(ml.z);
                    ml_pend = false;
                }
            }
#pragma unroll
            for (int k = 0; k < NL; ++k) {
                if ((pend >> k) & 1u) {
                    const uint32_t j = i * NL + k;
                    const uint32_t t = t_lo + j / nchunk, c = j % nchunk;
                    const TW w = ld_tw(p.part + (size_t)(unit0 + c) * total + t);
                    if (w.tag == tag) {
                        pv[j] = w.v;
                        pend &= ~(1u << k);
                    }
                }
            }
            if ((ml_pend || pend) && !poll_continue(p, s, pg)) break;
        }
    }
    trace_stamp(p, s, blockIdx.x, layer, 5, ctid);
    consumer_bar<SM>();
    // one warp per head: maximum and normaliser by butterfly reductions (every lane ends with the same value)
    for (uint32_t h = ctid >> 5; h < G; h += SM::NCW) {
        const uint32_t lane = ctid & 31u;
        float Mx = -INFINITY;
        for (uint32_t c = lane; c < nchunk; c += 32) Mx = fmaxf(Mx, wtab[h * nchunk + c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Mx = fmaxf(Mx, __shfl_xor_sync(0xffffffffu, Mx, o));
        float Lx = 0.f;
        for (uint32_t c = lane; c < nchunk; c += 32) {
            const float sc = rescale(wtab[h * nchunk + c], Mx);
            Lx += wtab[nml + h * nchunk + c] * sc;
            wtab[h * nchunk + c] = sc;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Lx += __shfl_xor_sync(0xffffffffu, Lx, o);
        const float inv = 1.0f / Lx;
        for (uint32_t c = lane; c < nchunk; c += 32) wtab[h * nchunk + c] *= inv;
    }
    consumer_bar<SM>();
    for (uint32_t j = ctid; j < ns; j += SM::NCT) {
        const uint32_t t = t_lo + j, h = t / hd, d = t % hd;
        float acc = 0.f;
        for (uint32_t c = 0; c < nchunk; ++c) acc += pv[j * nchunk + c] * wtab[h * nchunk + c];
        st_tw(p.o + (size_t)b * p.QD + (size_t)(g * G + h) * hd + d, acc, otag);
    }
}

// Split-K decode attention of one layer (flash-decoding): CTA `cta` owns at most one unit (kv head, chunk of the
// cached positions); its cached K/V rows arrive through the ring, requested while the QKV stage was still running.
// The unit polls the q (and, for the chunk that ends with the new position, k and v) rows it needs, runs its ring
// chunks, merges its warps and publishes the partial result; then every unit of the kv head merges its slice of
// the outputs (attn_merge).  Scores use q pre-multiplied by log2(e)/sqrt(hd): the softmax runs in base 2.
// GT > 0 selects the CUDA-core inner loop for GT query heads per KV head; GT == 0 the tensor-core loop.
template <int GT, class SM>
__device__ __noinline__ void attention_stage(const Params& p, const SM& s, const StepCtx& cx, uint32_t layer, uint32_t cta,
                                                 uint32_t ctid, uint32_t warp, uint32_t lane, RingCursor& rc, WarpRing& wr) {
    const AttnUnit u = attn_unit(p, cta, cx.pos);
    if (!u.active) return;
    const uint32_t G = GT > 0 ? (uint32_t)GT : p.G;
    const uint32_t hd = p.hd, half = hd >> 1;
    const uint32_t b = 0u, g = u.g, nchunk = u.nchunk;   // b: slot of the sequence in the scratch vectors

    // shared workspace inside the vector area
    float* q_s = s.vec(p);                         // [G][hd]
    float* new_k = q_s + G * hd;                // [hd]
    float* new_v = new_k + hd;                  // [hd]
    // Staging "tile" of the position written by this step: only row 0 of each 64-column box is ever valid, so the
    // boxes are packed 128 bytes apart; the 15 ignored rows the tile loop also reads overlap whatever follows.
    uint8_t* stage_k = reinterpret_cast<uint8_t*>(new_v + hd);   // [hd/64][128 B]
    uint8_t* stage_v = stage_k + 256;
    float* comb = reinterpret_cast<float*>(stage_v + 256);       // [SM::NCW][G][hd + 2]

    // q (and, for the unit that owns the new position, k and v) of this step: tagged words written by whichever CTAs
    // own those rows of the QKV projection.  The unit waits for exactly the rows it needs, not for the whole stage.
    consumer_bar<SM>();   // the workspace below overlays the QKV stage's input vector: wait for this CTA's last QKV chunk
    const TW* qkv = p.qkv + (size_t)b * (p.QD + 2 * p.KVD);
    const uint32_t qtag = tag_of(p, cx, layer, TG_QKV);
    const float* cs = cx.rope_cs + (size_t)b * hd;  // [half][2]
    const float qscale = 1.4426950408889634f * rsqrtf((float)hd);
    // biases of the projections (decoders that have them): added to the polled values, before the rotation
    const __nv_bfloat16* bias = p.bqkv ? p.bqkv + (size_t)layer * p.layer_stride : nullptr;
    for (uint32_t idx = ctid; idx < G * half; idx += SM::NCT) {
        const uint32_t h = idx / half, i = idx % half;
        const TW* qr = qkv + (size_t)(g * G + h) * hd;
        float a, bb;
        poll_pair(p, s, qr + i, qr + i + half, qtag, a, bb);
        if (bias) {
            a += __bfloat162float(bias[(g * G + h) * hd + i]);
            bb += __bfloat162float(bias[(g * G + h) * hd + i + half]);
        }
        const float c = cs[2 * i], sn = cs[2 * i + 1];
        q_s[h * hd + i] = (a * c - bb * sn) * qscale;
        q_s[h * hd + i + half] = (bb * c + a * sn) * qscale;
    }
    if (u.has_new) {
        const TW* kr = qkv + p.QD + (size_t)g * hd;
        const TW* vr = qkv + p.QD + p.KVD + (size_t)g * hd;
        // row 0 of a swizzled box is stored unswizzled: column k of box k/64 sits at byte (k % 64) * 2 of the box
        for (uint32_t i = ctid; i < half; i += SM::NCT) {
            float a, bb;
            poll_pair(p, s, kr + i, kr + i + half, qtag, a, bb);
            if (bias) {
                a += __bfloat162float(bias[p.QD + g * hd + i]);
                bb += __bfloat162float(bias[p.QD + g * hd + i + half]);
            }
            const float c = cs[2 * i], sn = cs[2 * i + 1];
            const __nv_bfloat16 k0 = __float2bfloat16_rn(a * c - bb * sn);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(bb * c + a * sn);
            new_k[i] = __bfloat162float(k0);   // the cache row itself is written after the stage (attention_flush_new_row)
            new_k[i + half] = __bfloat162float(k1);
            if (GT == 0) {
                const uint32_t j = i + half;
                *reinterpret_cast<__nv_bfloat16*>(stage_k + (i >> 6) * 128u + (i & 63u) * 2u) = k0;
                *reinterpret_cast<__nv_bfloat16*>(stage_k + (j >> 6) * 128u + (j & 63u) * 2u) = k1;
            }
        }
        for (uint32_t d = ctid; d < hd; d += SM::NCT) {
            float va, vb;
            poll_pair(p, s, vr + d, vr + d, qtag, va, vb);
            if (bias) va += __bfloat162float(bias[p.QD + p.KVD + g * hd + d]);
            const __nv_bfloat16 v0 = __float2bfloat16_rn(va);
            new_v[d] = __bfloat162float(v0);
            if (GT == 0) *reinterpret_cast<__nv_bfloat16*>(stage_v + (d >> 6) * 128u + (d & 63u) * 2u) = v0;
        }
    }
    consumer_bar<SM>();
    trace_stamp(p, s, cta, layer, 14, ctid);

    uint32_t first;
    if constexpr (SM::kTmem) {
        // stash mode: chunk i of the unit is chunk rc.start + i / 2 of pipeline i & 1 and sits in slot (that % 4) of the
        // pipeline; slot 4 T + q is read by warp 4 T + q, whose chunks are therefore eight apart, each in the next phase
        first = 2u * (((warp & 3u) - rc.start) & 3u) + (warp >> 2);
        wr.cslot = 0u;
        wr.cphase = KL_T_OHEAD ? (rc.n0 & 1u)   // K/V chunks this warp has read from its slot so far
                               : (((rc.start + (first >> 1)) >> 2) & 1u);
    } else {
        first = rc.first_chunk(warp, p.nslots);
    }
    if constexpr (GT == 0) {
        if (hd == 128) {
            if (G <= 4) attn_chunks_tc<128, true>(p, s, u, cta, warp, lane, first, rc, wr, q_s, comb, stage_k, stage_v);
            else attn_chunks_tc<128, false>(p, s, u, cta, warp, lane, first, rc, wr, q_s, comb, stage_k, stage_v);
        } else {
            if (G <= 4) attn_chunks_tc<64, true>(p, s, u, cta, warp, lane, first, rc, wr, q_s, comb, stage_k, stage_v);
            else attn_chunks_tc<64, false>(p, s, u, cta, warp, lane, first, rc, wr, q_s, comb, stage_k, stage_v);
        }
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
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 1);
            const uint32_t slot = warp * p.nsw + wr.cslot;
            mbar_wait(p, s, smem_u32(s.kv_bar(slot)), wr.cphase);
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 2);
            ring_advance_consume(p, wr);
            const uint8_t* kp = s.ring() + (size_t)slot * SLOT_BYTES;
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
            ring_release(p, s, wr, warp, lane);
            if (lane == 0) chunk_stamp(p, s, cta, rc.n0 + i, 3);
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
    trace_stamp(p, s, cta, layer, 15, ctid);
    consumer_bar<SM>();

    // merge the warps.  First one thread per (warp, head) turns that warp's maximum into its weight exp2(m - M_h);
    // then thread t owns (head, column) and adds the SM::NCW weighted terms in warp order.
    const uint32_t unit = u.bg * p.cps + u.ch;
    float* ftab = s.unit_part();   // [SM::NCW][G] weights, then [G] maxima (the unit table is idle outside the GEMV stages)
    if (ctid < SM::NCW * G) {
        const uint32_t w = ctid / G, h = ctid % G;
        float Mh = -INFINITY;
#pragma unroll
        for (int ww = 0; ww < SM::NCW; ++ww) Mh = fmaxf(Mh, comb[((size_t)ww * G + h) * (hd + 2) + hd]);
        ftab[w * G + h] = rescale(comb[((size_t)w * G + h) * (hd + 2) + hd], Mh);
        if (w == 0) ftab[SM::NCW * G + h] = Mh;
    }
    consumer_bar<SM>();
    for (uint32_t t = ctid; t < G * hd; t += SM::NCT) {
        const uint32_t h = t / hd, d = t % hd;
        float A = 0.f, Lsum = 0.f;
#pragma unroll
        for (int w = 0; w < SM::NCW; ++w) {
            const float* src = comb + ((size_t)w * G + h) * (hd + 2);
            const float c = ftab[w * G + h];
            A += src[d] * c;
            Lsum += src[hd + 1] * c;
        }
        if (nchunk == 1) {
            st_tw(p.o + (size_t)b * p.QD + (size_t)(g * G + h) * hd + d, A / Lsum, tag_of(p, cx, layer, TG_O));
        } else {
            const uint32_t ptag = tag_of(p, cx, layer, TG_PART);
            st_tw(p.part + ((size_t)unit * G + h) * hd + d, A, ptag);
            if (d == 0) {
                st_tw(p.part_ml + ((size_t)unit * G + h) * 2, ftab[SM::NCW * G + h], ptag);
                st_tw(p.part_ml + ((size_t)unit * G + h) * 2 + 1, Lsum, ptag);
            }
        }
    }
    trace_stamp(p, s, cta, layer, 3, ctid);
    // every unit of the group merges its slice of the outputs
    if (nchunk > 1) attn_merge(p, s, cx, u, layer, G, ctid, comb);
}

// Appends the K/V row of the position written by this step to the cache (16-byte stores).  Nothing in the running
// kernel reads that row from memory -- the unit that owns it works from the shared-memory copy -- so the store is
// kept off the stage's critical path: it runs after the CTA has signalled, and before the shared-memory copy is
// overwritten by the next stage's input vector.
template <class SM>
__device__ __forceinline__ void attention_flush_new_row(const Params& p, const SM& s, const StepCtx& cx, uint32_t layer,
                                                        uint32_t cta, uint32_t ctid) {
    const AttnUnit u = attn_unit(p, cta, cx.pos);
    if (!u.active || !u.has_new) return;
    const uint32_t hd = p.hd;
    const float* new_k = s.vec(p) + p.G * hd;
    const float* new_v = new_k + hd;
    const uint32_t per = hd / 8;
    if (ctid < 2 * per) {
        const uint32_t which = ctid / per, j = (ctid % per) * 8;
        const float* src = (which ? new_v : new_k) + j;
        uint4 v;
        v.x = (__float_as_uint(src[0]) >> 16) | (__float_as_uint(src[1]) & 0xffff0000u);
        v.y = (__float_as_uint(src[2]) >> 16) | (__float_as_uint(src[3]) & 0xffff0000u);
        v.z = (__float_as_uint(src[4]) >> 16) | (__float_as_uint(src[5]) & 0xffff0000u);
        v.w = (__float_as_uint(src[6]) >> 16) | (__float_as_uint(src[7]) & 0xffff0000u);
        __nv_bfloat16* row = const_cast<__nv_bfloat16*>(kv_head(p, layer, which, u.b, u.g)) + (size_t)u.pos * hd + j;
        *reinterpret_cast<uint4*>(row) = v;
    }
}

// Runs the attention stage and moves the ring cursor past the unit's chunks (also for CTAs without a unit).
template <int GT, class SM>
__device__ __forceinline__ void attention_stage_and_advance(const Params& p, const SM& s, const StepCtx& cx, uint32_t layer,
                                                            uint32_t cta, uint32_t ctid, uint32_t warp, uint32_t lane,
                                                            RingCursor& rc, WarpRing& wr) {
    attention_stage<GT>(p, s, cx, layer, cta, ctid, warp, lane, rc, wr);
    rc.advance(attn_unit(p, cta, cx.pos).nring, p.nslots);
}

}  // namespace kl
