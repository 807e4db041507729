// Kernels and C ABI of the kernel-looped decoder (see include/kl.h for the contract of every entry point).
//
// Kernel schedule per decode step (Section 2 of the paper, call-schedule figure):
//   looped    : embed -> decoder(layers 0..L-1, ONE persistent launch) -> classifier      (+ sampling)
//   per-layer : embed -> decoder(l), l = 0..L-1 (L launches of the same body) -> classifier (+ sampling)
//
// The decoder kernel is persistent: one CTA per SM, one producer warp that streams this CTA's share of every
// weight matrix through a shared-memory ring with TMA bulk copies, and NCW consumer warps.  Weight addresses do
// not depend on activations, so the producer runs ahead of the consumers across stage boundaries and, in looped
// mode, across layer boundaries: while the CTAs poll the tagged words that replace a kernel boundary, HBM keeps
// streaming the next stage's (next layer's) chunks until the ring is full.
#include "kl_device.cuh"
#include "kl_batched.cuh"
#include "kl_bloop.cuh"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <utility>

#include "../../include/kl.h"

namespace kl {

// ------------------------------------------------------------------------------------------------ kernels

// Step numbers behind the tags.  A tag holds (step * L + layer) in 28 bits, so step numbers are reused after
// 2^28 / L steps; a tagged word that is not rewritten in every step (a split-K slot above the current split count)
// could then meet its own old tag.  Before that can happen -- when the next step number reaches step_wrap(L), at a
// launch boundary -- every tagged area is cleared and the numbering restarts at 1.  The margin covers the steps one
// launch may take without passing such a boundary (TOKENS_PER_LAUNCH) and the look-ahead of the tags (step + 1).
constexpr uint32_t STEP_WRAP_MARGIN = 260u;
__host__ __device__ __forceinline__ uint32_t step_wrap(uint32_t L) { return (1u << 28) / L - STEP_WRAP_MARGIN; }

// All tagged words of the handle to zero (zero is no tag).  Called by every thread of ONE block at a launch boundary of
// the chain: nothing else reads or writes these areas then.  The caller puts a block barrier behind it.
__device__ __noinline__ void clear_tagged(const Params& p, uint32_t tid, uint32_t nthreads) {
    const uint32_t nq = p.QD + 2u * p.KVD, npart = p.P * p.G * p.hd, nml = p.P * p.G * 2u;
    for (uint32_t i = tid; i < p.H; i += nthreads) {
        st_tw(p.xa + i, 0.f, 0u);
        st_tw(p.xb + i, 0.f, 0u);
    }
    for (uint32_t i = tid; i < nq; i += nthreads) st_tw(p.qkv + i, 0.f, 0u);
    for (uint32_t i = tid; i < p.QD; i += nthreads) st_tw(p.o + i, 0.f, 0u);
    for (uint32_t i = tid; i < npart; i += nthreads) st_tw(p.part + i, 0.f, 0u);
    for (uint32_t i = tid; i < nml; i += nthreads) st_tw(p.part_ml + i, 0.f, 0u);
}

__global__ void __launch_bounds__(256) kl_embed_kernel(const Params p) {
    const uint32_t b = 0u, tid = threadIdx.x;   // b: slot of the sequence in the scratch vectors
    int32_t tok = p.tokens[p.b0];
    const int32_t pos = p.positions[p.b0];
    // the launch for the first sequence checks the whole batch, so that a bad entry anywhere makes the step a no-op
    // before any sequence has been decoded
    if (p.b0 == 0u)
        for (uint32_t i = tid; i < p.B; i += blockDim.x) {
            const int32_t t = p.tokens[i], q = p.positions[i];
            if (t < 0 || t >= (int32_t)p.V || q < 0 || q >= (int32_t)p.max_ctx) atomicCAS(p.status, 0, ERR_OUT_OF_RANGE);
        }
    if (tok < 0 || tok >= (int32_t)p.V) tok = 0;
    const __nv_bfloat16* row = p.embed + (size_t)tok * p.H;
    // one more sequence on this handle: every tag of this launch sequence differs from all earlier ones
    uint32_t step = *p.step_dev + 1u;   // every thread reads the word; thread 0 writes it behind the barrier
    const bool wrap = step >= step_wrap(p.L);
    if (wrap) {
        clear_tagged(p, tid, blockDim.x);
        step = 1u;
    }
    __syncthreads();
    if (tid == 0) *p.step_dev = step;
    const uint32_t xtag = tag_from(step, p.L, 0, TG_XA);
    for (uint32_t i = tid; i < p.H; i += blockDim.x) st_tw(p.xa + (size_t)b * p.H + i, __bfloat162float(row[i]), xtag);
    // RoPE table of this step: angle in double so that large positions keep their phase
    for (uint32_t i = tid; i < p.hd / 2; i += blockDim.x) {
        double sn, cs;
        sincos((double)pos * p.inv_freq[i], &sn, &cs);
        p.rope_cs[((size_t)b * (p.hd / 2) + i) * 2] = (float)cs;
        p.rope_cs[((size_t)b * (p.hd / 2) + i) * 2 + 1] = (float)sn;
    }
    if (b == 0)
        for (uint32_t i = tid; i < p.L; i += blockDim.x) p.counters[i] = 0u;
}

// The attention half of a layer as one call: RoPE, the unit's ring chunks, the merges, the deferred cache append.
template <class SM>
__device__ __noinline__ void attention_block(const Params& p, const SM& s, const StepCtx& cx, uint32_t l, uint32_t cta,
                                             uint32_t ctid, uint32_t warp, uint32_t lane, RingCursor& rc, WarpRing& wr) {
    if (!SM::kCudaCoreAttn || p.attn_tc) {   // kernels without the CUDA-core loops are launched only when this one runs
        attention_stage_and_advance<0>(p, s, cx, l, cta, ctid, warp, lane, rc, wr);
    } else switch (p.G) {
        case 1: attention_stage_and_advance<1>(p, s, cx, l, cta, ctid, warp, lane, rc, wr); break;
        case 2: attention_stage_and_advance<2>(p, s, cx, l, cta, ctid, warp, lane, rc, wr); break;
        case 4: attention_stage_and_advance<4>(p, s, cx, l, cta, ctid, warp, lane, rc, wr); break;
        default: attention_stage_and_advance<8>(p, s, cx, l, cta, ctid, warp, lane, rc, wr); break;
    }
    // the row written by this step is copied from the workspace to the cache here; the next vector load starts with
    // a CTA barrier, so the workspace is not overwritten before this copy has read it
    attention_flush_new_row(p, s, cx, l, cta, ctid);
}

// Set-up every persistent kernel starts with: the ring's barriers, the abort flag, the unit table.  False: an earlier
// kernel of this step flagged bad input and the launch is a no-op.
template <class SM>
__device__ __forceinline__ bool cta_begin(const Params& p, const SM& s, uint32_t tid, const float* rope) {
    if (tid == 0) {
        // step number and position as the launch finds them: read before any CTA can have finished a token
        s.ctx()->step = ld_step(p.step_dev);
        s.ctx()->pos = (uint32_t)p.positions[p.b0];
        s.ctx()->rope_cs = rope;
        s.ctx()->wait_ns = p.wait_ns;
        s.ctx()->status = p.status;
        if constexpr (SM::kMoe) s.moe()->seq = 0u;
        for (uint32_t i = 0; i < p.nslots * p.nsw; ++i) {
            mbar_init(smem_u32(&s.full()[i]), 1);
            mbar_init(smem_u32(&s.empty()[i]), SM::kTmem ? 2 : 1);   // stash mode: the stash thread and the slot's reader
        }
        if constexpr (SM::kTmem) {
            for (uint32_t i = 0; i < 2u * T_NREG; ++i) {
                mbar_init(smem_u32(&s.tfull()[i]), 1);
                mbar_init(smem_u32(&s.tfree()[i]), 4);   // the four warps of the team
            }
            for (uint32_t i = 0; i < 2u * T_NSP; ++i) mbar_init(smem_u32(&s.kvready()[i]), 1);
            mbar_init(smem_u32(&s.tdone()[0]), 1);
            mbar_init(smem_u32(&s.tdone()[1]), 1);
        }
        *s.abort_flag() = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (tid < UNIT_SLOTS) s.unit_cnt()[tid] = 0;
    if constexpr (SM::kTmem) {
        if (tid < 2u * T_USLOTS) s.t_ucnt()[tid] = 0;
    }
    if (__syncthreads_or(*p.status != 0)) return false;   // the same answer in every thread
    if constexpr (SM::kTmem) {
        // all of tensor memory (one CTA per SM; the tensor-core kernels of the batched path never overlap this one)
        if ((tid >> 5) == (uint32_t)SM::NCW + 1u) tm_alloc(smem_u32(s.tbase()), 512u);
        tm_fence_before();
        __syncthreads();
        tm_fence_after();
    }
    return true;
}
// ... and ends with in stash mode: every warp has left its loop; the warp that allocated tensor memory releases it.
template <class SM>
__device__ __forceinline__ void cta_end(const SM& s, uint32_t tid) {
    if constexpr (SM::kTmem) {
        tm_fence_before();
        __syncthreads();
        tm_fence_after();
        if ((tid >> 5) == (uint32_t)SM::NCW + 1u) tm_dealloc(*s.tbase(), 512u);
    }
}

// ONE stage of one layer on the consumer warps -- the only copy of the stage sequence; every persistent kernel calls
// it from the single call site of its loop, so the GEMV loop is inlined into the kernel's own frame and the cold
// parts (vector loads with their polls, the attention block) are calls made between stages, when nothing is live.
//   l < L : stage st of decoder layer l (QKV, attention, O, gate/up, down)
//   l == L: the classifier, as stage 0 of one more pass (one more stage on the same ring, same code)
// xa_slot: tag slot under which the hidden state entering stage 0 was published (TG_XA; TG_NEXT for an embedding
// written inside the running launch).  ctr_target: value of the layer's gate/up counter when all CTAs have signalled.
template <class SM>
__device__ __forceinline__ void run_stage(const Params& p, const SM& s, uint32_t l, uint32_t st,
                                          uint32_t xa_slot, uint32_t ctr_target, uint32_t cta, uint32_t ctid, uint32_t warp,
                                          uint32_t lane, RingCursor& rc, WarpRing& wr, TCur& tc) {
    const StepCtx& cx = *s.ctx();
    stage_jitter(p, s, cta, cx.step, l, st);
    const size_t lo = (size_t)l * p.layer_stride;
    const bool cls = l == p.L;
    // test hook: the results of one stage of layer 0 get a tag nobody waits for
    const int skip = (l == 0) ? p.skip_stage : -1;
    const uint32_t bad = 0x2u;
    GemvOut out = {nullptr, nullptr, nullptr, 0u};
    int plan = PL_QKV, ep = EP_STORE;
    const float* xsrc = nullptr;
    float xscale = 1.f;   // RMSNorm's normaliser of the stage's input vector, applied to the stage's outputs
    if (st == ST_QKV) {
        // RMSNorm + QKV projection (classifier: final RMSNorm + W_lm).  The poll on xa's tags is the wait for the
        // previous layer (or the embedding).
        trace_stamp(p, s, cta, l, 0, ctid);
        xscale = load_vec(p, s, p.xa, p.H, tag_of(p, cx, l, xa_slot), true, cls ? p.gf : p.g1 + lo, ctid);
        trace_stamp(p, s, cta, l, 1, ctid);
        if (cls) {
            out = {nullptr, p.logits, nullptr, 0u};
            plan = PL_LM;
        } else {
            out = {p.qkv, nullptr, nullptr, skip == ST_QKV ? bad : tag_of(p, cx, l, TG_QKV)};
        }
    } else if (st == ST_ATTN) {
        trace_stamp(p, s, cta, l, 2, ctid);
        // RoPE, split-K attention, merge.  Each unit polls the q (k, v) rows it needs.
        if constexpr (SM::kTmem) {
            // chunks so far in this warp's pipeline: behind the head of W_o where that has been streamed ahead
            uint32_t c0 = tc.c;
            if (tc.ohead) {
                const CtaRange co = cta_units(p.plan[PL_O], cta, p.P);
                c0 += t_count(tc.uc, t_o_head(p.plan[PL_O], co.u1 - co.u0), warp >> 2) * p.plan[PL_O].npieces;
            }
            RingCursor ac = {c0, tc.kv};
            attention_block(p, s, cx, l, cta, ctid, warp, lane, ac, wr);
            const uint32_t nring = attn_unit(p, cta, cx.pos).nring;
            const uint32_t first = 2u * (((warp & 3u) - c0) & 3u) + (warp >> 2);   // as in attention_stage
            if (first < nring) tc.kv += (nring - first + 7u) >> 3;
            tc.c += (nring + ((warp >> 2) == 0u ? 1u : 0u)) >> 1;
        } else {
            attention_block(p, s, cx, l, cta, ctid, warp, lane, rc, wr);
        }
        trace_stamp(p, s, cta, l, 4, ctid);
        return;
    } else if (st == ST_O) {
        // output projection + residual (xa -> xb).  The poll on o's tags waits for the attention units.
        load_vec(p, s, p.o, p.QD, skip == ST_ATTN ? bad : tag_of(p, cx, l, TG_O), false, nullptr, ctid);
        trace_stamp(p, s, cta, l, 6, ctid);
        out = {p.xb, nullptr, p.xa, skip == ST_O ? bad : tag_of(p, cx, l, TG_XB)};
        plan = PL_O;
        ep = EP_RESIDUAL;
    } else if (st == ST_GU) {
        trace_stamp(p, s, cta, l, 7, ctid);
        // RMSNorm + gate/up projections + SwiGLU
        xscale = load_vec(p, s, p.xb, p.H, tag_of(p, cx, l, TG_XB), true, p.g2 + lo, ctid);
        if constexpr (SM::kMoe) moe_router(p, s, l, xscale, ctid);   // which experts, with which gate weights
        trace_stamp(p, s, cta, l, 9, ctid);
        out = {nullptr, p.h, nullptr, 0u};
        plan = PL_GU;
        ep = EP_SWIGLU;
    } else {
        // down projection + residual (xb -> xa of the next layer).  h is plain fp32 read per warp and per column piece
        // straight from L2 into registers (too wide for shared memory): its readiness is a counter, signalled with
        // release at the end of the gate/up stage and awaited with acquire here
        stage_wait(p, s, p.counters + l, ctr_target, ctid);
        trace_stamp(p, s, cta, l, 12, ctid);
        out = {p.xa, nullptr, p.xb, skip == ST_D ? bad : tag_of(p, cx, l + 1, TG_XA)};
        plan = PL_D;
        ep = EP_RESIDUAL;
        xsrc = p.h;
        if constexpr (SM::kTmem) load_plain_vec(p, s, p.h, p.F, ctid);   // stash mode multiplies against shared memory
    }
    if constexpr (SM::kMoe) {
        if (st == ST_GU || st == ST_D) {
            // the stage runs over the chosen experts: their (gate, up) rows one expert after the other; in the down
            // projection their matrices side by side, the input vector being the experts' (gated) SwiGLU outputs
            GemvPlan pm = p.plan[plan];
            if (st == ST_GU) {
                pm.R *= p.top_k;
                pm.nunits *= p.top_k;
            } else {
                pm.nseg = p.top_k;
            }
            gemv_stage(p, s, pm, ep, out, cta, warp, lane, rc, wr, xsrc, xscale);
        } else {
            gemv_stage(p, s, p.plan[plan], ep, out, cta, warp, lane, rc, wr, xsrc, xscale);
        }
    } else if constexpr (SM::kTmem) {
        gemv_stage_t(p, s, p.plan[plan], ep, out, cta, warp, lane, tc, xscale);
    } else {
        gemv_stage(p, s, p.plan[plan], ep, out, cta, warp, lane, rc, wr, xsrc, xscale);
    }
    if (st == ST_GU) {
        stage_signal<SM>(p.counters + l, ctid, skip == ST_GU);
        trace_stamp(p, s, cta, l, 10, ctid);
    } else if (st == ST_D) {
        trace_stamp(p, s, cta, l, 13, ctid);
    }
}

// Stages [sbeg, send) of layers [l0, l1) of the decoder.  All five stages of all L layers is the looped kernel; all
// stages of one layer the per-layer launch; one stage of one layer the per-stage launch (the schedule with a kernel
// boundary after every operator group).
template <bool TR, bool MOE, int TM, bool CC>
__global__ void __launch_bounds__(NTHREADS, 1) kl_decoder_kernel(const __grid_constant__ Params p, uint32_t l0, uint32_t l1,
                                                                 uint32_t sbeg, uint32_t send) {
    using SM = SmemT<TR, MOE, TM, CC>;
    const SM s;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x;
    if (!cta_begin(p, s, tid, p.rope_cs)) return;   // an earlier kernel of this step flagged bad input: the step is a no-op
    if (warp >= (uint32_t)SM::NCW) {
        // producer warp: one thread streams the CTA's chunk sequence into the ring (stash mode: two more warps, one
        // thread each, move the chunks on into tensor memory)
        if (lane == 0) produce_decoder(p, s, cta, l0, l1, sbeg, send, warp - SM::NCW);
    } else {
        WarpRing wr = ring_begin();
        RingCursor rc = {0u, 0u};
        TCur tc = {0u, 0u, 0u, 0u, (sbeg <= ST_ATTN && send > ST_O) ? 1u : 0u, 0u};
        for (uint32_t l = l0; l < l1; ++l)
            for (uint32_t st = sbeg; st < send; ++st) run_stage(p, s, l, st, TG_XA, p.P, cta, tid, warp, lane, rc, wr, tc);
    }
    cta_end(s, tid);
}

// Classifier block: logits = W_lm rmsnorm(x; g_f).  Same ring, one stage, no inter-CTA dependency.
template <int TM>
__global__ void __launch_bounds__(NTHREADS, 1) kl_classifier_kernel(const __grid_constant__ Params p) {
    using SM = SmemT<false, false, TM>;
    const SM s;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x;
    if (!cta_begin(p, s, tid, p.rope_cs)) return;
    if (warp >= (uint32_t)SM::NCW) {
        if (lane == 0) produce_classifier(p, s, cta, warp - SM::NCW);
    } else {
        WarpRing wr = ring_begin();
        RingCursor rc = {0u, 0u};
        TCur tc = {0u, 0u, 0u, 0u, 0u, 0u};
        run_stage(p, s, p.L, ST_QKV, TG_XA, p.P, cta, tid, warp, lane, rc, wr, tc);
    }
    cta_end(s, tid);
}

// Sampling block (greedy): lowest index among the maxima; then advance the position.  ARGMAX_BLOCKS CTAs per
// sequence scan slices of the row; the last one to finish (ticket) reduces the partial results.
constexpr int ARGMAX_BLOCKS = 64;

__device__ __forceinline__ void argmax_merge(float& bv, uint32_t& bi, float ov, uint32_t oi) {
    if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
    }
}

__global__ void __launch_bounds__(256) kl_argmax_kernel(const float* logits, uint32_t V, int32_t* tokens, int32_t* positions,
                                                        float* part_val, uint32_t* part_idx, uint32_t* tickets) {
    __shared__ float sv[8];
    __shared__ uint32_t si[8];
    __shared__ uint32_t last;
    const uint32_t b = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x;
    const float* row = logits + (size_t)b * V;
    const uint32_t per = (V + ARGMAX_BLOCKS - 1) / ARGMAX_BLOCKS;
    const uint32_t i0 = blk * per, i1 = min(V, i0 + per);
    float bv = -INFINITY;
    uint32_t bi = 0xffffffffu;
    for (uint32_t i = i0 + tid; i < i1; i += blockDim.x) argmax_merge(bv, bi, row[i], i);
    for (int o = 16; o > 0; o >>= 1)
        argmax_merge(bv, bi, __shfl_xor_sync(0xffffffffu, bv, o), __shfl_xor_sync(0xffffffffu, bi, o));
    if ((tid & 31) == 0) {
        sv[tid >> 5] = bv;
        si[tid >> 5] = bi;
    }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) argmax_merge(bv, bi, sv[w], si[w]);
        part_val[b * ARGMAX_BLOCKS + blk] = bv;
        part_idx[b * ARGMAX_BLOCKS + blk] = bi;
        last = (atom_add_acq_rel(tickets + b, 1u) == ARGMAX_BLOCKS - 1) ? 1u : 0u;
    }
    __syncthreads();
    if (!last) return;
    if (tid < 32) {
        bv = -INFINITY;
        bi = 0xffffffffu;
        for (uint32_t j = tid; j < ARGMAX_BLOCKS; j += 32)
            argmax_merge(bv, bi, __ldcg(part_val + b * ARGMAX_BLOCKS + j), __ldcg(part_idx + b * ARGMAX_BLOCKS + j));
        for (int o = 16; o > 0; o >>= 1)
            argmax_merge(bv, bi, __shfl_xor_sync(0xffffffffu, bv, o), __shfl_xor_sync(0xffffffffu, bi, o));
        if (tid == 0) {
            tokens[b] = (int32_t)(bi == 0xffffffffu ? 0u : bi);
            positions[b] += 1;
            tickets[b] = 0u;  // ready for the next call (calls on one handle do not overlap)
        }
    }
}

// ------------------------------------------------------------------------------------------------ tokens per launch
// The paper's looped schedule still pays four calls per token: embedding, the looped decoder, classifier, sampling
// (Section 2).  kl_token_kernel is all four for one sequence, and for K consecutive tokens: the decoder layers and the
// classifier as consecutive stages of one persistent kernel (the ring runs on from the last down projection into
// W_lm), then greedy sampling -- every CTA reduces the logits rows it has just produced, the CTA that draws the token's
// last ticket reduces the per-CTA results, advances token and position and writes the NEXT token's embedding; all other
// CTAs are by then polling for exactly those words, with the first weight tiles of the next token already in their
// rings -- no launch boundary, no pipeline restart.  Behind the launch's last token that CTA also keeps the final hidden
// state for kl_read_hidden and leaves the rotary table and the step counter of the next token, so that the next launch
// starts at its first layer at once (K = 1: one launch per token).
// What changes from token to token inside the launch is arithmetic (position and step number advance by one) except
// the rotary tables, which kl_token_plan_kernel lays out beforehand, one per token.  Counters that are zeroed between
// launches count on instead: the gate/up counter of a layer reaches P * (k + 1) during token k, and so does the
// sampling ticket.
// Tag slot of an embedding written INSIDE the launch.  The hidden state that enters the classifier carries
// (step, layer L, TG_XA), which is the same number as (step + 1, layer 0, TG_XA): across a launch boundary that is
// harmless, inside the launch the CTAs polling for the next embedding would take the old hidden state for it.
constexpr uint32_t TG_NEXT = 5;
struct TokenParams {
    int32_t* tokens;        // [1] in: the token the launch starts from (already embedded); out: the token after the last step
    int32_t* positions;     // [1] advanced by K
    float* part_val;        // [P] per-CTA maxima
    uint32_t* part_idx;     // [P] and their indices
    uint32_t* ticket;       // zero between launches
    float* hidden;          // [H] final hidden state of the launch's last step
    int32_t* out_tokens;    // [K] the token picked after each step, or null
    uint32_t K;             // tokens of this launch
    const float* rope;      // [K][head_dim] rotary tables of the K positions (K = 1: the handle's own table)
};

// Rotary tables of the K positions of a launch, and the check that all of them lie inside the cache.
__global__ void kl_token_plan_kernel(const __grid_constant__ Params p, float* rope_arr, uint32_t K) {
    const int32_t pos0 = p.positions[0];
    if (pos0 < 0 || (uint32_t)pos0 + K > p.max_ctx) {   // every position of the launch has to be inside the cache
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ERR_OUT_OF_RANGE);
        return;
    }
    const uint32_t half = p.hd / 2;
    for (uint32_t i = threadIdx.x; i < K * half; i += blockDim.x) {
        const uint32_t k = i / half, j = i % half;
        double sn, cs;
        sincos((double)(pos0 + (int32_t)k) * p.inv_freq[j], &sn, &cs);
        rope_arr[(size_t)k * p.hd + 2 * j] = (float)cs;
        rope_arr[(size_t)k * p.hd + 2 * j + 1] = (float)sn;
    }
}

template <class SM>
__device__ __forceinline__ void produce_tokens(const Params& p, const SM& s, uint32_t cta, const TokenParams& t, uint32_t role = 0u) {
    RingProd r = ring_prod_begin(role);
    const uint32_t step0 = ld_step(p.step_dev), pos0 = (uint32_t)p.positions[0];
    uint32_t routed = 0, ex[MAX_TOP_K] = {0u, 0u, 0u, 0u};   // mixture of experts: layers routed so far, the chosen experts
    uint32_t ohead = 0u;   // stash mode: the head of W_o goes ahead of the K/V chunks
    if constexpr (SM::kTmem) {
        const CtaRange co = cta_units(p.plan[PL_O], cta, p.P);
        ohead = t_o_head(p.plan[PL_O], co.u1 - co.u0);
    }
    for (uint32_t k = 0; k < t.K && !r.aborted; ++k) {
        const AttnUnit u = attn_unit(p, cta, pos0 + k);
        for (uint32_t l = 0; l < p.L && !r.aborted; ++l) {
            const size_t lo = (size_t)l * p.layer_stride;
            produce_matrix(p, s, r, p.plan[PL_QKV], p.wqkv + lo, cta);
            if (k > 0 && l == 0 && role == 0u) {
                // The cache rows of the previous token are read by this token's copies: none is requested before the
                // previous token is complete in every CTA, which the first word of this token's embedding says (it
                // keeps its tag until the first down projection of this token, which cannot start before this point
                // has been passed in every CTA).  Weight tiles do not wait: the ring is full of them by now.
                const uint32_t want = tag_from(step0 + k, p.L, 0, TG_NEXT);
                PollGuard g = {0ull, 0u, 700};
                while (ld_tw(p.xa).tag != want) {
                    if (!poll_continue(p, s, g)) {
                        r.aborted = true;
                        break;
                    }
                }
                __threadfence();
                asm volatile("fence.proxy.async;" ::: "memory");
                if (r.aborted) break;
            }
            if (ohead) produce_matrix(p, s, r, p.plan[PL_O], p.wo + lo, cta, 0u, ohead);
            produce_attention(p, s, r, u, l);
            produce_matrix(p, s, r, p.plan[PL_O], p.wo + lo, cta, ohead);
            if constexpr (SM::kMoe) {
                if (!moe_wait_route(p, s, ++routed, ex)) r.aborted = true;   // the experts of this layer are known now
                if (!r.aborted) produce_matrix_moe(p, s, r, p.plan[PL_GU], p.wgu + lo, cta, ex, false);
                if (!r.aborted) produce_matrix_moe(p, s, r, p.plan[PL_D], p.wd + lo, cta, ex, true);
            } else {
                produce_matrix(p, s, r, p.plan[PL_GU], p.wgu + lo, cta);
                produce_matrix(p, s, r, p.plan[PL_D], p.wd + lo, cta);
            }
        }
        if (!r.aborted) produce_matrix(p, s, r, p.plan[PL_LM], p.wlm, cta);
    }
    produce_drain(p, s, r);
}

// Sampling at the end of token k (step cx.step, position cx.pos), out of line: once per token.  Every CTA reduces the
// logits rows it has just produced; the CTA that draws the token's last ticket reduces the per-CTA results, records the
// token and writes the next embedding.  false: that was the last token of the launch, or a wait of this launch gave up
// -- in which case token, position and the next embedding are left alone (the step's outputs are meaningless; the
// chain has to be restarted).
template <class SM>
__device__ __noinline__ bool sample_token(const Params& p, const SM& s, const TokenParams& t, uint32_t k,
                                          uint32_t cta, uint32_t ctid, uint32_t warp, uint32_t lane) {
    const bool final = k + 1u == t.K;
    const StepCtx cx = *s.ctx();   // a copy: the shared one moves on to the next token below
    // ---- greedy sampling: this CTA's rows first
    const GemvPlan& plm = p.plan[PL_LM];
    asm volatile("fence.proxy.async;" ::: "memory");   // the cache rows this thread appended: readable by later bulk copies
    consumer_bar<SM>();   // the rows this CTA stored are visible to all of its threads
    float* sv = s.unit_part();                                           // [NCW] maxima, then [NCW] indices, then flags
    uint32_t* si = reinterpret_cast<uint32_t*>(s.unit_part()) + SM::NCW;
    // [0] this CTA drew the last ticket, [1] token, [2] position, [3] next step number, [4] stop: a wait of this launch gave up
    volatile uint32_t* sh = reinterpret_cast<volatile uint32_t*>(s.unit_part()) + 2 * SM::NCW;
    const CtaRange cr = cta_units(plm, cta, p.P);
    const uint32_t r0 = cr.u0 * plm.rpc, r1 = min(cr.u1 * plm.rpc, p.V);
    float bv = -INFINITY;
    uint32_t bi = 0xffffffffu;
    for (uint32_t i = r0 + ctid; i < r1; i += SM::NCT) argmax_merge(bv, bi, p.logits[i], i);
    for (int o = 16; o > 0; o >>= 1)
        argmax_merge(bv, bi, __shfl_xor_sync(0xffffffffu, bv, o), __shfl_xor_sync(0xffffffffu, bi, o));
    if (lane == 0) {
        sv[warp] = bv;
        si[warp] = bi;
    }
    consumer_bar<SM>();
    if (ctid == 0) {
        for (uint32_t w = 1; w < (uint32_t)SM::NCW; ++w) argmax_merge(bv, bi, sv[w], si[w]);
        t.part_val[cta] = bv;
        t.part_idx[cta] = bi;
        sh[0] = (atom_add_acq_rel(t.ticket, 1u) == p.P * (k + 1u) - 1u) ? 1u : 0u;
        sh[4] = (*s.abort_flag() != 0 || __ldcg(p.status) != 0) ? 1u : 0u;
    }
    consumer_bar<SM>();
    const bool last_cta = sh[0] != 0u, stop = sh[4] != 0u;
    if (last_cta && stop) {
        if (ctid == 0) *t.ticket = 0u;
    } else if (last_cta) {
        // all logits of this token are written.  Next token, next position, the next embedding.
        if (warp == 0) {
            bv = -INFINITY;
            bi = 0xffffffffu;
            for (uint32_t j = lane; j < p.P; j += 32) argmax_merge(bv, bi, __ldcg(t.part_val + j), __ldcg(t.part_idx + j));
            for (int o = 16; o > 0; o >>= 1)
                argmax_merge(bv, bi, __shfl_xor_sync(0xffffffffu, bv, o), __shfl_xor_sync(0xffffffffu, bi, o));
            if (lane == 0) {
                const uint32_t tok = bi == 0xffffffffu ? 0u : bi;
                const int32_t pos = (int32_t)cx.pos + 1;
                t.tokens[0] = (int32_t)tok;
                t.positions[0] = pos;
                if (t.out_tokens != nullptr) t.out_tokens[k] = (int32_t)tok;
                if (final) *t.ticket = 0u;   // ready for the next launch
                if (final && pos >= (int32_t)p.max_ctx) atomicCAS(p.status, 0, ERR_OUT_OF_RANGE);   // the next step would leave the cache
                sh[1] = tok;
                sh[2] = (uint32_t)pos;
            }
        }
        consumer_bar<SM>();
        uint32_t next_step = cx.step + 1u;
        if (final) {   // what the next launch needs: hidden state kept, rotary table, counters at zero, step number
            for (uint32_t i = ctid; i < p.H; i += SM::NCT) t.hidden[i] = ld_tw(p.xa + i).v;   // before xa is overwritten below
            for (uint32_t i = ctid; i < p.hd / 2; i += SM::NCT) {
                double sn, cs;
                sincos((double)sh[2] * p.inv_freq[i], &sn, &cs);
                p.rope_cs[2 * i] = (float)cs;
                p.rope_cs[2 * i + 1] = (float)sn;
            }
            for (uint32_t i = ctid; i < p.L; i += SM::NCT) p.counters[i] = 0u;
            consumer_bar<SM>();
            if (next_step >= step_wrap(p.L)) {   // every other CTA has left its last stage: the step numbers start over
                clear_tagged(p, ctid, SM::NCT);
                next_step = 1u;
                consumer_bar<SM>();
            }
            if (ctid == 0) *p.step_dev = next_step;
        }
        const __nv_bfloat16* row = p.embed + (size_t)sh[1] * p.H;
        // the next launch expects the usual tag, the next token of this launch the one of its own
        const uint32_t xtag = tag_from(next_step, p.L, 0, final ? (uint32_t)TG_XA : TG_NEXT);
        __threadfence();   // release side of the token boundary (the producers' poll above is the acquire side)
        for (uint32_t i = ctid; i < p.H; i += SM::NCT) st_tw(p.xa + i, __bfloat162float(row[i]), xtag);
    }
    if (ctid == 0) {   // the next token of the launch: one step and one position further, the next rotary table
        s.ctx()->step = cx.step + 1u;
        s.ctx()->pos = cx.pos + 1u;
        s.ctx()->rope_cs = cx.rope_cs + p.hd;
    }
    consumer_bar<SM>();   // the flags above are read before the next stage reuses the area
    return !stop && !final;
}

// K tokens of one sequence per launch (K = 1: one launch per token).  ONE loop over (token, layer) pairs, the
// classifier being the only stage of a layer L behind the decoder layers and the sampling a call behind that: with a
// loop over tokens around the loop over layers the compiler holds more in registers through the stage code.
template <bool TR, bool MOE, int TM, bool CC>
__global__ void __launch_bounds__(NTHREADS, 1) kl_token_kernel(const __grid_constant__ Params p, const __grid_constant__ TokenParams t) {
    using SM = SmemT<TR, MOE, TM, CC>;
    const SM s;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x;
    if (!cta_begin(p, s, tid, t.rope)) return;
    if (warp >= (uint32_t)SM::NCW) {
        if (lane == 0) produce_tokens(p, s, cta, t, warp - SM::NCW);
    } else {
        WarpRing wr = ring_begin();
        RingCursor rc = {0u, 0u};
        TCur tc = {0u, 0u, 0u, 0u, 1u, 0u};
        uint32_t k = 0, l = 0;
#pragma unroll 1
        for (;;) {
            const bool cls = l == p.L;
            for (uint32_t st = 0; st < (cls ? 1u : 5u); ++st)
                run_stage(p, s, l, st, (k > 0 && l == 0) ? TG_NEXT : (uint32_t)TG_XA, p.P * (k + 1u), cta, tid, warp, lane, rc, wr, tc);
            if (cls) {
                if (!sample_token(p, s, t, k, cta, tid, warp, lane)) break;
                ++k;
                l = 0;
            } else {
                ++l;
            }
        }
    }
    cta_end(s, tid);
}

}  // namespace kl

// ------------------------------------------------------------------------------------------------ host side

using namespace kl;

struct kl_handle {
    kl_model_desc desc;
    Params prm;
    int mode;
    int mode_explicit;     // kl_set_mode has been called: batches follow `mode` too (until then they take the per-operator schedule)
    int device;
    int num_sms;
    size_t smem_bytes;
    uint8_t* weights;  // arena
    uint8_t* scratch;  // arena
    size_t weight_bytes, scratch_bytes;
    // scratch sub-allocations used by the host-buffer entry point
    int32_t* stage_tokens;
    int32_t* stage_positions;
    float* stage_logits;
    float* argmax_val;
    float* hidden_all;     // [max_batch][H] hidden states of the sequences of the latest batched step
    // batched (tensor-core) path
    int bt_ok;             // 1: available for this shape
    int bl_ok;             // 1: the looped kernel of the batched path can be resident (cooperative launch)
    uint32_t* bbar;        // grid-barrier counters of the looped kernel: 16 per layer launch + 16
    int use_bt;            // 1 (default): batches take it; 0: sequence after sequence on the batch-1 kernels
    int use_pdl;           // 1 (default): the kernels of a batched step are launched with programmatic stream serialisation
    int use_stream;        // 1 (default): stream schedule for the projections of the layers; 0: (row tile, K split) items
    float* bx;             // [32][H] hidden states of the batch (== hidden_all)
    __nv_bfloat16* bxop[3];   // operands [64][H], [64][QD], [64][F]: rows 0..31 hi halves, 32..63 lo halves
    float* bssq;           // [32][BV_MAX_CHUNKS] partial sums of squares of the residual stream
    float* bpart;          // partial sums of the projection in flight
    float* bq;             // [32][QD] rotated queries
    float* bao;            // attention partial outputs
    float* baml;           // attention partial (max, sum) pairs
    CUtensorMap bmap_x[3];   // operand buffer seen as [64][H], [64][QD], [64][F]
    CUtensorMap bmap_w[5];   // QKV, O, gate/up, down, classifier
    CUtensorMap bmap_wl[5];  // last column piece of the matrices stored in chunk order
    uint32_t bsplit[5];      // K splits of the five projections
    // kl_decode_step_host: one batched step (323 launches at 32 layers) kept as an instantiated CUDA graph, so that the
    // host cost of the launches is paid once and not between two synchronisations of every step
    cudaStream_t cap_stream;       // capture only; nothing ever executes on it
    cudaGraphExec_t bgraph;        // null: none cached
    void* bgraph_kv;               // the buffers the graph was captured for
    const void* bgraph_tok;
    const void* bgraph_pos;
    void* bgraph_logits;
    uint32_t bgraph_batch;
    uint64_t bgraph_launches;      // kernels per replay
    uint32_t last_batch;
    int hidden_is_copy;    // 1: the latest step left its final hidden state in hidden_all (kl_decode_greedy, batch 1)
    const void* chain_tok; // kl_decode_greedy, batch 1: the token buffer whose next embedding the latest launch prepared
                           // (null: no chain to continue -- another decode call came in between)
    float* tok_val;        // [P] per-CTA maxima of kl_token_kernel
    uint32_t* tok_idx;     // [P]
    uint32_t* tok_ticket;
    int token_ok;          // kl_token_kernel can be resident
    int32_t* plan_out;     // [TOKENS_PER_LAUNCH] picked tokens of the host-buffer entry point
    float* plan_rope;      // [TOKENS_PER_LAUNCH][head_dim]
    uint32_t* argmax_idx;
    uint32_t* argmax_tickets;
    uint64_t launches;
    uint64_t loaded_layer_mask_count;  // number of (tensor, layer) pairs loaded
    uint8_t* loaded;                   // [12][L] flags (host)
    int pending_skip_stage;
    int use_tc_attention;
    int stash;             // 1: the batch-1 kernels run in stash mode (ring -> TMEM -> registers; plans cut for it)
    void* encode_tiled;  // cuTensorMapEncodeTiled, resolved through the runtime (no link against libcuda)
    // optional event recording around the decoder and classifier launches
    uint32_t prof_capacity;
    uint64_t prof_steps;
    cudaEvent_t* prof_events;  // [capacity][3]
};

namespace {

constexpr size_t ALIGN = 256;
constexpr size_t TOKENS_PER_LAUNCH = 256;   // most tokens one launch of kl_token_kernel decodes (see STEP_WRAP_MARGIN)
inline size_t align_up(size_t v, size_t a = ALIGN) { return (v + a - 1) / a * a; }
inline uint32_t ceil_div(uint32_t a, uint32_t b) { return (a + b - 1) / b; }

struct Layout {
    // weight arena, element offsets (bf16)
    size_t off_qkv, off_o, off_gu, off_d, off_g1, off_g2, off_bqkv, off_router, expert_stride, layer_stride;
    size_t off_gf, off_lm, off_embed, weight_elems;
    // scratch arena, byte offsets
    size_t sxa, sxb, sqkv, so, sh, spart, spart_ml, srope, sinvf, scounters, sstatus, sstep, stok, spos, slogits, samax, shid, stokp, stplan, sbxop, sbssq, sbpart, sbq, sbao, sbaml, sbbar, scratch_bytes;
    uint32_t bsplit[5];
    uint32_t cps;
};

bool shape_supported(const kl_model_desc& d, int num_sms) {
    if (!d.n_layers || !d.hidden || !d.n_q_heads || !d.n_kv_heads || !d.head_dim || !d.ffn || !d.vocab) return false;
    if (!d.max_batch || !d.max_ctx || (d.flags & ~(uint32_t)(KL_FLAG_QKV_BIAS | KL_FLAG_NO_STASH)) != 0) return false;
    if (d.head_dim != 32 && d.head_dim != 64 && d.head_dim != 128 && d.head_dim != 256) return false;
    if (d.hidden % 8 || d.ffn % 8) return false;
    if (d.n_q_heads % d.n_kv_heads) return false;
    const uint32_t G = d.n_q_heads / d.n_kv_heads;
    // the CUDA-core attention loop is instantiated for 1, 2, 4 and 8 query heads per kv head; the tensor-core loop
    // (head size 64 or 128) takes any group size up to 8
    const bool pow2 = G == 1 || G == 2 || G == 4 || G == 8;
    if (!pow2 && !(G <= 8 && (d.head_dim == 64 || d.head_dim == 128))) return false;
    if ((uint64_t)d.n_kv_heads > (uint64_t)num_sms) return false;
    if (!(d.rms_eps >= 0.f) || !(d.rope_theta > 0.f)) return false;
    if (d.n_experts || d.top_k) {
        if (d.n_experts > (uint32_t)MAX_EXPERTS || d.top_k < 1 || d.top_k > (uint32_t)MAX_TOP_K || d.top_k > d.n_experts) return false;
    }
    return true;
}

// K splits of a batched projection [R x K]: the (row tile, split) items are dealt round-robin to the P CTAs.  More
// splits fill the last round better but every split writes and the consumer re-reads a [32 x R] fp32 partial result;
// pick the count that minimises streamed bytes (idle CTAs of the last round counted as if they streamed) plus that
// partial traffic, with at least four K blocks per split and at most eight splits.
static uint32_t pick_split(uint32_t R, uint32_t K, uint32_t P) {
    const uint32_t tiles = (R + 127) / 128, nkb = (K + 63) / 64;
    uint32_t best = 1;
    double best_cost = 0.0;
    for (uint32_t sp = 1; sp <= 8 && (sp == 1 || nkb / sp >= 4); ++sp) {
        const uint32_t items = tiles * sp;
        const double stream = (double)((items + P - 1) / P) * P * (128.0 * K * 2.0 / sp);
        const double cost = stream + 2.0 * sp * R * 32.0 * 4.0;
        if (sp == 1 || cost < best_cost) {
            best_cost = cost;
            best = sp;
        }
    }
    return best;
}

// Dynamic shared memory of kl_b_attn_kernel: alignment slack, the warps' ring slots, their barriers, the abort flag.
static size_t batched_attn_smem() { return 1024 + (size_t)BA_WARPS * BA_SLOTS * BA_SLOT_BYTES + (size_t)BA_WARPS * BA_SLOTS * 8 + 16; }

Layout make_layout(const kl_model_desc& d, int num_sms) {
    Layout y;
    const size_t H = d.hidden, QD = (size_t)d.n_q_heads * d.head_dim, KVD = (size_t)d.n_kv_heads * d.head_dim, F = d.ffn,
                 V = d.vocab, B = d.max_batch;
    size_t o = 0;
    y.off_qkv = o; o += (QD + 2 * KVD) * H;
    y.off_o = o;   o += H * QD;
    // dense: gate/up | down; mixture of experts: that pair once per expert, expert_stride elements apart
    const size_t NE = d.n_experts ? d.n_experts : 1;
    y.expert_stride = 3 * F * H;
    y.off_gu = o;
    y.off_d = o + 2 * F * H;
    o += NE * y.expert_stride;
    y.off_g1 = o;  o += H;
    y.off_g2 = o;  o += H;
    y.off_bqkv = o; o += (d.flags & KL_FLAG_QKV_BIAS) ? align_up((QD + 2 * KVD) * 2, 16) / 2 : 0;
    y.off_router = o; o += d.n_experts ? align_up((size_t)d.n_experts * H * 2, 16) / 2 : 0;
    y.layer_stride = align_up(o * 2, ALIGN) / 2;
    o = y.layer_stride * d.n_layers;
    y.off_gf = o;    o += align_up(H * 2, ALIGN) / 2;
    y.off_lm = o;    o += align_up(V * H * 2, ALIGN) / 2;
    y.off_embed = o; o += align_up(V * H * 2, ALIGN) / 2;
    y.weight_elems = o;

    y.cps = (uint32_t)num_sms / (uint32_t)(B * d.n_kv_heads);
    const uint32_t G = d.n_q_heads / d.n_kv_heads;
    const size_t units = (size_t)num_sms;  // at most one attention unit per CTA
    size_t s = 0;
    // tagged words (8 bytes each): xa, xb, qkv, o, split-K partials; h is plain fp32
    y.sxa = s;       s += align_up(B * H * 8);
    y.sxb = s;       s += align_up(B * H * 8);
    y.sqkv = s;      s += align_up(B * (QD + 2 * KVD) * 8);
    y.so = s;        s += align_up(B * QD * 8);
    y.sh = s;        s += align_up(B * F * 4 * (d.top_k ? d.top_k : 1));
    y.spart = s;     s += align_up(units * G * d.head_dim * 8);
    y.spart_ml = s;  s += align_up(units * G * 2 * 8);
    y.srope = s;     s += align_up((B > 1 ? 32 : B) * d.head_dim * 4);
    y.sinvf = s;     s += align_up((size_t)(d.head_dim / 2) * 8);
    y.scounters = s; s += align_up((size_t)d.n_layers * 4);
    y.sstatus = s;   s += ALIGN;
    y.sstep = s;     s += ALIGN;
    y.stok = s;      s += align_up(B * 4);
    y.spos = s;      s += align_up(B * 4);
    y.slogits = s;   s += align_up(B * V * 4);
    y.samax = s;     s += align_up(B * ARGMAX_BLOCKS * 8 + B * 4);
    y.shid = s;      s += align_up((B > 1 ? 32 : B) * H * 4);
    y.stokp = s;     s += align_up((size_t)num_sms * 8 + ALIGN);
    y.stplan = s;    s += align_up(TOKENS_PER_LAUNCH * 4) + align_up((size_t)TOKENS_PER_LAUNCH * d.head_dim * 4);
    // batched path (max_batch > 1): operand, partial sums, queries, attention partials
    {
        const size_t QR = QD + 2 * KVD;
        const size_t rows[5] = {QR, H, 2 * F, H, V}, ks[5] = {H, QD, H, F, H};
        size_t part_max = 0;
        for (int i = 0; i < 5; ++i) {
            y.bsplit[i] = i == 4 ? 1u : pick_split((uint32_t)rows[i], (uint32_t)ks[i], (uint32_t)num_sms);
            if (i < 4 && y.bsplit[i] * rows[i] > part_max) part_max = y.bsplit[i] * rows[i];
        }
        const bool on = B > 1;
        // one operand buffer per input width (hidden, q width, ffn), each on a 1024-byte boundary
        y.sbxop = s;  s += on ? align_up(64 * H * 2 + 1024) + align_up(64 * QD * 2 + 1024) + align_up(64 * F * 2 + 1024) : 0;
        y.sbssq = s;  s += on ? align_up((size_t)32 * BV_MAX_CHUNKS * 4) : 0;
        // stream schedule: one partial tile [32][128] per (row tile + CTA)
        const size_t stream_max = (ceil_div((uint32_t)(2 * F > QR ? 2 * F : QR), 128u) + (size_t)num_sms) * 128;
        if (stream_max > part_max) part_max = stream_max;
        y.sbpart = s; s += on ? align_up(part_max * 32 * 4) : 0;
        y.sbq = s;    s += on ? align_up(32 * QD * 4) : 0;
        const size_t aslots = B * d.n_kv_heads + (size_t)num_sms * BA_WARPS;   // attention partial results: pair + warp
        y.sbao = s;   s += on ? align_up(aslots * G * d.head_dim * 4) : 0;
        y.sbaml = s;  s += on ? align_up(aslots * G * 2 * 4) : 0;
        y.sbbar = s;  s += on ? align_up(((size_t)d.n_layers + 1) * 16 * 4) : 0;
    }
    y.scratch_bytes = s;
    return y;
}

// `align`: units must not straddle multiples of `align` rows (sources that are concatenated row-wise, such as
// Wq | Wk | Wv, start at multiples of it); 0 = no constraint.
// `x_in_smem`: the stage's input vector is staged in shared memory, so whole rows of any length that fit a slot are fine.
GemvPlan make_plan(uint32_t R, uint32_t K, bool pairs, uint32_t P, uint32_t align, bool x_in_smem) {
    GemvPlan pl;
    memset(&pl, 0, sizeof(pl));
    pl.R = R;
    pl.K = K;
    const uint32_t rowbytes = K * 2;
    const uint32_t minrows = pairs ? 2u : 1u;
    if ((K <= MAX_KP || x_in_smem) && rowbytes * minrows <= (uint32_t)SLOT_BYTES) {
        // whole rows: as many as fit a slot, but keep at least ~2 chunks per CTA on small matrices
        uint32_t rpc = SLOT_BYTES / rowbytes;
        uint32_t cap = R / (2 * P);
        if (cap < minrows) cap = minrows;
        if (rpc > cap) rpc = cap;
        if (pairs) rpc &= ~1u;
        while (align && rpc > 1 && align % rpc) --rpc;
        pl.rpc = rpc;
        pl.kp = K;
        pl.npieces = 1;
    } else {
        // units cut into column pieces.  A piece count that divides the consumer count (or is a multiple of it)
        // keeps every consumer on the same column piece for a whole stage, so its share of the input vector
        // stays in registers.
        // pieces multiplied against shared memory may be as long as a slot allows; pieces whose vector slice lives in
        // registers are capped
        const uint32_t kp_max = x_in_smem ? (uint32_t)SLOT_BYTES / (2u * minrows) / 256u * 256u : MAX_KP / 256u * 256u;
        uint32_t np = ceil_div(K, kp_max);
        const uint32_t cand[5] = {1, 2, 3, NCW, 2 * NCW};
        for (int q = 0; q < 5; ++q)
            if (cand[q] >= np) { np = cand[q]; break; }
        // a piece multiplied against shared memory starts at a block of 256 columns; one read from global memory
        // only needs 16-byte pieces per lane
        const uint32_t gran = x_in_smem ? 256u : 8u;
        pl.kp = ceil_div(ceil_div(K, np), gran) * gran;
        pl.npieces = ceil_div(K, pl.kp);
        uint32_t rpc = SLOT_BYTES / (pl.kp * 2);
        if (rpc > (uint32_t)MAX_RPC_SPLIT) rpc = MAX_RPC_SPLIT;
        if (pairs) rpc &= ~1u;
        while (align && rpc > 1 && align % rpc) --rpc;
        if (rpc < 1) rpc = 1;
        pl.rpc = rpc;
    }
    pl.nunits = ceil_div(R, pl.rpc);
    return pl;
}

bool plans_ok(const Params& p) {
    for (int i = 0; i < PL_COUNT; ++i) {
        const GemvPlan& pl = p.plan[i];
        if (pl.npieces > (uint32_t)MAX_PIECES || pl.rpc < 1) return false;
        if (pl.kp > MAX_KP && (i == PL_D || pl.rpc > (uint32_t)MAX_RPC_SPLIT)) return false;
        if (pl.rpc * pl.kp * 2 > (uint32_t)SLOT_BYTES) return false;
        if (pl.npieces > 1 && (pl.rpc > (uint32_t)MAX_RPC_SPLIT || pl.kp % (i == PL_D ? 8 : 256))) return false;
        if (i == PL_GU && (pl.rpc & 1u)) return false;
    }
    return true;
}

// Plans of the stash mode: pieces of kp columns with kp a multiple of 1024 that divides K (whole rows where two of them,
// or a (gate, up) pair, fit a slot), chunks of 16 KB at most.  rpc == 0: the matrix cannot be cut this way.
GemvPlan make_plan_t(uint32_t R, uint32_t K, bool pairs, uint32_t P, uint32_t align) {
    GemvPlan pl;
    memset(&pl, 0, sizeof(pl));
    pl.R = R;
    pl.K = K;
    pl.nseg = 1;
    const uint32_t minrows = pairs ? 2u : 1u;
    uint32_t kp = 0;
    const uint32_t cand[4] = {4096u, 3072u, 2048u, 1024u};   // the widths the consumer loop is instantiated for
    for (int i = 0; i < 4 && !kp; ++i)
        if (K % cand[i] == 0 && cand[i] * 2u * minrows <= (uint32_t)SLOT_BYTES) kp = cand[i];
    if (!kp) return pl;
    pl.kp = kp;
    pl.npieces = K / kp;
    uint32_t rpc = SLOT_BYTES / (kp * 2u);
    if (pl.npieces == 1) {   // whole rows: keep at least ~2 chunks per CTA on small matrices
        uint32_t cap = R / (2 * P);
        if (cap < minrows) cap = minrows;
        if (rpc > cap) rpc = cap;
    }
    if (pairs) rpc &= ~1u;
    while (align && rpc > 1 && align % rpc) --rpc;
    pl.rpc = rpc;
    pl.nunits = rpc ? ceil_div(R, rpc) : 0;
    return pl;
}
bool plans_ok_t(const Params& p) {
    for (int i = 0; i < PL_COUNT; ++i) {
        const GemvPlan& pl = p.plan[i];
        if (pl.rpc < 1 || pl.rpc * pl.kp * 2 > (uint32_t)SLOT_BYTES || pl.npieces > 32) return false;
        if (i == PL_GU && (pl.rpc & 1u)) return false;
    }
    return true;
}

// Writes `rows` source rows (row-major [rows, K]) into the library's copy of a matrix in chunk order (see GemvPlan):
// source row s becomes row v0 + s * vstep of the matrix.  vstep = 1 with v0 a multiple of the unit size, or
// vstep = 2 (gate / up rows interleaved) with units of two rows.
cudaError_t store_rows(const GemvPlan& pl, __nv_bfloat16* mat, const __nv_bfloat16* src, size_t rows, uint32_t v0,
                       uint32_t vstep, cudaStream_t st) {
    const size_t K = pl.K;
    cudaError_t e = cudaSuccess;
    if (pl.npieces == 1) {
        // plain row-major
        if (vstep == 1) return cudaMemcpyAsync(mat + (size_t)v0 * K, src, rows * K * 2, cudaMemcpyDefault, st);
        return cudaMemcpy2DAsync(mat + (size_t)v0 * K, vstep * K * 2, src, K * 2, K * 2, rows, cudaMemcpyDefault, st);
    }
    const size_t rpc = pl.rpc;
    for (uint32_t j = 0; j < pl.npieces && e == cudaSuccess; ++j) {
        const size_t c0 = (size_t)j * pl.kp;
        const size_t len = (j == pl.npieces - 1) ? K - c0 : pl.kp;
        if (vstep == 2) {
            // units of rpc/2 (gate f, up f) row pairs: source row s of this tensor is row 2 * (s % (rpc/2)) + v0 of
            // unit s / (rpc/2)
            const size_t ppu = rpc / 2;
            for (size_t t = 0; t < ppu && e == cudaSuccess; ++t) {
                if (rows <= t) break;
                const size_t cnt = (rows - t + ppu - 1) / ppu;
                e = cudaMemcpy2DAsync(mat + rpc * c0 + (2 * t + v0) * len, rpc * K * 2, src + t * K + c0, ppu * K * 2,
                                      len * 2, cnt, cudaMemcpyDefault, st);
            }
            continue;
        }
        const size_t u_first = v0 / rpc;
        const size_t full = rows / rpc;           // whole units covered by this tensor
        for (size_t rr = 0; rr < rpc && e == cudaSuccess && full > 0; ++rr)
            e = cudaMemcpy2DAsync(mat + u_first * rpc * K + rpc * c0 + rr * len, rpc * K * 2, src + rr * K + c0, rpc * K * 2,
                                  len * 2, full, cudaMemcpyDefault, st);
        const size_t rest = rows - full * rpc;    // rows of a last, short unit (end of the matrix)
        for (size_t rr = 0; rr < rest && e == cudaSuccess; ++rr)
            e = cudaMemcpyAsync(mat + (u_first + full) * rpc * K + rest * c0 + rr * len, src + (full * rpc + rr) * K + c0,
                                len * 2, cudaMemcpyDefault, st);
    }
    return e;
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// Launch with programmatic stream serialisation: the kernel may start while its predecessor in the stream still runs
// and orders itself behind it with griddepcontrol.wait (see griddep_wait in kl_batched.cuh).
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent(int allowed, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = allowed ? 1 : 0;   // 0: the kernel starts when its predecessor has ended
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

}  // namespace

extern "C" {

const char* kl_status_string(kl_status s) {
    switch (s) {
        case KL_OK: return "KL_OK";
        case KL_ERR_INVALID_ARG: return "KL_ERR_INVALID_ARG";
        case KL_ERR_UNSUPPORTED_SHAPE: return "KL_ERR_UNSUPPORTED_SHAPE";
        case KL_ERR_NOT_LOADED: return "KL_ERR_NOT_LOADED";
        case KL_ERR_CUDA: return "KL_ERR_CUDA";
        case KL_ERR_SYNC_TIMEOUT: return "KL_ERR_SYNC_TIMEOUT";
        case KL_ERR_OUT_OF_RANGE: return "KL_ERR_OUT_OF_RANGE";
        case KL_ERR_TOO_LARGE: return "KL_ERR_TOO_LARGE";
        default: return "KL_ERR_UNKNOWN";
    }
}

static int query_sms(int* dev_out) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    if (dev_out) *dev_out = dev;
    return sms;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A row-major bf16 matrix [rows, cols] as a 2-D tensor with boxes of [box_rows] x [64 columns] and the 128-byte swizzle.
static bool encode_bf16_2d(void* encode_fn, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    if (!encode_fn || ((uintptr_t)base & 15u) || (cols * 2) % 16) return false;
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return ((encode_tiled_fn)encode_fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A bf16 tensor of rank `rank` (dimensions innermost first, byte strides of dimensions 1 .. rank-1), 128-byte swizzle,
// zeros outside the tensor.
static bool encode_bf16_nd(void* encode_fn, CUtensorMap* map, const void* base, uint32_t rank, const cuuint64_t* dims,
                           const cuuint64_t* strides, const cuuint32_t* box) {
    if (!encode_fn || ((uintptr_t)base & 15u)) return false;
    for (uint32_t i = 0; i + 1 < rank; ++i)
        if (strides[i] % 16) return false;
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return ((encode_tiled_fn)encode_fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides, box, estr,
                                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps of one weight matrix (R rows, plan pl, `layers` copies layer_stride elements apart) for the batched
// projections: tiles of 128 rows x 64 columns.  A matrix stored whole-row is a rank-3 tensor (column, row, layer).  One
// stored in chunk order (units of rpc rows, each cut into column pieces of kp) is a rank-5 tensor (column in piece, row
// in unit, piece, unit, layer) for the full pieces and a rank-4 one for the last, shorter piece.
static bool encode_weight_maps(void* fn, CUtensorMap* map, CUtensorMap* map_last, const __nv_bfloat16* mat, const GemvPlan& pl,
                               uint32_t R, uint32_t layers, uint64_t layer_stride) {
    const uint64_t K = pl.K;
    if (R < (uint32_t)BG_TILE_M || K < (uint64_t)BG_TILE_K || K % 8) return false;
    const uint64_t lbytes = layers > 1 ? layer_stride * 2 : (((uint64_t)R * K * 2 + 15) & ~15ull);
    if (pl.npieces == 1) {
        const cuuint64_t dims[3] = {K, R, layers};
        const cuuint64_t strides[2] = {K * 2, lbytes};
        const cuuint32_t box[3] = {(cuuint32_t)BG_TILE_K, (cuuint32_t)BG_TILE_M, 1};
        return encode_bf16_nd(fn, map, mat, 3, dims, strides, box);
    }
    const uint64_t rpc = pl.rpc, kp = pl.kp, np = pl.npieces, last = K - (np - 1) * kp;
    if (R % rpc || BG_TILE_M % rpc || kp % 8 || last % 8 || kp < (uint64_t)BG_TILE_K || last == 0) return false;
    {
        const cuuint64_t dims[5] = {kp, rpc, np - 1, R / rpc, layers};
        const cuuint64_t strides[4] = {kp * 2, rpc * kp * 2, rpc * K * 2, lbytes};
        const cuuint32_t box[5] = {(cuuint32_t)BG_TILE_K, (cuuint32_t)rpc, 1, (cuuint32_t)(BG_TILE_M / rpc), 1};
        if (!encode_bf16_nd(fn, map, mat, 5, dims, strides, box)) return false;
    }
    const cuuint64_t dims[4] = {last, rpc, R / rpc, layers};
    const cuuint64_t strides[3] = {last * 2, rpc * K * 2, lbytes};
    const cuuint32_t box[4] = {(cuuint32_t)BG_TILE_K, (cuuint32_t)rpc, (cuuint32_t)(BG_TILE_M / rpc), 1};
    return encode_bf16_nd(fn, map_last, mat + rpc * (np - 1) * kp, 4, dims, strides, box);
}

kl_status kl_workspace_bytes(const kl_model_desc* desc, size_t* weight_bytes, size_t* scratch_bytes) {
    if (!desc || !weight_bytes || !scratch_bytes) return KL_ERR_INVALID_ARG;
    int sms = query_sms(nullptr);
    if (sms <= 0) sms = 148;  // sizes must be computable without a device; B200 has 148 SMs
    if (!shape_supported(*desc, sms)) return KL_ERR_UNSUPPORTED_SHAPE;
    const Layout y = make_layout(*desc, sms);
    *weight_bytes = y.weight_elems * 2;
    *scratch_bytes = y.scratch_bytes;
    return KL_OK;
}

kl_status kl_create(const kl_model_desc* desc, void* weight_arena_d, void* scratch_arena_d, kl_handle** out) {
    if (!desc || !weight_arena_d || !scratch_arena_d || !out) return KL_ERR_INVALID_ARG;
    if (((uintptr_t)weight_arena_d | (uintptr_t)scratch_arena_d) & (ALIGN - 1)) return KL_ERR_INVALID_ARG;
    int dev = 0;
    const int sms = query_sms(&dev);
    if (sms <= 0) return KL_ERR_CUDA;
    if (!shape_supported(*desc, sms)) return KL_ERR_UNSUPPORTED_SHAPE;
    const kl_model_desc& d = *desc;
    const Layout y = make_layout(d, sms);

    kl_handle* h = new (std::nothrow) kl_handle();
    if (!h) return KL_ERR_INVALID_ARG;
    memset(h, 0, sizeof(*h));
    h->desc = d;
    h->mode = KL_MODE_LOOPED;
    h->device = dev;
    h->num_sms = sms;
    h->weights = (uint8_t*)weight_arena_d;
    h->scratch = (uint8_t*)scratch_arena_d;
    h->weight_bytes = y.weight_elems * 2;
    h->scratch_bytes = y.scratch_bytes;
    h->pending_skip_stage = -1;
    h->use_tc_attention = 1;
    {
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            h->encode_tiled = fn;
        else
            h->use_tc_attention = 0;
    }
    // one flag per (tensor, layer), then one per (expert matrix kind, expert, layer)
    h->loaded = (uint8_t*)calloc((size_t)(KL_WROUTER + 1 + 3 * (size_t)d.n_experts) * (size_t)d.n_layers, 1);
    if (!h->loaded) { delete h; return KL_ERR_INVALID_ARG; }

    Params& p = h->prm;
    p.L = d.n_layers; p.H = d.hidden; p.nq = d.n_q_heads; p.nkv = d.n_kv_heads; p.hd = d.head_dim; p.F = d.ffn;
    p.V = d.vocab; p.G = d.n_q_heads / d.n_kv_heads; p.QD = d.n_q_heads * d.head_dim; p.KVD = d.n_kv_heads * d.head_dim;
    p.max_ctx = d.max_ctx; p.B = 1;
    if (!h->use_tc_attention && p.G != 1 && p.G != 2 && p.G != 4 && p.G != 8) {   // only the tensor-core loop takes this group size
        free(h->loaded); delete h; return KL_ERR_UNSUPPORTED_SHAPE;
    }
    p.P = (uint32_t)sms;
    p.cps = y.cps;
    p.eps = d.rms_eps;
    p.skip_stage = -1;
    p.wait_ns = 2000000000ull;
    p.layer_stride = y.layer_stride;
    // stash mode where the shape allows it (dense layers, the tensor-core attention loop, widths the mode is built for)
    h->stash = 0;
    {
        const char* e = getenv("KL_STASH");
        if (d.n_experts == 0 && h->use_tc_attention && !(d.flags & KL_FLAG_NO_STASH) && !(e && e[0] == '0')) {
            p.plan[PL_QKV] = make_plan_t(p.QD + 2 * p.KVD, p.H, false, p.P, p.KVD);
            p.plan[PL_O] = make_plan_t(p.H, p.QD, false, p.P, 0);
            p.plan[PL_GU] = make_plan_t(2 * p.F, p.H, true, p.P, 0);
            p.plan[PL_D] = make_plan_t(p.H, p.F, false, p.P, 0);
            p.plan[PL_LM] = make_plan_t(p.V, p.H, false, p.P, 0);
            // the vector area holds the widest input (the down projection's too), the ring is 2 x T_NSP slots
            const size_t vmax = (size_t)ceil_div(p.F > p.H ? (p.F > p.QD ? p.F : p.QD) : (p.H > p.QD ? p.H : p.QD), 256) * 256;
            int optin = 0;
            h->stash = plans_ok_t(p) && cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) == cudaSuccess &&
                       (size_t)2 * T_NSP * SLOT_BYTES + vmax * 4 + SMEM_MISC_BYTES + 16384 <= (size_t)optin;
            if (h->stash)   // 1: chunks of 2048 / 4096 columns only (the kernel without the other widths), 2: any
                for (int i = 0; i < PL_COUNT; ++i)
                    if (p.plan[i].kp != 2048u && p.plan[i].kp != 4096u) h->stash = 2;
        }
    }
    if (!h->stash) {
        p.plan[PL_QKV] = make_plan(p.QD + 2 * p.KVD, p.H, false, p.P, p.KVD, true);  // KVD divides QD: Wq | Wk | Wv stay aligned
        p.plan[PL_O] = make_plan(p.H, p.QD, false, p.P, 0, true);
        p.plan[PL_GU] = make_plan(2 * p.F, p.H, true, p.P, 0, true);
        p.plan[PL_D] = make_plan(p.H, p.F, false, p.P, 0, false);
        p.plan[PL_LM] = make_plan(p.V, p.H, false, p.P, 0, true);
        if (!plans_ok(p)) { free(h->loaded); delete h; return KL_ERR_UNSUPPORTED_SHAPE; }
    }
    p.n_experts = d.n_experts;
    p.top_k = d.top_k;
    p.expert_stride = y.expert_stride;
    for (int i = 0; i < PL_COUNT; ++i) p.plan[i].nseg = 1;
    if (d.n_experts) {
        // the chosen experts' pieces of a down-projection unit meet in one table; (gate, up) units must not straddle experts
        if (p.plan[PL_D].npieces * d.top_k > (uint32_t)MAX_PIECES || (2 * p.F) % p.plan[PL_GU].rpc || p.plan[PL_GU].R % p.plan[PL_GU].rpc) {
            free(h->loaded); delete h; return KL_ERR_UNSUPPORTED_SHAPE;
        }
    }

    // shared memory: input vector area (also the attention workspace), then as many ring slots as fit
    uint32_t vecf = p.H > p.QD ? p.H : p.QD;  // the down projection reads its input from L2, not from this area
    vecf = ceil_div(vecf, 256) * 256;
    // attention workspace: rotated q, the new K/V row, per-warp partial results, the staging tile of the new row
    // and, behind them, the merge tables: 2 * G * nchunk pairs and the unit's slice of every partial output
    const uint32_t comb_f = NCW * p.G * (p.hd + 2), merge_f = 2 * p.G * (p.P / p.nkv) + p.G * p.hd + 2 * (p.P / p.nkv);  // batch 1 has the most chunks
    const uint32_t attnf = p.G * p.hd + 2 * p.hd + 128 + comb_f + merge_f;
    if (attnf > vecf) vecf = ceil_div(attnf, 256) * 256;
    p.vec_floats = vecf;
    int max_optin = 0;
    if (cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
        free(h->loaded); delete h; return KL_ERR_CUDA;
    }
    if (h->stash) {
        // the down projection multiplies against shared memory too; the ring is two pipelines of T_NSP slots
        if (p.F > vecf) vecf = ceil_div(p.F, 256) * 256;
        p.vec_floats = vecf;
        p.nslots = 2 * T_NSP;
        p.nsw = 1;
        h->smem_bytes = (size_t)2 * T_NSP * SLOT_BYTES + (size_t)vecf * 4 + SMEM_MISC_BYTES;
        if (h->smem_bytes > (size_t)max_optin) { free(h->loaded); delete h; return KL_ERR_UNSUPPORTED_SHAPE; }
    } else {
    const long avail = (long)max_optin - (long)vecf * 4 - SMEM_MISC_BYTES;
    long nsw = avail / ((long)NCW * SLOT_BYTES);
    if (nsw > MAX_NSW) nsw = MAX_NSW;
    if (nsw < 1) { free(h->loaded); delete h; return KL_ERR_UNSUPPORTED_SHAPE; }
    p.nslots = NCW;
    p.nsw = (uint32_t)nsw;
    h->smem_bytes = (size_t)NCW * nsw * SLOT_BYTES + (size_t)vecf * 4 + SMEM_MISC_BYTES;
    }
    // The shared-memory limit is an attribute of the kernel, not of a handle: it is raised to the device's opt-in
    // maximum, so that handles of different shapes (each launching with its own smem_bytes) can be alive together.
    cudaError_t ce = cudaSuccess;
    {
        const void* fns[] = {(const void*)kl_decoder_kernel<false, false, 0, false>, (const void*)kl_decoder_kernel<false, false, 0, true>,
                             (const void*)kl_decoder_kernel<true, false, 0, false>, (const void*)kl_decoder_kernel<true, false, 0, true>,
                             (const void*)kl_decoder_kernel<false, true, 0, false>, (const void*)kl_decoder_kernel<false, true, 0, true>,
                             (const void*)kl_decoder_kernel<false, false, 1, false>, (const void*)kl_decoder_kernel<true, false, 1, false>,
                             (const void*)kl_decoder_kernel<false, false, 2, false>, (const void*)kl_decoder_kernel<true, false, 2, false>,
                             (const void*)kl_classifier_kernel<0>, (const void*)kl_classifier_kernel<1>, (const void*)kl_classifier_kernel<2>};
        for (const void* f : fns)
            if (ce == cudaSuccess) ce = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, max_optin);
    }
    {
        int tocc = 0;
        const void* fns[] = {(const void*)kl_token_kernel<false, false, 0, false>, (const void*)kl_token_kernel<false, false, 0, true>,
                             (const void*)kl_token_kernel<true, false, 0, false>, (const void*)kl_token_kernel<true, false, 0, true>,
                             (const void*)kl_token_kernel<false, true, 0, false>, (const void*)kl_token_kernel<false, true, 0, true>,
                             (const void*)kl_token_kernel<false, false, 1, false>, (const void*)kl_token_kernel<true, false, 1, false>,
                             (const void*)kl_token_kernel<false, false, 2, false>, (const void*)kl_token_kernel<true, false, 2, false>};
        h->token_ok = 1;
        for (const void* f : fns)
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, max_optin) != cudaSuccess) h->token_ok = 0;
        if (h->token_ok)
            h->token_ok = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&tocc, kl_token_kernel<true, false, 0, true>, NTHREADS, h->smem_bytes) == cudaSuccess && tocc >= 1;
        (void)cudaGetLastError();
    }
    int occ = 0;
    if (ce == cudaSuccess) ce = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kl_decoder_kernel<true, false, 0, true>, NTHREADS, h->smem_bytes);
    if (ce != cudaSuccess || occ < 1) {
        fprintf(stderr, "kl_create: the persistent kernel cannot be resident (%s; %zu bytes of shared memory, %d threads, "
                        "occupancy %d)\n", cudaGetErrorString(ce), h->smem_bytes, NTHREADS, occ);
        free(h->loaded); delete h; return KL_ERR_CUDA;
    }

    const __nv_bfloat16* w = reinterpret_cast<const __nv_bfloat16*>(h->weights);
    p.wqkv = w + y.off_qkv; p.wo = w + y.off_o; p.wgu = w + y.off_gu; p.wd = w + y.off_d;
    p.bqkv = (d.flags & KL_FLAG_QKV_BIAS) ? w + y.off_bqkv : nullptr;
    p.g1 = w + y.off_g1; p.g2 = w + y.off_g2; p.gf = w + y.off_gf; p.wlm = w + y.off_lm; p.embed = w + y.off_embed;
    p.wrouter = d.n_experts ? w + y.off_router : nullptr;
    uint8_t* sc = h->scratch;
    p.xa = (TW*)(sc + y.sxa); p.xb = (TW*)(sc + y.sxb); p.qkv = (TW*)(sc + y.sqkv); p.o = (TW*)(sc + y.so);
    p.h = (float*)(sc + y.sh);
    p.part = (TW*)(sc + y.spart); p.part_ml = (TW*)(sc + y.spart_ml); p.rope_cs = (float*)(sc + y.srope);
    p.inv_freq = (const double*)(sc + y.sinvf);
    p.counters = (uint32_t*)(sc + y.scounters);
    p.step_dev = (uint32_t*)(sc + y.sstep);
    p.status = (int32_t*)(sc + y.sstatus);
    h->stage_tokens = (int32_t*)(sc + y.stok);
    h->stage_positions = (int32_t*)(sc + y.spos);
    h->stage_logits = (float*)(sc + y.slogits);
    h->argmax_val = (float*)(sc + y.samax);
    h->hidden_all = (float*)(sc + y.shid);
    h->tok_val = (float*)(sc + y.stokp);
    h->tok_idx = (uint32_t*)(h->tok_val + sms);
    h->tok_ticket = h->tok_idx + sms;
    h->plan_out = (int32_t*)(sc + y.stplan);
    h->plan_rope = (float*)((uint8_t*)h->plan_out + align_up(TOKENS_PER_LAUNCH * 4));
    h->hidden_is_copy = 0;
    h->chain_tok = nullptr;
    h->last_batch = 1;
    // tensor-core path for batches of up to 32 sequences
    h->bx = h->hidden_all;
    {
        uintptr_t a = ((uintptr_t)(sc + y.sbxop) + 1023u) & ~(uintptr_t)1023u;
        const size_t widths[3] = {p.H, p.QD, p.F};
        for (int i = 0; i < 3; ++i) {
            h->bxop[i] = (__nv_bfloat16*)a;
            a = (a + 64 * widths[i] * 2 + 1023u) & ~(uintptr_t)1023u;
        }
    }
    h->bssq = (float*)(sc + y.sbssq);
    h->bpart = (float*)(sc + y.sbpart);
    h->bq = (float*)(sc + y.sbq);
    h->bao = (float*)(sc + y.sbao);
    h->baml = (float*)(sc + y.sbaml);
    h->bbar = (uint32_t*)(sc + y.sbbar);
    for (int i = 0; i < 5; ++i) h->bsplit[i] = y.bsplit[i];
    h->use_bt = 1;
    h->use_stream = 1;
    h->use_pdl = 1;
    h->cap_stream = nullptr;
    h->bgraph = nullptr;
    h->bgraph_kv = nullptr;
    h->bgraph_tok = h->bgraph_pos = nullptr;
    h->bgraph_logits = nullptr;
    h->bgraph_batch = 0;
    h->bgraph_launches = 0;
    h->bt_ok = 0;
    h->bl_ok = 0;
    if (d.n_experts == 0 && d.max_batch > 1 && d.max_batch <= (uint32_t)BG_MAX_BATCH && (p.hd == 64 || p.hd == 128) && p.G <= (uint32_t)MAX_G &&
        p.H % 8 == 0 && p.QD % 8 == 0 && p.F % 8 == 0) {
        const uint32_t QR = p.QD + 2 * p.KVD;
        const size_t ba_smem = batched_attn_smem();
        bool ok = encode_weight_maps(h->encode_tiled, &h->bmap_w[0], &h->bmap_wl[0], p.wqkv, p.plan[PL_QKV], QR, p.L, p.layer_stride) &&
                  encode_weight_maps(h->encode_tiled, &h->bmap_w[1], &h->bmap_wl[1], p.wo, p.plan[PL_O], p.H, p.L, p.layer_stride) &&
                  encode_weight_maps(h->encode_tiled, &h->bmap_w[2], &h->bmap_wl[2], p.wgu, p.plan[PL_GU], 2 * p.F, p.L, p.layer_stride) &&
                  encode_weight_maps(h->encode_tiled, &h->bmap_w[3], &h->bmap_wl[3], p.wd, p.plan[PL_D], p.H, p.L, p.layer_stride) &&
                  encode_weight_maps(h->encode_tiled, &h->bmap_w[4], &h->bmap_wl[4], p.wlm, p.plan[PL_LM], p.V, 1, 0) &&
                  encode_bf16_2d(h->encode_tiled, &h->bmap_x[0], h->bxop[0], 64, p.H, BG_TILE_N) &&
                  encode_bf16_2d(h->encode_tiled, &h->bmap_x[1], h->bxop[1], 64, p.QD, BG_TILE_N) &&
                  encode_bf16_2d(h->encode_tiled, &h->bmap_x[2], h->bxop[2], 64, p.F, BG_TILE_N);
        ok = ok && p.H <= (uint32_t)(BV_CHUNK * BV_MAX_CHUNKS);
        ok = ok && cudaFuncSetAttribute(kl_bgemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BG_SMEM_BYTES) == cudaSuccess &&
             cudaFuncSetAttribute(kl_b_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ba_smem) == cudaSuccess;
        (void)cudaGetLastError();
        h->bt_ok = ok ? 1 : 0;
        int bocc = 0;
        h->bl_ok = ok && cudaFuncSetAttribute(kl_bloop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BL_SMEM_BYTES) == cudaSuccess &&
                   cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bocc, kl_bloop_kernel, BL_THREADS, BL_SMEM_BYTES) == cudaSuccess && bocc >= 1;
        (void)cudaGetLastError();
    }
    h->argmax_idx = (uint32_t*)(h->argmax_val + (size_t)d.max_batch * ARGMAX_BLOCKS);
    h->argmax_tickets = h->argmax_idx + (size_t)d.max_batch * ARGMAX_BLOCKS;

    if (cudaMemset(h->scratch, 0, h->scratch_bytes) != cudaSuccess) { free(h->loaded); delete h; return KL_ERR_CUDA; }
    double invf[128];
    for (uint32_t i = 0; i < d.head_dim / 2; ++i) invf[i] = pow((double)d.rope_theta, -2.0 * (double)i / (double)d.head_dim);
    if (cudaMemcpy(sc + y.sinvf, invf, (d.head_dim / 2) * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) {
        free(h->loaded); delete h; return KL_ERR_CUDA;
    }
    *out = h;
    return KL_OK;
}

kl_status kl_load_weights(kl_handle* h, int tensor, int layer, const void* src, size_t bytes, void* stream) {
    if (!h || !src) return KL_ERR_INVALID_ARG;
    const Params& p = h->prm;
    const Layout y = make_layout(h->desc, h->num_sms);
    const bool global_t = (tensor == KL_EMBED || tensor == KL_NORM_F || tensor == KL_LM_HEAD);
    if (tensor < 0 || tensor > KL_WROUTER) return KL_ERR_INVALID_ARG;
    if (tensor > KL_LM_HEAD && tensor <= KL_BV && !(h->desc.flags & KL_FLAG_QKV_BIAS)) return KL_ERR_INVALID_ARG;   // this model has no biases
    if (tensor == KL_WROUTER && !p.n_experts) return KL_ERR_INVALID_ARG;   // this model has no router
    if (global_t ? (layer != -1) : (layer < 0 || layer >= (int)p.L)) return KL_ERR_INVALID_ARG;
    __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(h->weights);
    const size_t lo = global_t ? 0 : (size_t)layer * y.layer_stride;
    size_t rows = 0, cols = 0, dst = 0;
    const GemvPlan* pl = nullptr;   // matrices streamed through the ring are stored in chunk order
    uint32_t v0 = 0, vstep = 1;
    switch (tensor) {
        case KL_EMBED: rows = p.V; cols = p.H; dst = y.off_embed; break;
        case KL_LM_HEAD: rows = p.V; cols = p.H; dst = y.off_lm; pl = &p.plan[PL_LM]; break;
        case KL_NORM_F: rows = 1; cols = p.H; dst = y.off_gf; break;
        case KL_WQ: rows = p.QD; cols = p.H; dst = lo + y.off_qkv; pl = &p.plan[PL_QKV]; break;
        case KL_WK: rows = p.KVD; cols = p.H; dst = lo + y.off_qkv; pl = &p.plan[PL_QKV]; v0 = p.QD; break;
        case KL_WV: rows = p.KVD; cols = p.H; dst = lo + y.off_qkv; pl = &p.plan[PL_QKV]; v0 = p.QD + p.KVD; break;
        case KL_WO: rows = p.H; cols = p.QD; dst = lo + y.off_o; pl = &p.plan[PL_O]; break;
        // gate and up rows are interleaved (row 2f = gate f, row 2f+1 = up f) so one chunk holds both halves of a pair
        case KL_WGATE: rows = p.F; cols = p.H; dst = lo + y.off_gu; pl = &p.plan[PL_GU]; v0 = 0; vstep = 2; break;
        case KL_WUP: rows = p.F; cols = p.H; dst = lo + y.off_gu; pl = &p.plan[PL_GU]; v0 = 1; vstep = 2; break;
        case KL_WDOWN: rows = p.H; cols = p.F; dst = lo + y.off_d; pl = &p.plan[PL_D]; break;
        case KL_NORM1: rows = 1; cols = p.H; dst = lo + y.off_g1; break;
        case KL_NORM2: rows = 1; cols = p.H; dst = lo + y.off_g2; break;
        case KL_BQ: rows = 1; cols = p.QD; dst = lo + y.off_bqkv; break;
        case KL_BK: rows = 1; cols = p.KVD; dst = lo + y.off_bqkv + p.QD; break;
        case KL_BV: rows = 1; cols = p.KVD; dst = lo + y.off_bqkv + p.QD + p.KVD; break;
        case KL_WROUTER: rows = p.n_experts; cols = p.H; dst = lo + y.off_router; break;
        default: return KL_ERR_INVALID_ARG;
    }
    if (p.n_experts && (tensor == KL_WGATE || tensor == KL_WUP || tensor == KL_WDOWN)) return KL_ERR_INVALID_ARG;   // per expert
    if (bytes != rows * cols * 2) return KL_ERR_INVALID_ARG;
    cudaError_t e;
    if (pl) e = store_rows(*pl, w + dst, reinterpret_cast<const __nv_bfloat16*>(src), rows, v0, vstep, as_stream(stream));
    else e = cudaMemcpyAsync(w + dst, src, bytes, cudaMemcpyDefault, as_stream(stream));
    if (e != cudaSuccess) return KL_ERR_CUDA;
    h->loaded[(size_t)tensor * p.L + (global_t ? 0 : layer)] = 1;
    return KL_OK;
}

kl_status kl_load_expert_weights(kl_handle* h, int tensor, int layer, int expert, const void* src, size_t bytes, void* stream) {
    if (!h || !src) return KL_ERR_INVALID_ARG;
    const Params& p = h->prm;
    if (!p.n_experts || expert < 0 || expert >= (int)p.n_experts || layer < 0 || layer >= (int)p.L) return KL_ERR_INVALID_ARG;
    if (tensor != KL_WGATE && tensor != KL_WUP && tensor != KL_WDOWN) return KL_ERR_INVALID_ARG;
    const Layout y = make_layout(h->desc, h->num_sms);
    __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(h->weights);
    const size_t lo = (size_t)layer * y.layer_stride + (size_t)expert * y.expert_stride;
    const bool down = tensor == KL_WDOWN;
    const size_t rows = down ? p.H : p.F, cols = down ? p.F : p.H;
    if (bytes != rows * cols * 2) return KL_ERR_INVALID_ARG;
    const cudaError_t e = down ? store_rows(p.plan[PL_D], w + lo + y.off_d, reinterpret_cast<const __nv_bfloat16*>(src), rows, 0, 1, as_stream(stream))
                               : store_rows(p.plan[PL_GU], w + lo + y.off_gu, reinterpret_cast<const __nv_bfloat16*>(src), rows,
                                            tensor == KL_WUP ? 1u : 0u, 2, as_stream(stream));
    if (e != cudaSuccess) return KL_ERR_CUDA;
    const int kind = tensor == KL_WGATE ? 0 : tensor == KL_WUP ? 1 : 2;
    h->loaded[((size_t)(KL_WROUTER + 1) + (size_t)kind * p.n_experts + (size_t)expert) * p.L + (size_t)layer] = 1;
    return KL_OK;
}

// The KV cache as a 2-D bf16 tensor [n_layers*2*batch*n_kv_heads*max_ctx rows, head_dim columns]; boxes of
// [positions per chunk] x [64 columns] with the 128-byte swizzle.  Encoded per call because the cache is the caller's.
// The cache as the 4-D tensor of the batch-1 kernels' ring copies (see Params::kv_map4): dimension 0 = 64 columns,
// 1 = rows (all slabs one after the other), 2 = 64-column halves of a row, 3 = K | V, a slab of `batch` sequences apart.
static kl_status encode_kv_map4(kl_handle* h, CUtensorMap* map, void* kv_cache_d, uint32_t batch, uint32_t slot_bytes = SLOT_BYTES) {
    if (!h->encode_tiled) return KL_ERR_CUDA;
    if ((uintptr_t)kv_cache_d & 15u) return KL_ERR_INVALID_ARG;
    const kl_model_desc& d = h->desc;
    const cuuint64_t rows = (cuuint64_t)d.n_layers * 2 * batch * d.n_kv_heads * d.max_ctx;
    if (rows > 0x7fffffffull) return KL_ERR_UNSUPPORTED_SHAPE;  // box coordinates are 32-bit signed
    const cuuint64_t vdelta = (cuuint64_t)batch * d.n_kv_heads * d.max_ctx;   // rows between a K slab and its V slab
    const cuuint64_t gdim[4] = {64, rows, d.head_dim / 64, 2};
    const cuuint64_t gstride[3] = {(cuuint64_t)d.head_dim * 2, 128, vdelta * d.head_dim * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)(slot_bytes / (4 * d.head_dim)), d.head_dim / 64, 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = ((encode_tiled_fn)h->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, kv_cache_d, gdim, gstride, box,
                                                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                         CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KL_OK : KL_ERR_CUDA;
}

static kl_status encode_kv_map(kl_handle* h, CUtensorMap* map, void* kv_cache_d, uint32_t batch, uint32_t slot_bytes = SLOT_BYTES) {
    if (!h->encode_tiled) return KL_ERR_CUDA;
    if ((uintptr_t)kv_cache_d & 15u) return KL_ERR_INVALID_ARG;
    const kl_model_desc& d = h->desc;
    const cuuint64_t rows = (cuuint64_t)d.n_layers * 2 * batch * d.n_kv_heads * d.max_ctx;
    if (rows > 0x7fffffffull) return KL_ERR_UNSUPPORTED_SHAPE;  // box coordinates are 32-bit signed
    const cuuint64_t gdim[2] = {d.head_dim, rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)d.head_dim * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)(slot_bytes / (4 * d.head_dim))};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = ((encode_tiled_fn)h->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, kv_cache_d, gdim, gstride, box,
                                                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                         CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KL_OK : KL_ERR_CUDA;
}

static bool all_loaded(const kl_handle* h) {
    const uint32_t L = h->prm.L;
    const uint32_t E = h->prm.n_experts;
    for (int t = 0; t <= KL_WROUTER; ++t) {
        if (t > KL_LM_HEAD && t <= KL_BV && !(h->desc.flags & KL_FLAG_QKV_BIAS)) continue;
        if (t == KL_WROUTER && !E) continue;
        if (E && (t == KL_WGATE || t == KL_WUP || t == KL_WDOWN)) continue;   // loaded per expert, checked below
        const bool global_t = (t == KL_EMBED || t == KL_NORM_F || t == KL_LM_HEAD);
        for (uint32_t l = 0; l < (global_t ? 1u : L); ++l)
            if (!h->loaded[(size_t)t * L + l]) return false;
    }
    for (size_t i = 0; i < (size_t)3 * E * L; ++i)
        if (!h->loaded[(size_t)(KL_WROUTER + 1) * L + i]) return false;
    return true;
}

size_t kl_kv_cache_bytes(const kl_handle* h, uint32_t batch) {
    if (!h) return 0;
    const kl_model_desc& d = h->desc;
    return (size_t)d.n_layers * 2 * batch * d.n_kv_heads * d.max_ctx * d.head_dim * 2;
}

static void drop_batched_graph(kl_handle* h);

kl_status kl_set_mode(kl_handle* h, int mode) {
    if (!h || (mode != KL_MODE_LOOPED && mode != KL_MODE_PER_LAYER && mode != KL_MODE_PER_STAGE)) return KL_ERR_INVALID_ARG;
    if (mode != h->mode || !h->mode_explicit) drop_batched_graph(h);   // a cached graph holds the launches of the old schedule
    h->mode = mode;
    h->mode_explicit = 1;
    return KL_OK;
}

static kl_status launch_persistent(kl_handle* h, const void* func, void** args, cudaStream_t st) {
    // cooperative launch: the driver guarantees that all CTAs are co-resident (the counters depend on it)
    const cudaError_t e = cudaLaunchCooperativeKernel(func, dim3(h->prm.P), dim3(NTHREADS), args, h->smem_bytes, st);
    if (e != cudaSuccess) return KL_ERR_CUDA;
    ++h->launches;
    return KL_OK;
}

// One projection of the batched path: out[s][b][r] = partial sums over K split s of W[idx](layer) . operand.
static kl_status launch_bgemm(kl_handle* h, int idx, uint32_t layer, float* out, uint32_t batch, cudaStream_t st,
                              BgPartials* parts = nullptr) {
    const Params& p = h->prm;
    static const int plan_of[5] = {PL_QKV, PL_O, PL_GU, PL_D, PL_LM};
    static const int xmap_of[5] = {0, 1, 0, 2, 0};
    const uint32_t rows[5] = {p.QD + 2 * p.KVD, p.H, 2 * p.F, p.H, p.V};
    const GemvPlan& pl = p.plan[plan_of[idx]];
    BgemmParams g;
    g.map_w = h->bmap_w[idx];
    g.map_wl = h->bmap_wl[idx];
    g.map_x = h->bmap_x[xmap_of[idx]];
    g.out = out;
    g.R = rows[idx];
    g.K = pl.K;
    g.B = batch;
    g.S = h->bsplit[idx];
    g.layer = layer;
    g.kp = pl.kp;
    g.rpc = pl.rpc;
    g.kb_piece = ceil_div(pl.kp, (uint32_t)BG_TILE_K);
    if (pl.npieces == 1) {
        g.pieces = 0;
        g.nkb = ceil_div(pl.K, (uint32_t)BG_TILE_K);
    } else {
        g.pieces = pl.npieces;
        g.nkb = (pl.npieces - 1) * g.kb_piece + ceil_div(pl.K - (pl.npieces - 1) * pl.kp, (uint32_t)BG_TILE_K);
    }
    const bool normed = idx == 0 || idx == 2 || idx == 4;   // inputs that are RMSNorm outputs: the factor is applied here
    g.ssq = normed ? h->bssq : nullptr;
    g.ssq_n = ceil_div(p.H, (uint32_t)BV_CHUNK);
    g.eps = p.eps;
    g.status = p.status;
    g.wait_ns = p.wait_ns;
    // the projections of the layers run on the stream schedule (every CTA the same share of the K blocks of all
    // tiles); the classifier writes its result directly and keeps whole tiles
    const uint32_t ntiles = ceil_div(g.R, (uint32_t)BG_TILE_M), T = ntiles * g.nkb;
    g.stream = (idx != 4 && h->use_stream && T >= (uint32_t)h->num_sms) ? 1u : 0u;
    const uint32_t items = g.stream ? T : ntiles * g.S;
    const uint32_t grid = items < (uint32_t)h->num_sms ? items : (uint32_t)h->num_sms;
    if (parts) {
        parts->part = out;
        parts->R = g.R;
        parts->S = g.S;
        parts->stream = g.stream;
        parts->nkb = g.nkb;
        parts->T = T;
        parts->P = grid;
    }
    if (launch_dependent(h->use_pdl, kl_bgemm_kernel, dim3(grid), dim3(BG_THREADS), BG_SMEM_BYTES, st, g) != cudaSuccess) return KL_ERR_CUDA;
    ++h->launches;
    return KL_OK;
}

static void drop_batched_graph(kl_handle* h) {
    if (h->bgraph) cudaGraphExecDestroy(h->bgraph);
    h->bgraph = nullptr;
    h->bgraph_kv = nullptr;
    h->bgraph_tok = h->bgraph_pos = nullptr;
    h->bgraph_logits = nullptr;
    h->bgraph_batch = 0;
}

// Decode step of a batch on the tensor-core path: one launch per operator group, every weight matrix streamed once.
static kl_status decode_step_batched(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d,
                                     float* logits_d, uint32_t batch, cudaStream_t st) {
    const Params& p = h->prm;
    BAttnParams a;
    const kl_status trc = encode_kv_map4(h, &a.kv_map, kv_cache_d, batch, BA_SLOT_BYTES);
    if (trc != KL_OK) return trc;
    a.kv = reinterpret_cast<__nv_bfloat16*>(kv_cache_d);
    a.positions = positions_d;
    a.cs = p.rope_cs;
    a.q = h->bq;
    a.part_o = h->bao;
    a.part_ml = h->baml;
    a.xop = h->bxop[1];
    a.QD = p.QD; a.KVD = p.KVD; a.nq = p.nq; a.nkv = p.nkv; a.G = p.G; a.hd = p.hd;
    a.bias = nullptr;
    BgPartials parts = {};   // of the latest projection; part == nullptr: nothing to add
    a.B = batch;
    a.max_ctx = h->desc.max_ctx;
    a.NW = (uint32_t)h->num_sms * BA_WARPS;
    a.status = p.status;
    a.wait_ns = p.wait_ns;
    const size_t ba_smem = batched_attn_smem();
    cudaEvent_t* ev = h->prof_capacity ? h->prof_events + 3 * (h->prof_steps++ % h->prof_capacity) : nullptr;
    kl_status rc;
#define KL_B_LAUNCH(kernel, grid, block, smem, ...)                                                              \
    do {                                                                                                         \
        if (launch_dependent(h->use_pdl, kernel, dim3(grid), dim3(block), smem, st, __VA_ARGS__) != cudaSuccess) return KL_ERR_CUDA; \
        ++h->launches;                                                                                           \
    } while (0)
    KL_B_LAUNCH(kl_b_embed_kernel, batch, 256, 0, tokens_d, positions_d, p.embed, h->bx, p.H, p.V, h->desc.max_ctx, p.inv_freq,
                p.rope_cs, p.hd / 2, p.status);
    if (ev && cudaEventRecord(ev[0], st) != cudaSuccess) return KL_ERR_CUDA;
    const dim3 grid_h(batch, ceil_div(p.H, (uint32_t)BV_CHUNK)), grid_f(batch, ceil_div(p.F, (uint32_t)BV_CHUNK));
    for (uint32_t l = 0; l < p.L; ++l) {
        const size_t lo = (size_t)l * p.layer_stride;
        a.layer = l;
        a.bias = p.bqkv ? p.bqkv + lo : nullptr;
        // x += down projection of the previous layer; operand = g1 * x, sums of squares for the RMSNorm factor
        KL_B_LAUNCH(kl_b_finish_kernel, grid_h, 256, 0, parts, h->bx, h->bx, p.g1 + lo, 0, p.H, h->bxop[0], h->bssq, p.status);
        if ((rc = launch_bgemm(h, 0, l, h->bpart, batch, st, &a.qkv)) != KL_OK) return rc;
        KL_B_LAUNCH(kl_b_rope_kernel, dim3(batch, p.nq + 2 * p.nkv), 128, 0, a);
        KL_B_LAUNCH(kl_b_attn_kernel, (uint32_t)h->num_sms, BA_THREADS, ba_smem, a);
        KL_B_LAUNCH(kl_b_attn_merge_kernel, dim3(p.nq, batch), p.hd / 2, 0, a);
        if ((rc = launch_bgemm(h, 1, l, h->bpart, batch, st, &parts)) != KL_OK) return rc;
        // x += attention output projection; operand = g2 * x
        KL_B_LAUNCH(kl_b_finish_kernel, grid_h, 256, 0, parts, h->bx, h->bx, p.g2 + lo, 0, p.H, h->bxop[0], h->bssq, p.status);
        if ((rc = launch_bgemm(h, 2, l, h->bpart, batch, st, &parts)) != KL_OK) return rc;
        // operand = silu(gate) * up
        KL_B_LAUNCH(kl_b_finish_kernel, grid_f, 256, 0, parts, nullptr, nullptr, nullptr, 1, p.F, h->bxop[2], nullptr, p.status);
        if ((rc = launch_bgemm(h, 3, l, h->bpart, batch, st, &parts)) != KL_OK) return rc;
    }
    if (ev && cudaEventRecord(ev[1], st) != cudaSuccess) return KL_ERR_CUDA;
    // x += last down projection (kept for kl_read_hidden); operand = gf * x; logits = RMSNorm factor * W_lm . operand
    KL_B_LAUNCH(kl_b_finish_kernel, grid_h, 256, 0, parts, h->bx, h->bx, p.gf, 0, p.H, h->bxop[0], h->bssq, p.status);
    if ((rc = launch_bgemm(h, 4, 0, logits_d, batch, st)) != KL_OK) return rc;
    if (ev && cudaEventRecord(ev[2], st) != cudaSuccess) return KL_ERR_CUDA;
#undef KL_B_LAUNCH
    return KL_OK;
}

// Decode step of a batch as the looped kernel: one cooperative launch for the whole step (KL_MODE_LOOPED), or one
// launch per layer from the same kernel (KL_MODE_PER_LAYER).
static kl_status decode_step_batched_looped(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d,
                                            float* logits_d, uint32_t batch, cudaStream_t st, bool per_layer) {
    const Params& p = h->prm;
    BLoopParams* b = new (std::nothrow) BLoopParams();   // 2.3 KB of kernel parameters (fourteen tensor maps)
    if (!b) return KL_ERR_INVALID_ARG;
    struct Free { BLoopParams* p; ~Free() { delete p; } } guard{b};
    const kl_status trc = encode_kv_map4(h, &b->kv_map, kv_cache_d, batch, BA_SLOT_BYTES);
    if (trc != KL_OK) return trc;
    static const int plan_of[5] = {PL_QKV, PL_O, PL_GU, PL_D, PL_LM};
    static const uint32_t xmap_of[5] = {0, 1, 0, 2, 0};
    const uint32_t rows[5] = {p.QD + 2 * p.KVD, p.H, 2 * p.F, p.H, p.V};
    for (int i = 0; i < 5; ++i) {
        b->map_w[i] = h->bmap_w[i];
        b->map_wl[i] = h->bmap_wl[i];
        const GemvPlan& pl = p.plan[plan_of[i]];
        BlGemm& g = b->g[i];
        g.R = rows[i];
        g.K = pl.K;
        g.S = h->bsplit[i];
        g.kp = pl.kp;
        g.rpc = pl.rpc;
        g.kb_piece = ceil_div(pl.kp, (uint32_t)BG_TILE_K);
        if (pl.npieces == 1) {
            g.pieces = 0;
            g.nkb = ceil_div(pl.K, (uint32_t)BG_TILE_K);
        } else {
            g.pieces = pl.npieces;
            g.nkb = (pl.npieces - 1) * g.kb_piece + ceil_div(pl.K - (pl.npieces - 1) * pl.kp, (uint32_t)BG_TILE_K);
        }
        const uint32_t T = ceil_div(g.R, (uint32_t)BG_TILE_M) * g.nkb;
        g.stream = (i != 4 && h->use_stream && T >= (uint32_t)h->num_sms) ? 1u : 0u;
        g.xmap = xmap_of[i];
        g.normed = (i == 0 || i == 2 || i == 4) ? 1u : 0u;
    }
    for (int i = 0; i < 3; ++i) {
        b->map_x[i] = h->bmap_x[i];
        b->xop[i] = h->bxop[i];
    }
    b->tokens = tokens_d; b->positions = positions_d;
    b->embed = p.embed; b->g1 = p.g1; b->g2 = p.g2; b->gf = p.gf; b->bqkv = p.bqkv;
    b->layer_stride = p.layer_stride;
    b->x = h->bx; b->ssq = h->bssq; b->part = h->bpart; b->q = h->bq; b->part_o = h->bao; b->part_ml = h->baml;
    b->logits = logits_d; b->rope_cs = p.rope_cs; b->inv_freq = p.inv_freq;
    b->kv = reinterpret_cast<__nv_bfloat16*>(kv_cache_d);
    b->H = p.H; b->QD = p.QD; b->KVD = p.KVD; b->F = p.F; b->V = p.V; b->nq = p.nq; b->nkv = p.nkv; b->G = p.G; b->hd = p.hd;
    b->B = batch; b->max_ctx = h->desc.max_ctx;
    b->NW = (uint32_t)h->num_sms * BA_WARPS;
    b->eps = p.eps;
    b->status = p.status;
    b->wait_ns = p.wait_ns;
    if (cudaMemsetAsync(h->bbar, 0, ((size_t)p.L + 1) * 16 * 4, st) != cudaSuccess) return KL_ERR_CUDA;
    cudaEvent_t* ev = h->prof_capacity ? h->prof_events + 3 * (h->prof_steps++ % h->prof_capacity) : nullptr;
    if (ev && cudaEventRecord(ev[0], st) != cudaSuccess) return KL_ERR_CUDA;
    const uint32_t nlaunch = per_layer ? p.L : 1u;
    for (uint32_t i = 0; i < nlaunch; ++i) {
        b->l0 = per_layer ? i : 0u;
        b->l1 = per_layer ? i + 1u : p.L;
        b->first = i == 0 ? 1u : 0u;
        b->last = i + 1u == nlaunch ? 1u : 0u;
        b->bar = h->bbar + (size_t)i * 16;
        void* args[] = {b};
        if (cudaLaunchCooperativeKernel((const void*)kl_bloop_kernel, dim3(h->num_sms), dim3(BL_THREADS), args, BL_SMEM_BYTES, st) != cudaSuccess)
            return KL_ERR_CUDA;
        ++h->launches;
    }
    // the classifier is part of the (last) launch: both marks behind it
    if (ev && (cudaEventRecord(ev[1], st) != cudaSuccess || cudaEventRecord(ev[2], st) != cudaSuccess)) return KL_ERR_CUDA;
    return KL_OK;
}

// A batched step on the schedule kl_set_mode selected: the looped kernel (one launch), the same kernel launched per
// layer, or one launch per operator group.
static kl_status batched_step(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d, float* logits_d,
                              uint32_t batch, cudaStream_t st) {
    // Until kl_set_mode says otherwise a batch takes the per-operator schedule: with programmatic dependent launch its
    // kernel boundaries cost less on this GPU than the grid barriers that replace them in the looped kernel (measured).
    const int mode = h->mode_explicit ? h->mode : KL_MODE_PER_STAGE;
    if (h->bl_ok && mode != KL_MODE_PER_STAGE)
        return decode_step_batched_looped(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, st, mode == KL_MODE_PER_LAYER);
    return decode_step_batched(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, st);
}

// The instantiation a launch takes: mixture of experts, stash mode (1: chunks of 2048 / 4096 columns only, 2: all
// widths), the debug hooks (trace stamps, jitter) only while one of them is set, the CUDA-core attention loops only
// when the launch runs them.
static const void* token_fn(const kl_handle* h, const Params& p) {
    const bool dbg = p.jitter_seed != 0u || p.trace != nullptr, cc = !p.attn_tc;
    if (p.n_experts) return cc ? (const void*)kl_token_kernel<false, true, 0, true> : (const void*)kl_token_kernel<false, true, 0, false>;
    if (h->stash == 1) return dbg ? (const void*)kl_token_kernel<true, false, 1, false> : (const void*)kl_token_kernel<false, false, 1, false>;
    if (h->stash == 2) return dbg ? (const void*)kl_token_kernel<true, false, 2, false> : (const void*)kl_token_kernel<false, false, 2, false>;
    if (cc) return dbg ? (const void*)kl_token_kernel<true, false, 0, true> : (const void*)kl_token_kernel<false, false, 0, true>;
    return dbg ? (const void*)kl_token_kernel<true, false, 0, false> : (const void*)kl_token_kernel<false, false, 0, false>;
}
static const void* decoder_fn(const kl_handle* h, const Params& p) {
    const bool dbg = p.trace != nullptr || p.jitter_seed != 0u, cc = !p.attn_tc;
    if (p.n_experts) return cc ? (const void*)kl_decoder_kernel<false, true, 0, true> : (const void*)kl_decoder_kernel<false, true, 0, false>;
    if (h->stash == 1) return dbg ? (const void*)kl_decoder_kernel<true, false, 1, false> : (const void*)kl_decoder_kernel<false, false, 1, false>;
    if (h->stash == 2) return dbg ? (const void*)kl_decoder_kernel<true, false, 2, false> : (const void*)kl_decoder_kernel<false, false, 2, false>;
    if (cc) return dbg ? (const void*)kl_decoder_kernel<true, false, 0, true> : (const void*)kl_decoder_kernel<false, false, 0, true>;
    return dbg ? (const void*)kl_decoder_kernel<true, false, 0, false> : (const void*)kl_decoder_kernel<false, false, 0, false>;
}
static const void* classifier_fn(const kl_handle* h) {
    return h->stash == 1 ? (const void*)kl_classifier_kernel<1> : h->stash == 2 ? (const void*)kl_classifier_kernel<2>
                                                                                  : (const void*)kl_classifier_kernel<0>;
}

kl_status kl_decode_step(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d,
                         float* logits_d, uint32_t batch, void* stream) {
    if (!h || !tokens_d || !positions_d || !kv_cache_d || !logits_d) return KL_ERR_INVALID_ARG;
    if (batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    if (!all_loaded(h)) return KL_ERR_NOT_LOADED;
    cudaStream_t st = as_stream(stream);
    h->chain_tok = nullptr;   // whatever kl_decode_greedy prepared for its next launch is overwritten by this step
    if (batch > 1 && h->bt_ok && h->use_bt) {
        h->last_batch = batch;
        return batched_step(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, st);
    }
    Params p = h->prm;
    p.B = batch;
    p.cps = (uint32_t)h->num_sms / p.nkv;
    p.tokens = tokens_d;
    p.positions = positions_d;
    p.kv = reinterpret_cast<__nv_bfloat16*>(kv_cache_d);
    p.skip_stage = h->pending_skip_stage;
    h->pending_skip_stage = -1;
    p.attn_tc = 0;
    if (h->use_tc_attention && (p.hd == 64 || p.hd == 128)) {
        kl_status trc = encode_kv_map(h, &p.kv_map, kv_cache_d, batch);
        if (trc == KL_OK) trc = encode_kv_map4(h, &p.kv_map4, kv_cache_d, batch);
        if (trc != KL_OK) return trc;
        p.attn_tc = 1;
    }
    h->last_batch = batch;
    h->hidden_is_copy = 0;
    h->chain_tok = nullptr;
    cudaEvent_t* ev = h->prof_capacity ? h->prof_events + 3 * (h->prof_steps++ % h->prof_capacity) : nullptr;
    // Sequences of a batch are independent: without the batched path the batch-1 kernels decode them one after
    // another (the weights are streamed once per sequence).
    for (uint32_t b = 0; b < batch; ++b) {
        p.b0 = b;
        p.logits = logits_d + (size_t)b * p.V;
        kl_embed_kernel<<<1, 256, 0, st>>>(p);
        if (cudaGetLastError() != cudaSuccess) return KL_ERR_CUDA;
        ++h->launches;
        kl_status rc;
        if (ev && b == 0 && cudaEventRecord(ev[0], st) != cudaSuccess) return KL_ERR_CUDA;
        uint32_t sbeg = 0, send = 5;
        // the instantiation with the trace stamps compiled in only while a trace buffer is set
        const void* decoder_fn = ::decoder_fn(h, p);
        if (h->mode == KL_MODE_LOOPED) {
            uint32_t l0 = 0, l1 = p.L;
            void* args[] = {&p, &l0, &l1, &sbeg, &send};
            if ((rc = launch_persistent(h, decoder_fn, args, st)) != KL_OK) return rc;
        } else if (h->mode == KL_MODE_PER_LAYER) {
            for (uint32_t l = 0; l < p.L; ++l) {
                uint32_t l0 = l, l1 = l + 1;
                void* args[] = {&p, &l0, &l1, &sbeg, &send};
                if ((rc = launch_persistent(h, decoder_fn, args, st)) != KL_OK) return rc;
            }
        } else {
            for (uint32_t l = 0; l < p.L; ++l)
                for (uint32_t sg = 0; sg < (p.n_experts ? 4u : 5u); ++sg) {
                    // mixture of experts: the down projection needs the router's choice, which lives in the launch
                    // that made it -- gate/up and down stay together
                    uint32_t l0 = l, l1 = l + 1, s0 = sg, s1 = (p.n_experts && sg == 3) ? 5u : sg + 1;
                    void* args[] = {&p, &l0, &l1, &s0, &s1};
                    if ((rc = launch_persistent(h, decoder_fn, args, st)) != KL_OK) return rc;
                }
        }
        if (ev && b == 0 && cudaEventRecord(ev[1], st) != cudaSuccess) return KL_ERR_CUDA;
        {
            Params pc = p;
            pc.chunk_trace = nullptr;  // the chunk log covers the decoder kernel only
            void* cargs[] = {&pc};
            if ((rc = launch_persistent(h, classifier_fn(h), cargs, st)) != KL_OK) return rc;
        }
        if (ev && b == 0 && cudaEventRecord(ev[2], st) != cudaSuccess) return KL_ERR_CUDA;
        if (batch > 1) {
            // keep this sequence's hidden state (the value half of every tagged word) for kl_read_hidden
            if (cudaMemcpy2DAsync(h->hidden_all + (size_t)b * p.H, 4, p.xa, 8, 4, p.H, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return KL_ERR_CUDA;
        }
    }
    return KL_OK;
}

// A batched step replayed from the handle's cached CUDA graph: captured once per set of buffers (tokens, positions,
// cache, logits, batch) on a stream of its own, where nothing executes.  False: not replayed (profiling is on, `st`
// is itself being captured, or the capture was refused) -- the caller launches the step kernel by kernel.
static bool replay_batched(kl_handle* h, const int32_t* tokens_d, const int32_t* positions_d, void* kv_cache_d, float* logits_d,
                           uint32_t batch, cudaStream_t st) {
    if (!(batch > 1 && h->bt_ok && h->use_bt && !h->prof_capacity && all_loaded(h))) return false;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
        (void)cudaGetLastError();
        return false;
    }
    if (!h->bgraph || h->bgraph_kv != kv_cache_d || h->bgraph_batch != batch || h->bgraph_tok != tokens_d ||
        h->bgraph_pos != positions_d || h->bgraph_logits != logits_d) {
        drop_batched_graph(h);
        if (!h->cap_stream && cudaStreamCreateWithFlags(&h->cap_stream, cudaStreamNonBlocking) != cudaSuccess) h->cap_stream = nullptr;
        if (h->cap_stream && cudaStreamBeginCapture(h->cap_stream, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
            const uint64_t l0 = h->launches;
            const kl_status crc = batched_step(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, h->cap_stream);
            cudaGraph_t graph = nullptr;
            const cudaError_t e = cudaStreamEndCapture(h->cap_stream, &graph);
            h->bgraph_launches = h->launches - l0;
            h->launches = l0;   // captured, not launched
            if (crc == KL_OK && e == cudaSuccess && graph && cudaGraphInstantiate(&h->bgraph, graph, 0) == cudaSuccess) {
                h->bgraph_kv = kv_cache_d;
                h->bgraph_batch = batch;
                h->bgraph_tok = tokens_d;
                h->bgraph_pos = positions_d;
                h->bgraph_logits = logits_d;
            } else {
                h->bgraph = nullptr;
            }
            if (graph) cudaGraphDestroy(graph);
        }
        (void)cudaGetLastError();   // a refused capture is not an error
    }
    if (h->bgraph && cudaGraphLaunch(h->bgraph, st) == cudaSuccess) {
        h->launches += h->bgraph_launches;
        h->last_batch = batch;
        h->chain_tok = nullptr;
        return true;
    }
    return false;
}

// Parameters of a batch-1 launch that samples on the device; starts a chain (embedding, rotary table, step counter as
// in kl_decode_step; sampling ticket at zero) unless the latest launch already prepared this token buffer's next step.
static kl_status token_chain_params(kl_handle* h, Params* out, int32_t* tokens_d, int32_t* positions_d, void* kv_cache_d,
                                    float* logits_d, int restart, cudaStream_t st) {
    Params p = h->prm;
    p.B = 1;
    p.b0 = 0;
    p.cps = (uint32_t)h->num_sms / p.nkv;
    p.tokens = tokens_d;
    p.positions = positions_d;
    p.kv = reinterpret_cast<__nv_bfloat16*>(kv_cache_d);
    p.logits = logits_d;
    p.skip_stage = h->pending_skip_stage;   // test hook of the bounded waits: applies to the next launch only
    h->pending_skip_stage = -1;
    // the stage stamps of kl_set_trace are taken here too (decoder layers only); the chunk log is not
    p.chunk_trace = nullptr;
    p.attn_tc = 0;
    if (h->use_tc_attention && (p.hd == 64 || p.hd == 128)) {
        kl_status trc = encode_kv_map(h, &p.kv_map, kv_cache_d, 1);
        if (trc == KL_OK) trc = encode_kv_map4(h, &p.kv_map4, kv_cache_d, 1);
        if (trc != KL_OK) return trc;
        p.attn_tc = 1;
    }
    if (restart || h->chain_tok != tokens_d) {
        if (cudaMemsetAsync(h->tok_ticket, 0, 4, st) != cudaSuccess) return KL_ERR_CUDA;   // a launch that gave up may have left it anywhere
        kl_embed_kernel<<<1, 256, 0, st>>>(p);
        if (cudaGetLastError() != cudaSuccess) return KL_ERR_CUDA;
        ++h->launches;
    }
    *out = p;
    return KL_OK;
}

kl_status kl_decode_greedy(kl_handle* h, int32_t* tokens_d, int32_t* positions_d, void* kv_cache_d, float* logits_d,
                           uint32_t batch, int restart, void* stream) {
    if (!h || !tokens_d || !positions_d || !kv_cache_d || !logits_d) return KL_ERR_INVALID_ARG;
    if (batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    if (batch > 1 || !h->token_ok) {
        // batches (and devices on which the one-launch kernel cannot be resident): the step, then the sampling kernel
        kl_status rc = KL_OK;
        if (!replay_batched(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, as_stream(stream)))
            rc = kl_decode_step(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, stream);
        return rc != KL_OK ? rc : kl_argmax_advance(h, logits_d, tokens_d, positions_d, batch, stream);
    }
    if (!all_loaded(h)) return KL_ERR_NOT_LOADED;
    cudaStream_t st = as_stream(stream);
    Params p;
    const kl_status prc = token_chain_params(h, &p, tokens_d, positions_d, kv_cache_d, logits_d, restart, st);
    if (prc != KL_OK) return prc;
    TokenParams t = {tokens_d, positions_d, h->tok_val, h->tok_idx, h->tok_ticket, h->hidden_all, nullptr, 1u, p.rope_cs};
    void* args[] = {&p, &t};
    const kl_status rc = launch_persistent(h, token_fn(h, p), args, st);
    if (rc != KL_OK) return rc;
    h->last_batch = 1;
    h->hidden_is_copy = 1;
    h->chain_tok = tokens_d;
    return KL_OK;
}

kl_status kl_decode_greedy_tokens(kl_handle* h, int32_t* tokens_d, int32_t* positions_d, void* kv_cache_d, float* logits_d,
                                  int32_t* out_tokens_d, uint32_t n_tokens, uint32_t batch, int restart, void* stream) {
    if (!h || !tokens_d || !positions_d || !kv_cache_d || !logits_d || !out_tokens_d) return KL_ERR_INVALID_ARG;
    if (batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    if (batch > 1 || !h->token_ok) {
        // batches: token after token (each step replayed from the handle's graph), the picked tokens copied out
        for (uint32_t k = 0; k < n_tokens; ++k) {
            const kl_status rc = kl_decode_greedy(h, tokens_d, positions_d, kv_cache_d, logits_d, batch, restart && k == 0, stream);
            if (rc != KL_OK) return rc;
            if (cudaMemcpyAsync(out_tokens_d + (size_t)k * batch, tokens_d, (size_t)batch * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return KL_ERR_CUDA;
        }
        return KL_OK;
    }
    if (!all_loaded(h)) return KL_ERR_NOT_LOADED;
    for (uint32_t done = 0; done < n_tokens;) {
        const uint32_t K = n_tokens - done < TOKENS_PER_LAUNCH ? n_tokens - done : (uint32_t)TOKENS_PER_LAUNCH;
        Params p;
        const kl_status prc = token_chain_params(h, &p, tokens_d, positions_d, kv_cache_d, logits_d, restart && done == 0, st);
        if (prc != KL_OK) return prc;
        kl_token_plan_kernel<<<1, 256, 0, st>>>(p, h->plan_rope, K);
        if (cudaGetLastError() != cudaSuccess) return KL_ERR_CUDA;
        ++h->launches;
        TokenParams t = {tokens_d, positions_d, h->tok_val, h->tok_idx, h->tok_ticket, h->hidden_all, out_tokens_d + done, K, h->plan_rope};
        void* args[] = {&p, &t};
        const kl_status rc = launch_persistent(h, token_fn(h, p), args, st);
        if (rc != KL_OK) return rc;
        h->last_batch = 1;
        h->hidden_is_copy = 1;
        h->chain_tok = tokens_d;
        done += K;
    }
    return KL_OK;
}

kl_status kl_decode_greedy_tokens_host(kl_handle* h, int32_t token, int32_t position, void* kv_cache_d, int32_t* out_tokens_h,
                                       uint32_t n_tokens, void* stream) {
    if (!h || !kv_cache_d || !out_tokens_h || n_tokens == 0 || n_tokens > TOKENS_PER_LAUNCH) return KL_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(h->stage_tokens, &token, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
    if (cudaMemcpyAsync(h->stage_positions, &position, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
    int32_t* out_d = h->plan_out;
    const kl_status rc = kl_decode_greedy_tokens(h, h->stage_tokens, h->stage_positions, kv_cache_d, h->stage_logits, out_d, n_tokens, 1, 1, stream);
    if (rc != KL_OK) return rc;
    if (cudaMemcpyAsync(out_tokens_h, out_d, (size_t)n_tokens * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KL_ERR_CUDA;
    return KL_OK;
}

// Tokens and positions from the host into the staging buffers, then one step into the staging logits (a batched
// step replayed from its cached graph).
static kl_status host_step(kl_handle* h, const int32_t* tokens_h, const int32_t* positions_h, void* kv_cache_d, uint32_t batch,
                           void* stream) {
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(h->stage_tokens, tokens_h, batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
    if (cudaMemcpyAsync(h->stage_positions, positions_h, batch * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
    if (replay_batched(h, h->stage_tokens, h->stage_positions, kv_cache_d, h->stage_logits, batch, st)) return KL_OK;
    return kl_decode_step(h, h->stage_tokens, h->stage_positions, kv_cache_d, h->stage_logits, batch, stream);
}

kl_status kl_decode_step_host(kl_handle* h, const int32_t* tokens_h, const int32_t* positions_h, void* kv_cache_d,
                              float* logits_h, uint32_t batch, void* stream) {
    if (!h || !tokens_h || !positions_h || !kv_cache_d || !logits_h) return KL_ERR_INVALID_ARG;
    if (batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    const kl_status rc = host_step(h, tokens_h, positions_h, kv_cache_d, batch, stream);
    if (rc != KL_OK) return rc;
    if (cudaMemcpyAsync(logits_h, h->stage_logits, (size_t)batch * h->prm.V * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return KL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KL_ERR_CUDA;
    return KL_OK;
}

kl_status kl_decode_greedy_host(kl_handle* h, const int32_t* tokens_h, const int32_t* positions_h, void* kv_cache_d,
                                int32_t* next_tokens_h, uint32_t batch, void* stream) {
    if (!h || !tokens_h || !positions_h || !kv_cache_d || !next_tokens_h) return KL_ERR_INVALID_ARG;
    if (batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    kl_status rc;
    if (batch == 1 && h->token_ok) {
        // one sequence: embedding, then decoder layers + classifier + sampling as one kernel (the tokens come from the
        // host every call, so every call starts a chain)
        if (cudaMemcpyAsync(h->stage_tokens, tokens_h, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
        if (cudaMemcpyAsync(h->stage_positions, positions_h, 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return KL_ERR_CUDA;
        if ((rc = kl_decode_greedy(h, h->stage_tokens, h->stage_positions, kv_cache_d, h->stage_logits, 1, 1, stream)) != KL_OK)
            return rc;
    } else {
        if ((rc = host_step(h, tokens_h, positions_h, kv_cache_d, batch, stream)) != KL_OK) return rc;
        // greedy sampling on the device: the staging tokens become the next tokens (the staging positions advance too)
        if ((rc = kl_argmax_advance(h, h->stage_logits, h->stage_tokens, h->stage_positions, batch, stream)) != KL_OK) return rc;
    }
    if (cudaMemcpyAsync(next_tokens_h, h->stage_tokens, batch * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KL_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KL_ERR_CUDA;
    return KL_OK;
}

kl_status kl_argmax_advance(kl_handle* h, const float* logits_d, int32_t* tokens_d, int32_t* positions_d, uint32_t batch,
                            void* stream) {
    if (!h || !logits_d || !tokens_d || !positions_d || batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    kl_argmax_kernel<<<dim3(ARGMAX_BLOCKS, batch), 256, 0, as_stream(stream)>>>(logits_d, h->prm.V, tokens_d, positions_d,
                                                                                 h->argmax_val, h->argmax_idx, h->argmax_tickets);
    if (cudaGetLastError() != cudaSuccess) return KL_ERR_CUDA;
    ++h->launches;
    return KL_OK;
}

// ---- sampling block without a handle and without any allocation.
// Some callers have no arena to lend: a sampler working on logits that came from elsewhere owns no kl_handle, and a
// serving process that has handed all device memory to its own pools can neither afford the device-wide
// synchronisation of an allocation nor expect it to succeed.  For them the partial results and the tickets of the
// argmax kernel sit in the array below, which is part of the module image on every device that loads it.
// Layout: [MAX_BATCH][ARGMAX_BLOCKS] fp32 maxima | [MAX_BATCH][ARGMAX_BLOCKS] u32 indices | [MAX_BATCH] u32 tickets.
namespace {
constexpr size_t STATIC_ARGMAX_PART = (size_t)KL_STATIC_ARGMAX_MAX_BATCH * ARGMAX_BLOCKS * 4;
constexpr size_t STATIC_ARGMAX_BYTES = 2 * STATIC_ARGMAX_PART + (size_t)KL_STATIC_ARGMAX_MAX_BATCH * 4;
constexpr int STATIC_MAX_DEVICES = 64;
}  // namespace
static __device__ __align__(256) unsigned char kl_static_argmax_scratch[STATIC_ARGMAX_BYTES];
static unsigned char* g_static_argmax_ptr[STATIC_MAX_DEVICES];   // per device; written once under the mutex
static std::mutex g_static_argmax_mutex;

kl_status kl_argmax_advance_static(const float* logits_d, uint32_t vocab, int32_t* tokens_d, int32_t* positions_d,
                                   uint32_t batch, void* stream) {
    if (!logits_d || !tokens_d || !positions_d || batch == 0 || vocab == 0) return KL_ERR_INVALID_ARG;
    if (batch > (uint32_t)KL_STATIC_ARGMAX_MAX_BATCH) return KL_ERR_TOO_LARGE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return KL_ERR_CUDA;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return KL_ERR_INVALID_ARG;
    unsigned char* base;
    {
        // set-up, once per device, with that device current: the address of this device's copy of the array
        std::lock_guard<std::mutex> lock(g_static_argmax_mutex);
        if (!g_static_argmax_ptr[dev]) {
            unsigned char* ptr = nullptr;
            if (cudaGetSymbolAddress((void**)&ptr, kl_static_argmax_scratch) != cudaSuccess || !ptr) return KL_ERR_CUDA;
            g_static_argmax_ptr[dev] = ptr;
        }
        base = g_static_argmax_ptr[dev];
    }
    float* part_val = reinterpret_cast<float*>(base);
    uint32_t* part_idx = reinterpret_cast<uint32_t*>(base + STATIC_ARGMAX_PART);
    uint32_t* tickets = reinterpret_cast<uint32_t*>(base + 2 * STATIC_ARGMAX_PART);
    cudaStream_t st = as_stream(stream);
    // the array keeps what the previous call left; only the tickets have to start at zero
    if (cudaMemsetAsync(tickets, 0, (size_t)batch * 4, st) != cudaSuccess) return KL_ERR_CUDA;
    kl_argmax_kernel<<<dim3(ARGMAX_BLOCKS, batch), 256, 0, st>>>(logits_d, vocab, tokens_d, positions_d, part_val, part_idx,
                                                                  tickets);
    if (cudaGetLastError() != cudaSuccess) return KL_ERR_CUDA;
    return KL_OK;
}

kl_status kl_read_hidden(kl_handle* h, float* hidden_d, uint32_t batch, void* stream) {
    if (!h || !hidden_d || batch == 0 || batch > h->desc.max_batch) return KL_ERR_INVALID_ARG;
    if (batch != h->last_batch) return KL_ERR_INVALID_ARG;
    cudaError_t e;
    if (batch == 1 && !h->hidden_is_copy)   // the hidden state leaving the last layer is an array of tagged words: the value halves
        e = cudaMemcpy2DAsync(hidden_d, 4, h->prm.xa, 8, 4, h->prm.H, cudaMemcpyDeviceToDevice, as_stream(stream));
    else
        e = cudaMemcpyAsync(hidden_d, h->hidden_all, (size_t)batch * h->prm.H * 4, cudaMemcpyDeviceToDevice, as_stream(stream));
    if (e != cudaSuccess) return KL_ERR_CUDA;
    return KL_OK;
}

kl_status kl_last_status(kl_handle* h) {
    if (!h) return KL_ERR_INVALID_ARG;
    int32_t v = 0;
    if (cudaMemcpy(&v, h->prm.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return KL_ERR_CUDA;
    if (v != 0) {
        const int32_t zero = 0;
        if (cudaMemcpy(h->prm.status, &zero, 4, cudaMemcpyHostToDevice) != cudaSuccess) return KL_ERR_CUDA;
        h->chain_tok = nullptr;   // whatever a chain of kl_decode_greedy had prepared is not to be trusted: the next call starts one
    }
    return (kl_status)v;
}

uint64_t kl_launch_count(const kl_handle* h) { return h ? h->launches : 0; }

kl_status kl_profile_enable(kl_handle* h, uint32_t capacity) {
    if (!h) return KL_ERR_INVALID_ARG;
    if (h->prof_events) {
        for (uint32_t i = 0; i < 3 * h->prof_capacity; ++i) cudaEventDestroy(h->prof_events[i]);
        free(h->prof_events);
        h->prof_events = nullptr;
    }
    h->prof_capacity = 0;
    h->prof_steps = 0;
    if (capacity == 0) return KL_OK;
    h->prof_events = (cudaEvent_t*)calloc(3 * (size_t)capacity, sizeof(cudaEvent_t));
    if (!h->prof_events) return KL_ERR_INVALID_ARG;
    for (uint32_t i = 0; i < 3 * capacity; ++i) {
        if (cudaEventCreate(&h->prof_events[i]) != cudaSuccess) {
            for (uint32_t j = 0; j < i; ++j) cudaEventDestroy(h->prof_events[j]);
            free(h->prof_events);
            h->prof_events = nullptr;
            return KL_ERR_CUDA;
        }
    }
    h->prof_capacity = capacity;
    return KL_OK;
}

kl_status kl_profile_read(kl_handle* h, uint32_t* n, float* decoder_ms, float* classifier_ms) {
    if (!h || !n || !decoder_ms || !classifier_ms) return KL_ERR_INVALID_ARG;
    const uint64_t have = h->prof_steps < h->prof_capacity ? h->prof_steps : h->prof_capacity;
    const uint32_t cnt = (uint32_t)(have < *n ? have : *n);
    for (uint32_t i = 0; i < cnt; ++i) {
        cudaEvent_t* ev = h->prof_events + 3 * ((h->prof_steps - 1 - i) % h->prof_capacity);
        if (cudaEventElapsedTime(&decoder_ms[i], ev[0], ev[1]) != cudaSuccess) return KL_ERR_CUDA;
        if (cudaEventElapsedTime(&classifier_ms[i], ev[1], ev[2]) != cudaSuccess) return KL_ERR_CUDA;
    }
    *n = cnt;
    return KL_OK;
}

kl_status kl_set_wait_limit_ns(kl_handle* h, uint64_t ns) {
    if (!h || ns == 0) return KL_ERR_INVALID_ARG;
    h->prm.wait_ns = ns;
    drop_batched_graph(h);   // the limit is a kernel argument
    return KL_OK;
}

kl_status kl_set_trace(kl_handle* h, uint64_t* trace_d, uint32_t* n_ctas, uint32_t* n_layers, uint32_t* n_stamps) {
    if (!h) return KL_ERR_INVALID_ARG;
    h->prm.trace = reinterpret_cast<unsigned long long*>(trace_d);
    // the per-chunk log of CTA 0 follows the stage stamps in the same buffer
    h->prm.chunk_trace = trace_d ? h->prm.trace + (size_t)h->prm.P * h->prm.L * TRACE_STAMPS : nullptr;
    if (n_ctas) *n_ctas = h->prm.P;
    if (n_layers) *n_layers = h->prm.L;
    if (n_stamps) *n_stamps = TRACE_STAMPS;
    return KL_OK;
}

int kl_stash_mode(const kl_handle* h) { return h ? (h->stash ? 1 : 0) : -1; }

kl_status kl_set_tensor_core_attention(kl_handle* h, int on) {
    if (!h) return KL_ERR_INVALID_ARG;
    if (!on && h->stash) return KL_ERR_UNSUPPORTED_SHAPE;   // the stash-mode kernels have no CUDA-core attention loop
    if (on && !h->encode_tiled) return KL_ERR_CUDA;
    const uint32_t G = h->prm.G;
    if (!on && G != 1 && G != 2 && G != 4 && G != 8) return KL_ERR_UNSUPPORTED_SHAPE;   // no CUDA-core loop for this group size
    h->use_tc_attention = on ? 1 : 0;
    return KL_OK;
}

kl_status kl_set_batched_path(kl_handle* h, int on) {
    if (!h) return KL_ERR_INVALID_ARG;
    if (on && !h->bt_ok) return KL_ERR_UNSUPPORTED_SHAPE;
    h->use_bt = on ? 1 : 0;
    drop_batched_graph(h);
    return KL_OK;
}

kl_status kl_set_dependent_launch(kl_handle* h, int on) {
    if (!h) return KL_ERR_INVALID_ARG;
    h->use_pdl = on ? 1 : 0;
    drop_batched_graph(h);
    return KL_OK;
}

kl_status kl_debug_skip_signal_once(kl_handle* h, int stage) {
    if (!h || stage < -1 || stage > 4) return KL_ERR_INVALID_ARG;
    h->pending_skip_stage = stage;
    return KL_OK;
}

kl_status kl_debug_set_jitter(kl_handle* h, uint32_t seed, uint32_t max_ns) {
    if (!h || max_ns > 1000000u) return KL_ERR_INVALID_ARG;
    h->prm.jitter_seed = max_ns ? seed : 0u;
    h->prm.jitter_ns = max_ns;
    return KL_OK;
}

kl_status kl_debug_set_step(kl_handle* h, uint32_t step, uint32_t* wrap_at) {
    if (!h) return KL_ERR_INVALID_ARG;
    if (wrap_at) *wrap_at = step_wrap(h->prm.L);
    if (step == 0xffffffffu) return KL_OK;   // query only
    if (cudaMemcpy(h->prm.step_dev, &step, 4, cudaMemcpyHostToDevice) != cudaSuccess) return KL_ERR_CUDA;
    h->chain_tok = nullptr;   // the next greedy call starts a chain (embedding under the new step number)
    return KL_OK;
}

void kl_destroy(kl_handle* h) {
    if (!h) return;
    kl_profile_enable(h, 0);
    drop_batched_graph(h);
    if (h->cap_stream) cudaStreamDestroy(h->cap_stream);
    free(h->loaded);
    delete h;
}

}  // extern "C"
