// The decode step of a BATCH as ONE persistent kernel: kernel looping (Section 3.2 of the paper, rules (1)-(10))
// applied to the batched tensor-core path.  The ten calls per layer of the per-operator schedule (kl_batched.cuh;
// Section 2, schedule (i)) become phases of one cooperative launch whose outer loop runs layers [l0, l1) -- all L of
// them in the looped schedule (with the embedding in front and the classifier behind: one launch per step), one layer
// per launch in the per-layer schedule (Section 2, schedule (ii)).  Every phase is the device function the
// per-operator kernels are made of, so the three schedules give the same bits.
//
// What replaces a kernel boundary: a grid barrier -- one release/acquire counter per phase, zeroed by the host before
// the launch -- between the phase warps of the CTAs, and NOTHING for the weight stream: warp 0 of every CTA is the
// projections' TMA producer for the whole launch.  Weight addresses do not depend on activations, so it requests the
// tiles of the next projection (of the next layer) while the phase warps are still in the vector phases or at a
// barrier, as far ahead as the ring has stages; only the INPUT tiles of a projection wait for the barrier behind the
// phase that writes its operand (the producer polls that barrier's counter).  TMEM is allocated once per launch, the
// ring, the two accumulator buffers and the attention warps' slots keep their barrier phases from layer to layer.
//
// Warps (384 threads, one CTA per SM):
//   warp 0        lane 0: weight/operand producer of all projections of the launch
//   warp 1        lane 0: MMA issuer (the warp owns TMEM)
//   warps 2..5    accumulator epilogue (TMEM lane quarter = warp % 4)
//   warps 4..11   256 threads for the vector phases (finish, rotation + cache append, merge, embedding)
//   warps 1..11   the attention stream (BA_WARPS = 11 independent workers)
// Shared memory: the projection ring (BG_STAGES tile pairs) and the attention warps' slots share one region -- the
// producer does not start the O projection's tiles before this CTA's attention warps are done (an mbarrier) -- then the
// barriers and small tables.
#pragma once

namespace kl {

constexpr int BL_THREADS = 384;
constexpr int BL_PHASE_WARPS = 11;      // warps 1..11
constexpr int BL_PHASE_THREADS = BL_PHASE_WARPS * 32;
constexpr int BL_WORK_THREADS = 256;    // warps 4..11
constexpr size_t BL_REGION_BYTES = (size_t)BG_STAGES * BG_STAGE_BYTES > (size_t)BA_WARPS * BA_SLOTS * BA_SLOT_BYTES
                                       ? (size_t)BG_STAGES * BG_STAGE_BYTES : (size_t)BA_WARPS * BA_SLOTS * BA_SLOT_BYTES;
constexpr size_t BL_MISC_BYTES = 4096;
constexpr size_t BL_SMEM_BYTES = 1024 /* alignment slack */ + BL_REGION_BYTES + BL_MISC_BYTES;
constexpr uint32_t BL_BARRIERS_PER_LAYER = 10;

// Static description of one of the five projections (QKV, O, gate/up, down, classifier).
struct BlGemm {
    uint32_t R, K, S, stream, nkb, pieces, kp, kb_piece, rpc, xmap, normed;
};

struct BLoopParams {
    CUtensorMap map_w[5], map_wl[5], map_x[3], kv_map;
    BlGemm g[5];
    const int32_t* tokens;
    const int32_t* positions;
    const __nv_bfloat16 *embed, *g1, *g2, *gf, *bqkv;   // per-layer tensors: layer_stride elements apart
    uint64_t layer_stride;
    float* x;                 // [32][H] residual stream
    __nv_bfloat16* xop[3];    // operands [64][H], [64][QD], [64][F]
    float* ssq;               // [32][BV_MAX_CHUNKS]
    float* part;              // partial results of the projection in flight
    float* q;                 // [32][QD] rotated queries
    float* part_o;            // attention partial outputs
    float* part_ml;           // and their (max, sum) pairs
    float* logits;
    float* rope_cs;
    const double* inv_freq;
    __nv_bfloat16* kv;
    uint32_t H, QD, KVD, F, V, nq, nkv, G, hd, B, max_ctx;
    uint32_t l0, l1;          // layers of this launch
    uint32_t first, last;     // 1: the embedding runs in front of layer l0 / the classifier behind layer l1 - 1
    uint32_t NW;              // attention workers of the grid
    float eps;
    uint32_t* bar;            // grid-barrier counters of this launch, zero at its start
    int32_t* status;
    uint64_t wait_ns;
};

struct BlSmem {
    BgSmem bg;                // projection ring + its barriers (tiles at the start of the shared region)
    uint64_t* attn_full;      // [BA_WARPS][BA_SLOTS]
    uint64_t* attn_done;      // one arrival per attention warp and layer
    volatile int* step_ok;    // written by one thread at the start and behind every grid barrier: the status word is still clear
    float* red;               // [8] sums of squares of a finish item
    BaMergeSmem* merge;       // [8] one per merge group
};

__device__ __forceinline__ BlSmem bl_carve(uint8_t* raw_ptr) {
    BlSmem m;
    const uint32_t raw = smem_u32(raw_ptr);
    m.bg.tiles = (raw + 1023u) & ~1023u;
    uint8_t* misc = raw_ptr + (m.bg.tiles - raw) + BL_REGION_BYTES;
    m.bg.full = reinterpret_cast<uint64_t*>(misc);
    m.bg.empty = m.bg.full + BG_STAGES;
    m.bg.acc_full = m.bg.empty + BG_STAGES;
    m.bg.acc_empty = m.bg.acc_full + 2;
    m.attn_full = m.bg.acc_empty + 2;
    m.attn_done = m.attn_full + BA_WARPS * BA_SLOTS;
    m.bg.tmem_base_s = reinterpret_cast<uint32_t*>(m.attn_done + 1);
    m.bg.abort_flag = reinterpret_cast<volatile int*>(m.bg.tmem_base_s + 1);
    m.step_ok = m.bg.abort_flag + 1;
    m.red = reinterpret_cast<float*>(misc + 512);
    m.merge = reinterpret_cast<BaMergeSmem*>(misc + 1024);
    static_assert(sizeof(BaMergeSmem) * 8 + 1024 <= BL_MISC_BYTES, "merge scratch does not fit");
    static_assert((2 * BG_STAGES + 4 + BA_WARPS * BA_SLOTS + 1) * 8 + 12 <= 512, "barriers do not fit");
    return m;
}

// ---- grid barrier.  Counter `idx` counts the CTAs whose phase warps have finished the phase in front of it.
__device__ __forceinline__ uint32_t bl_ld_relaxed(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Polls with relaxed loads; the caller's fence behind a successful wait is the acquire.
__device__ __forceinline__ bool bl_counter_wait(const BLoopParams& p, uint32_t idx, volatile int* abort_flag) {
    const uint32_t* ctr = p.bar + idx;
    if (bl_ld_relaxed(ctr) >= gridDim.x) return true;
    if (*abort_flag) return false;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (bl_ld_relaxed(ctr) < gridDim.x) {
        if ((++it & 31u) == 0) {
            if (*abort_flag) return false;
            if (__ldcg(p.status) != 0) {   // another CTA gave up: so does this one
                *abort_flag = 1;
                return false;
            }
            if (globaltimer_ns() - t0 > p.wait_ns) {
                atomicCAS(p.status, 0, ERR_SYNC_TIMEOUT);
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void bl_phase_bar() { asm volatile("bar.sync 1, %0;" ::"n"(BL_PHASE_THREADS) : "memory"); }
// Called by all phase warps (ptid = thread index among them).  Returns, the same value to every thread of the CTA,
// whether the step is still good: no wait has given up and no kernel has flagged an error so far.  (One thread reads
// the status word; were every thread to read it, a word that changes in between would split the CTA.)
__device__ __forceinline__ bool bl_gsync(const BLoopParams& p, uint32_t idx, uint32_t ptid, volatile int* abort_flag,
                                         volatile int* step_ok) {
    bl_phase_bar();
    if (ptid == 0) {
        __threadfence();
        red_release_add(p.bar + idx, 1u);
        const bool passed = bl_counter_wait(p, idx, abort_flag);
        __threadfence();
        const bool good = passed && __ldcg(p.status) == 0;
        if (!good) *abort_flag = 1;   // every other wait of this CTA (the producer's among them) gives up at once
        *step_ok = good ? 1 : 0;
    }
    bl_phase_bar();
    return *step_ok != 0;
}

__device__ __forceinline__ BgView bl_view(const BLoopParams& p, int idx, uint32_t layer) {
    const BlGemm& g = p.g[idx];
    BgView v;
    v.out = idx == 4 ? p.logits : p.part;
    v.R = g.R; v.K = g.K; v.B = p.B; v.S = g.S; v.layer = idx == 4 ? 0u : layer;
    v.stream = g.stream; v.nkb = g.nkb; v.pieces = g.pieces; v.kp = g.kp; v.kb_piece = g.kb_piece; v.rpc = g.rpc;
    v.ssq = g.normed ? p.ssq : nullptr;
    v.ssq_n = (p.H + BV_CHUNK - 1) / BV_CHUNK;
    v.eps = p.eps;
    v.status = p.status;
    v.wait_ns = p.wait_ns;
    return v;
}
__device__ __forceinline__ BgPartials bl_partials(const BLoopParams& p, int idx) {
    const BlGemm& g = p.g[idx];
    BgPartials q;
    q.part = p.part;
    q.R = g.R; q.S = g.S; q.stream = g.stream; q.nkb = g.nkb;
    q.T = ((g.R + BG_TILE_M - 1) / BG_TILE_M) * g.nkb;
    q.P = gridDim.x;
    return q;
}

// ---- phases on the 256 vector threads (wtid = 0..255)
__device__ __forceinline__ void bl_finish_phase(const BLoopParams& p, const BgPartials& parts, const __nv_bfloat16* gain,
                                                int swiglu, uint32_t K, __nv_bfloat16* xop, uint32_t wtid, float* red) {
    const uint32_t nc = (K + BV_CHUNK - 1) / BV_CHUNK, n = p.B * nc;
    for (uint32_t i = blockIdx.x; i < n; i += gridDim.x) {
        b_finish_item<2>(parts, p.x, p.x, gain, swiglu, K, xop, p.ssq, i / nc, i % nc, wtid, red);
        if (!swiglu) group_bar<2, BL_WORK_THREADS>();   // the next item of this CTA reuses `red`
    }
}
// SwiGLU between the gate/up and the down projection: no reduction, so the feature pairs of all sequences form one flat
// list over the phase threads of the grid; every thread takes two pairs at a time and issues the loads of both before
// it computes (the partial sums sit in L2: one round trip per two pairs).
__device__ __forceinline__ void bl_swiglu_phase(const BLoopParams& p, const BgPartials& parts, uint32_t ptid) {
    const uint32_t half = p.F / 2u, n = p.B * half, nthreads = gridDim.x * (uint32_t)BL_PHASE_THREADS;
    for (uint32_t e = blockIdx.x * (uint32_t)BL_PHASE_THREADS + ptid; e < n; e += 2u * nthreads) {
        const uint32_t e1 = e + nthreads;
        float g0[4], g1[4] = {0.f, 0.f, 0.f, 0.f};
        bg_sum_partials<4>(parts, e / half, 4u * (e % half), g0);
        if (e1 < n) bg_sum_partials<4>(parts, e1 / half, 4u * (e1 % half), g1);
        b_swiglu_store(g0, p.xop[2], p.F, e / half, 2u * (e % half));
        if (e1 < n) b_swiglu_store(g1, p.xop[2], p.F, e1 / half, 2u * (e1 % half));
    }
}

__device__ __forceinline__ BAttnView bl_attn_params(const BLoopParams& p, uint32_t layer) {
    BAttnView a;
    a.kv = p.kv;
    a.positions = p.positions;
    a.cs = p.rope_cs;
    a.qkv = bl_partials(p, 0);
    a.bias = p.bqkv ? p.bqkv + (size_t)layer * p.layer_stride : nullptr;
    a.q = p.q;
    a.part_o = p.part_o;
    a.part_ml = p.part_ml;
    a.xop = p.xop[1];
    a.QD = p.QD; a.KVD = p.KVD; a.nq = p.nq; a.nkv = p.nkv; a.G = p.G; a.hd = p.hd; a.B = p.B; a.max_ctx = p.max_ctx;
    a.layer = layer;
    a.NW = p.NW;
    a.status = p.status;
    a.wait_ns = p.wait_ns;
    return a;
}
__device__ __forceinline__ void bl_merge_phase(const BLoopParams& p, const BAttnView& a, uint32_t wtid, BaMergeSmem* sm) {
    const uint32_t n = p.nq * p.B;
    if (p.hd == 128) {   // four groups of 64 threads
        const uint32_t grp = wtid >> 6, t = wtid & 63u;
        for (uint32_t i = blockIdx.x * 4u + grp; i < n; i += gridDim.x * 4u) {
            switch (grp) {
                case 0: b_merge_item<3, 64>(a, i % p.nq, i / p.nq, t, sm[0]); break;
                case 1: b_merge_item<4, 64>(a, i % p.nq, i / p.nq, t, sm[1]); break;
                case 2: b_merge_item<5, 64>(a, i % p.nq, i / p.nq, t, sm[2]); break;
                default: b_merge_item<6, 64>(a, i % p.nq, i / p.nq, t, sm[3]); break;
            }
        }
    } else {             // eight groups of 32 threads
        const uint32_t grp = wtid >> 5, t = wtid & 31u;
        for (uint32_t i = blockIdx.x * 8u + grp; i < n; i += gridDim.x * 8u) {
            switch (grp) {
                case 0: b_merge_item<3, 32>(a, i % p.nq, i / p.nq, t, sm[0]); break;
                case 1: b_merge_item<4, 32>(a, i % p.nq, i / p.nq, t, sm[1]); break;
                case 2: b_merge_item<5, 32>(a, i % p.nq, i / p.nq, t, sm[2]); break;
                case 3: b_merge_item<6, 32>(a, i % p.nq, i / p.nq, t, sm[3]); break;
                case 4: b_merge_item<7, 32>(a, i % p.nq, i / p.nq, t, sm[4]); break;
                case 5: b_merge_item<8, 32>(a, i % p.nq, i / p.nq, t, sm[5]); break;
                case 6: b_merge_item<9, 32>(a, i % p.nq, i / p.nq, t, sm[6]); break;
                default: b_merge_item<10, 32>(a, i % p.nq, i / p.nq, t, sm[7]); break;
            }
        }
    }
}

__global__ void __launch_bounds__(BL_THREADS, 1) kl_bloop_kernel(const __grid_constant__ BLoopParams p) {
    extern __shared__ uint8_t bl_smem_raw[];
    const BlSmem m = bl_carve(bl_smem_raw);
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = m.bg.abort_flag;
    if (tid == 0) {
        for (int i = 0; i < BA_WARPS * BA_SLOTS; ++i) mbar_init(smem_u32(&m.attn_full[i]), 1);
        mbar_init(smem_u32(m.attn_done), BA_WARPS);
        bg_init_barriers(m.bg);   // also the fences behind the initialisations
        // a launch that finds the status word set is a no-op (an earlier launch of the step flagged an error)
        *m.step_ok = *p.status == 0 ? 1 : 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(m.bg.tmem_base_s), BG_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *m.bg.tmem_base_s;
    const uint32_t nl = p.l1 - p.l0;
    const bool dead = *m.step_ok == 0;

    if (warp == 0) {
        // ---------------------------------------------------------------- producer of all projections of the launch
        if (lane == 0 && !dead) {
            BgPipe pipe = {0u, 0u, 0u};
            bool ok = true;
            auto produce = [&](int idx, uint32_t layer, uint32_t ready_bar) {
                const BgView v = bl_view(p, idx, layer);
                ok = bg_produce(v, &p.map_w[idx], &p.map_wl[idx], &p.map_x[p.g[idx].xmap], m.bg, pipe, [&]() {
                    // the operand is complete when every CTA has passed the barrier behind the phase that writes it
                    if (!bl_counter_wait(p, ready_bar, abort_flag)) return false;
                    __threadfence();
                    asm volatile("fence.proxy.async;" ::: "memory");   // written by generic stores, read by bulk copies
                    return __ldcg(p.status) == 0;
                });
            };
            for (uint32_t li = 0; li < nl && ok; ++li) {
                const uint32_t l = p.l0 + li, base = p.first + li * BL_BARRIERS_PER_LAYER;
                produce(0, l, base + 0);
                if (!ok) break;
                // the ring's memory is the attention warps' until they are done with this layer
                if (!bg_wait(smem_u32(m.attn_done), li & 1u, p.status, p.wait_ns, abort_flag)) {
                    ok = false;
                    break;
                }
                produce(1, l, base + 4);
                if (ok) produce(2, l, base + 6);
                if (ok) produce(3, l, base + 8);
            }
            if (ok && p.last) produce(4, 0u, p.first + nl * BL_BARRIERS_PER_LAYER);
            if (!ok) bg_drain(m.bg, pipe, p.wait_ns);
        }
    } else if (!dead) {
        // ---------------------------------------------------------------- phase warps
        const uint32_t ptid = tid - 32u;                      // 0..351
        const bool worker = warp >= 4u;
        const uint32_t wtid = tid - 128u;                     // 0..255 for the vector threads
        BgPipe mma_pipe = {0u, 0u, 0u}, epi_pipe = {0u, 0u, 0u};
        uint32_t attn_uses = 0;
        const uint32_t attn_ring = m.bg.tiles + (warp - 1u) * BA_SLOTS * BA_SLOT_BYTES;
        uint64_t* attn_full = m.attn_full + (warp - 1u) * BA_SLOTS;
        uint32_t bi = 0;
        bool live = true;
        auto gemm_phase = [&](int idx, uint32_t layer) {
            const BgView v = bl_view(p, idx, layer);
            if (warp == 1u) {
                if (lane == 0) bg_mma(v, m.bg, mma_pipe, tmem_base);
            } else if (warp <= 5u) {
                bg_epilogue(v, m.bg, epi_pipe, tmem_base, warp & 3u, lane);
            }
        };
        if (p.first) {
            if (worker)
                for (uint32_t b = blockIdx.x; b < p.B; b += gridDim.x)
                    b_embed_item<BL_WORK_THREADS>(p.tokens, p.positions, p.embed, p.x, p.H, p.V, p.max_ctx, p.inv_freq, p.rope_cs,
                                                  p.hd / 2, p.status, b, wtid);
            // every token and position of the batch has been checked: a bad one makes the step a no-op
            live = bl_gsync(p, bi++, ptid, abort_flag, m.step_ok);
        }
        for (uint32_t li = 0; li < nl && live; ++li) {
            const uint32_t l = p.l0 + li;
            const size_t lo = (size_t)l * p.layer_stride;
            // V1: x += down projection of the previous layer; operand = g1 * x; sums of squares
            if (worker) {
                BgPartials prev = bl_partials(p, 3);
                if (l == 0) prev.part = nullptr;
                bl_finish_phase(p, prev, p.g1 + lo, 0, p.H, p.xop[0], wtid, m.red);
            }
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            gemm_phase(0, l);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            // V2: rotation, cache append
            const BAttnView a = bl_attn_params(p, l);
            {   // one (sequence, head) per warp, all eleven phase warps
                const uint32_t nh = p.nq + 2u * p.nkv, n = p.B * nh;
                for (uint32_t i = blockIdx.x * (uint32_t)BL_PHASE_WARPS + (warp - 1u); i < n; i += gridDim.x * (uint32_t)BL_PHASE_WARPS)
                    b_rope_item<32>(a, i / nh, i % nh, lane);
            }
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            // A: the attention stream (the rows appended above are read by bulk copies)
            {
                asm volatile("fence.proxy.async;" ::: "memory");
                b_attn_dispatch(a, &p.kv_map, warp - 1u, lane, attn_ring, attn_full, abort_flag, attn_uses);
                __syncwarp();
                if (lane == 0) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the slots go back to the projection ring
                    mbar_arrive(smem_u32(m.attn_done));
                }
            }
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            // V3: merge of the segments -> operand of the O projection
            if (worker) bl_merge_phase(p, a, wtid, m.merge);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            gemm_phase(1, l);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            // V4: x += attention output projection; operand = g2 * x
            if (worker) bl_finish_phase(p, bl_partials(p, 1), p.g2 + lo, 0, p.H, p.xop[0], wtid, m.red);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            gemm_phase(2, l);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            // V5: operand = silu(gate) * up
            bl_swiglu_phase(p, bl_partials(p, 2), ptid);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) { live = false; break; }
            gemm_phase(3, l);
            if (!bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) live = false;
        }
        if (p.last && live) {
            // x += last down projection (kept for kl_read_hidden); operand = gf * x; logits = factor * W_lm . operand
            if (worker) bl_finish_phase(p, bl_partials(p, 3), p.gf, 0, p.H, p.xop[0], wtid, m.red);
            if (bl_gsync(p, bi++, ptid, abort_flag, m.step_ok)) gemm_phase(4, 0u);
        }
    }
    // ---- common exit: nobody may still be using TMEM when it is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BG_TMEM_COLS);
    }
}

}  // namespace kl
