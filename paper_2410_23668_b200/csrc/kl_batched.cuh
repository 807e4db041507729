// Decode step for a BATCH of sequences: every projection is a dense contraction [rows x K] x [K x batch] on the
// 5th-generation tensor cores (tcgen05, accumulators in TMEM), so the weights are streamed once per step for all
// sequences (the paper's Table 1: ~20 FLOP/B at batch 32 -- still far below the ridge, i.e. HBM-bound, which is why the
// tiling is chosen for streaming and balance, not for tensor throughput).
//
// One projection = kl_bgemm_kernel:  result[b][r] = sum_k W[r, k] * x[b, k], left as partial results.
//   * M = 128 weight rows per tile; the inputs enter as the N operand split into bf16 hi and lo halves that sit in
//     columns 0..31 and 32..63 of ONE N = 64 operand: a single MMA per 16 columns of K yields W.x_hi and W.x_lo side by
//     side and the epilogue adds them (fp32-accurate inputs on a bf16 tensor pipe).
//   * Schedule (see BgIter): the K blocks (64 columns) of all row tiles form one list and each of the 148 persistent
//     CTAs takes a contiguous, equally long range of it, so every CTA streams the same number of bytes whatever the
//     tile count; a tile cut by a range boundary is left as partial tiles, one per CTA that shares it.  Small
//     projections (fewer blocks than CTAs) and the classifier use whole (row tile, K split) items instead.  The
//     partial results are added, in a fixed order, by the kernel that consumes them (kl_b_finish_kernel /
//     kl_b_rope_kernel) -- no floating-point atomics, the result is reproducible.
//   * The RMSNorm factor is applied behind the contraction (W.(g*x) * rsqrt(mean x^2 + eps)): the operand holds
//     g * x, the epilogue scales column b by the factor of sequence b, so no kernel waits for a whole-vector reduction.
//   * Per 64 columns of K one ring stage holds a [128 x 64] weight tile (16 KB) and the [64 x 64] input tile (8 KB),
//     written by TMA with the 128-byte swizzle the MMA's shared-memory descriptors expect.  Row-major matrices are read
//     through a 3-D tensor (column, row, layer); matrices stored in chunk order for the batch-1 kernel (unit of rpc
//     rows x column piece) through a 5-D tensor (column, row in unit, piece, unit, layer) plus a 4-D one for the
//     shorter last piece.
//   * Roles (192 threads): warp 0 lane 0 issues the TMA loads, warp 1 owns TMEM and its lane 0 issues tcgen05.mma and
//     the commits, warps 2..5 read the accumulators (tcgen05.ld) and store.  Two accumulator buffers overlap the
//     epilogue of one segment with the MMAs of the next.  Every mbarrier wait is bounded.
//   * The kernels of a step are launched with programmatic stream serialisation: a projection requests the weight
//     tiles of its first ring round while its predecessor still runs (see griddep_wait).
//
// Between the projections small kernels, spread over (sequence, chunk) blocks, do the vector work (sum of the partial
// results, residual, gain and sums of squares for the RMSNorm, SwiGLU, RoPE, cache append) and write the next
// projection's bf16 operand.  Doing this work in the projection's epilogue instead (the CTA that completes a tile,
// found by a ticket, finishes it) was measured and is slower: fence, ticket, re-read and store form a latency chain
// of ~10 us per tile on four warps, more than a separate kernel over hundreds of blocks costs.  Doing it as the
// prologue of the consuming kernel (shares of the work, then a grid barrier) was measured too and is no faster than a
// small kernel that is already resident, through programmatic dependent launch, when its predecessor ends.
// Attention is one balanced stream of K|V chunks over a persistent grid (kl_b_attn_kernel) followed by a merge per
// (sequence, query head) that writes the operand of the O projection.
#pragma once

namespace kl {

constexpr int BG_THREADS = 192;
constexpr int BG_STAGES = 6;
constexpr int BG_TILE_M = 128;
constexpr int BG_TILE_N = 64;   // 32 sequences x (hi, lo)
constexpr int BG_TILE_K = 64;   // bf16 columns per stage = one 128-byte swizzle row
constexpr int BG_A_BYTES = BG_TILE_M * BG_TILE_K * 2;
constexpr int BG_B_BYTES = BG_TILE_N * BG_TILE_K * 2;
constexpr int BG_STAGE_BYTES = BG_A_BYTES + BG_B_BYTES;
constexpr int BG_TMEM_COLS = 128;   // two accumulator buffers of 64 fp32 columns
constexpr size_t BG_SMEM_BYTES = (size_t)BG_STAGES * BG_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int BG_MAX_BATCH = 32;

// One projection as the three roles see it (everything but the tensor maps).
struct BgView {
    float* out;            // tile schedule: [S][32][R] partial sums (S = 1: the result itself);
                           // stream schedule: [row tiles + CTAs][32][128] partial tiles, slot = tile + CTA
    uint32_t R, K, B, S, layer;
    uint32_t stream;       // 0: tile schedule, items (row tile, K split) dealt round-robin; 1: stream schedule, see BgIter
    uint32_t nkb;          // K blocks of 64 columns in all (a block may reach past the end of K or of a piece: TMA fills zeros)
    uint32_t pieces;       // 0: row-major weights; otherwise the number of column pieces of the chunk order
    uint32_t kp;           // columns per full piece
    uint32_t kb_piece;     // K blocks per full piece = ceil(kp / 64)
    uint32_t rpc;          // rows per unit of the chunk order
    // RMSNorm folded behind the contraction: when ssq is set the operand holds gain * x (not normalised) and the epilogue
    // multiplies column b by rsqrt(sum_c ssq[b][c] / K + eps); ssq[b][c] are the partial sums of squares of x[b]
    const float* ssq;
    uint32_t ssq_n;        // partial sums per sequence
    float eps;
    int32_t* status;
    uint64_t wait_ns;
};
struct BgemmParams : BgView {
    CUtensorMap map_w;     // weights: rank 3 (column, row, layer) or, for chunk-ordered matrices, rank 5
    CUtensorMap map_wl;    // chunk-ordered matrices: the last (shorter) column piece, rank 4 (column, row in unit, unit, layer)
    CUtensorMap map_x;     // inputs [64 rows, K] bf16: rows 0..31 hi halves, 32..63 lo halves
};

constexpr int BV_CHUNK = 512;        // elements per block of the vector kernels (256 threads x 2)
constexpr int BV_MAX_CHUNKS = 64;    // partial sums of squares per sequence: hidden <= 32768

// ---- PTX wrappers (tcgen05 / TMEM / higher-rank TMA)

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]; M, N and the operand types are in the instruction descriptor.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (row) i.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tma_tensor_3d_g2s(uint32_t dst, const void* tmap, int32_t c0, int32_t c1, int32_t c2, uint32_t bar,
                                                  uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ void tma_tensor_5d_g2s(uint32_t dst, const void* tmap, int32_t c0, int32_t c1, int32_t c2, int32_t c3,
                                                  int32_t c4, uint32_t bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar), "l"(pol)
        : "memory");
}

// Programmatic dependent launch: the kernels of a step are launched with programmatic stream serialisation, so a
// kernel may start while its predecessor still runs.  griddep_wait() returns when the predecessor has completed and
// its writes are visible -- everything a kernel reads from or writes to buffers shared with other kernels comes after
// it; before it a kernel only sets itself up and prefetches data no kernel of the step writes (weights, cache rows of
// earlier steps).  griddep_launch() lets the successor start its own set-up.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the 128-byte swizzle
// (what TMA writes with CU_TENSOR_MAP_SWIZZLE_128B; the tile starts on a 1024-byte boundary): start address / 16 in
// bits 0..13, leading byte offset (unused for this layout) 1 in bits 16..29, stride between groups of eight rows
// 1024 / 16 in bits 32..45, descriptor version 1 in bits 46..47, layout type 2 (128-byte swizzle) in bits 61..63.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::f16: fp32 accumulator (bits 4..5 = 1), bf16 A and B (bits 7..9 and 10..12 = 1),
// both K-major (bits 15, 16 = 0), N / 8 in bits 17..22, M / 16 in bits 24..28.
__device__ __forceinline__ uint32_t umma_idesc_bf16(uint32_t M, uint32_t N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// The work of one CTA as a list of segments (row tile t, K blocks [kb0, kb1), partial-result slot).
//   tile schedule:   items (t, split) dealt round-robin; slot = split.
//   stream schedule: the K blocks of all tiles form one list of T = tiles * nkb blocks; CTA c takes the contiguous range
//                    [c * T / P, (c + 1) * T / P) of it, so every CTA streams the same number of bytes (+- one block of
//                    24 KB) whatever the tile count.  A tile cut by a range boundary is finished by the consumer
//                    kernel, which adds up the partial tiles of the CTAs that share it (slot = tile + CTA is unique,
//                    because along the list either the tile or the CTA advances from one segment to the next).
struct BgSeg {
    uint32_t t, kb0, kb1, slot;
};
struct BgIter {
    uint32_t stream, nkb, S, nitems, item;   // tile schedule
    uint32_t g0, g1;                         // stream schedule: blocks of the list still to do
    __device__ __forceinline__ BgIter(const BgView& p, uint32_t ntiles)
        : stream(p.stream), nkb(p.nkb), S(p.S), nitems(ntiles * p.S), item(blockIdx.x) {
        const uint32_t T = ntiles * p.nkb;
        g0 = (uint32_t)(((uint64_t)blockIdx.x * T) / gridDim.x);
        g1 = (uint32_t)(((uint64_t)(blockIdx.x + 1) * T) / gridDim.x);
    }
    __device__ __forceinline__ bool next(BgSeg& sg) {
        if (stream) {
            if (g0 >= g1) return false;
            sg.t = g0 / nkb;
            sg.kb0 = g0 - sg.t * nkb;
            sg.kb1 = min(nkb, sg.kb0 + (g1 - g0));
            sg.slot = sg.t + blockIdx.x;
            g0 += sg.kb1 - sg.kb0;
            return true;
        }
        if (item >= nitems) return false;
        const uint32_t sp = item % S;
        sg.t = item / S;
        sg.kb0 = (uint32_t)(((uint64_t)sp * nkb) / S);
        sg.kb1 = (uint32_t)(((uint64_t)(sp + 1) * nkb) / S);
        sg.slot = sp;
        item += gridDim.x;
        return true;
    }
};

// CTAs [first, last] whose ranges of the stream schedule meet row tile t (T = tiles * nkb blocks over P CTAs, T >= P).
__device__ __forceinline__ void bg_stream_sharers(uint32_t t, uint32_t nkb, uint32_t T, uint32_t P, uint32_t& first, uint32_t& last) {
    first = (uint32_t)((((uint64_t)t * nkb + 1u) * P - 1u) / T);
    last = (uint32_t)((((uint64_t)(t + 1u) * nkb) * P - 1u) / T);
}

// Where the partial results of a projection lie, for the kernels that consume them.
struct BgPartials {
    const float* part;
    uint32_t R;        // rows of the projection
    uint32_t S;        // tile schedule: K splits
    uint32_t stream;   // 1: stream schedule
    uint32_t nkb, T, P;   // stream schedule: K blocks per tile, blocks in all, CTAs
};

// v[i] = sum of the partial results of rows row .. row + N - 1 (one row tile; row % N == 0) of sequence b, added in
// split order (tile schedule) or CTA order (stream schedule): the same sum on every run.
template <int N>
__device__ __forceinline__ void bg_sum_partials(const BgPartials& q, uint32_t b, uint32_t row, float (&v)[N]) {
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = 0.f;
    const float* src;
    size_t stride;
    uint32_t n;
    if (q.stream) {
        const uint32_t t = row / BG_TILE_M;
        uint32_t first, last;
        bg_stream_sharers(t, q.nkb, q.T, q.P, first, last);
        src = q.part + ((size_t)(t + first) * BG_MAX_BATCH + b) * BG_TILE_M + (row - t * BG_TILE_M);
        stride = (size_t)BG_MAX_BATCH * BG_TILE_M;
        n = last - first + 1u;
    } else {
        src = q.part + (size_t)b * q.R + row;
        stride = (size_t)BG_MAX_BATCH * q.R;
        n = q.S;
    }
    // the loads of up to four partial results are issued together (one L2 round trip, not one per addend); the
    // additions keep their order
    for (uint32_t s0 = 0; s0 < n; s0 += 4, src += 4 * stride) {
        float a[4][N];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (s0 + j < n) {
                const float* sp = src + (size_t)j * stride;
                if (N == 4) {
                    const float4 t = *reinterpret_cast<const float4*>(sp);
                    a[j][0] = t.x; a[j][1] = t.y; a[j][2 % N] = t.z; a[j][3 % N] = t.w;
                } else if (N == 2) {
                    const float2 t = *reinterpret_cast<const float2*>(sp);
                    a[j][0] = t.x; a[j][1 % N] = t.y;
                } else {
                    a[j][0] = *sp;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (s0 + j < n) {
#pragma unroll
                for (int i = 0; i < N; ++i) v[i] += a[j][i];
            }
    }
}

__device__ __forceinline__ bool bg_wait(uint32_t bar, uint32_t parity, int32_t* status, uint64_t wait_ns, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > wait_ns) {
                atomicCAS(status, 0, ERR_SYNC_TIMEOUT);
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}

// Shared memory of the projection pipeline: BG_STAGES tile pairs on 1024-byte boundaries (the swizzle pattern repeats
// every 1024 bytes), then the barriers.
struct BgSmem {
    uint32_t tiles;        // shared-memory address of stage 0
    uint64_t* full;        // [BG_STAGES] tile pair landed
    uint64_t* empty;       // [BG_STAGES] MMAs that read the stage are done
    uint64_t* acc_full;    // [2] accumulator buffer complete
    uint64_t* acc_empty;   // [2] epilogue has read the buffer
    uint32_t* tmem_base_s;
    volatile int* abort_flag;
};
__device__ __forceinline__ BgSmem bg_carve(uint8_t* raw_ptr) {
    BgSmem m;
    const uint32_t raw = smem_u32(raw_ptr);
    m.tiles = (raw + 1023u) & ~1023u;
    uint8_t* misc = raw_ptr + (m.tiles - raw) + (size_t)BG_STAGES * BG_STAGE_BYTES;
    m.full = reinterpret_cast<uint64_t*>(misc);
    m.empty = m.full + BG_STAGES;
    m.acc_full = m.empty + BG_STAGES;
    m.acc_empty = m.acc_full + 2;
    m.tmem_base_s = reinterpret_cast<uint32_t*>(m.acc_empty + 2);
    m.abort_flag = reinterpret_cast<volatile int*>(m.tmem_base_s + 1);
    return m;
}
__device__ __forceinline__ void bg_init_barriers(const BgSmem& m) {   // one thread
    for (int i = 0; i < BG_STAGES; ++i) {
        mbar_init(smem_u32(&m.full[i]), 1);
        mbar_init(smem_u32(&m.empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
        mbar_init(smem_u32(&m.acc_full[i]), 1);
        mbar_init(smem_u32(&m.acc_empty[i]), 4);   // one arrival per epilogue warp
    }
    *m.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Where each of the three roles stands in the pipeline.  One launch of kl_bgemm_kernel starts at zero; the looped
// kernel carries the state from projection to projection (the ring and the two accumulator buffers never drain).
struct BgPipe {
    uint32_t stage, use;   // producer / MMA issuer: ring stage of the next tile pair and how often the ring has wrapped
    uint32_t it;           // MMA issuer / epilogue: segments so far (accumulator buffer it & 1, its use it >> 1)
};

// Producer (one thread): TMA loads of the weight tile and the input tile of every (row tile, K block) of this CTA's
// segments.  Weight tiles never wait for anything but a free stage (nothing writes weights); the input tiles of a
// projection may only be requested once `ready()` has returned true -- the kernel or phase that writes the operand
// has completed and its writes are visible.  Until then up to BG_STAGES weight tiles are requested ahead and their
// input tiles follow afterwards.  Returns false when a wait gave up or `ready` refused (the step is a no-op).
template <class Ready>
__device__ __forceinline__ bool bg_produce(const BgView& p, const CUtensorMap* map_w, const CUtensorMap* map_wl,
                                           const CUtensorMap* map_x, const BgSmem& m, BgPipe& pipe, Ready&& ready) {
    const uint64_t pol = l2_policy_evict_first();
    // the input tiles are read again by every row tile: they should outlive the weights in L2
    uint64_t polx;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(polx));
    const uint32_t ntiles = (p.R + BG_TILE_M - 1) / BG_TILE_M;
    uint32_t npend = 0;
    uint32_t pend_stage[BG_STAGES], pend_col[BG_STAGES];
    bool waited = false, ok = true;
    auto flush = [&]() {   // the operand is there: request the input tiles of the stages that went ahead
        if (!waited) {
            ok = ready();
            waited = true;
        }
        // (also when the step has turned out to be a no-op: the armed barriers have to complete)
        for (uint32_t i = 0; i < npend; ++i)
                tma_tensor_2d_g2s(m.tiles + pend_stage[i] * BG_STAGE_BYTES + BG_A_BYTES, map_x, (int32_t)pend_col[i], 0,
                                  smem_u32(&m.full[pend_stage[i]]), polx);
        npend = 0;
    };
    BgIter iter(p, ntiles);
    BgSeg sg;
    while (ok && !*m.abort_flag && iter.next(sg)) {
        const uint32_t t = sg.t;
        for (uint32_t kb = sg.kb0; kb < sg.kb1 && ok; ++kb) {
            // a stage whose input tile is still pending can never come free: when every stage holds such a tile, the
            // operand has to be waited for
            if (!waited && npend == (uint32_t)BG_STAGES) flush();
            if (!ok) break;
            if (pipe.use > 0 && !bg_wait(smem_u32(&m.empty[pipe.stage]), (pipe.use - 1u) & 1u, p.status, p.wait_ns, m.abort_flag)) {
                ok = false;
                break;
            }
            const uint32_t bar = smem_u32(&m.full[pipe.stage]);
            const uint32_t dst = m.tiles + pipe.stage * BG_STAGE_BYTES;
            mbar_arrive_expect_tx(bar, (uint32_t)BG_STAGE_BYTES);
            uint32_t xcol = kb * BG_TILE_K;
            if (p.pieces == 0u) {
                tma_tensor_3d_g2s(dst, map_w, (int32_t)xcol, (int32_t)(t * BG_TILE_M), (int32_t)p.layer, bar, pol);
            } else {
                // a block that reaches past the end of its piece gets zeros there from TMA, so whatever the input
                // tile holds in those columns (the next piece's values) does not count
                const uint32_t j = kb / p.kb_piece, cin = (kb - j * p.kb_piece) * BG_TILE_K, unit0 = t * BG_TILE_M / p.rpc;
                xcol = j * p.kp + cin;
                if (j + 1u < p.pieces)
                    tma_tensor_5d_g2s(dst, map_w, (int32_t)cin, 0, (int32_t)j, (int32_t)unit0, (int32_t)p.layer, bar, pol);
                else
                    tma_tensor_4d_g2s(dst, map_wl, (int32_t)cin, 0, (int32_t)unit0, (int32_t)p.layer, bar, pol);
            }
            if (waited) {
                tma_tensor_2d_g2s(dst + BG_A_BYTES, map_x, (int32_t)xcol, 0, bar, polx);
            } else {
                pend_stage[npend] = pipe.stage;
                pend_col[npend] = xcol;
                ++npend;
            }
            if (++pipe.stage == BG_STAGES) {
                pipe.stage = 0;
                ++pipe.use;
            }
        }
    }
    if (!waited || npend) flush();
    return ok && !*m.abort_flag;
}

// After an abandoned run no copy may still be writing this CTA's shared memory when it exits: wait (bounded) for the
// last copy armed on every stage.
__device__ __forceinline__ void bg_drain(const BgSmem& m, const BgPipe& pipe, uint64_t wait_ns) {
    const uint64_t t0 = globaltimer_ns();
    for (uint32_t sidx = 0; sidx < (uint32_t)BG_STAGES; ++sidx) {
        const uint32_t cnt = pipe.use + (sidx < pipe.stage ? 1u : 0u);
        if (cnt == 0) continue;
        while (!mbar_try_wait(smem_u32(&m.full[sidx]), (cnt - 1u) & 1u))
            if (globaltimer_ns() - t0 > wait_ns) break;
    }
}

// MMA issuer (one thread of the warp that owns TMEM).
__device__ __forceinline__ void bg_mma(const BgView& p, const BgSmem& m, BgPipe& pipe, uint32_t tmem_base) {
    const uint32_t idesc = umma_idesc_bf16(BG_TILE_M, BG_TILE_N);
    const uint32_t ntiles = (p.R + BG_TILE_M - 1) / BG_TILE_M;
    BgIter iter(p, ntiles);
    BgSeg sg;
    for (; !*m.abort_flag && iter.next(sg); ++pipe.it) {
        const uint32_t kb0 = sg.kb0, kb1 = sg.kb1;
        const uint32_t buf = pipe.it & 1u, buse = pipe.it >> 1;
        if (buse > 0 && !bg_wait(smem_u32(&m.acc_empty[buf]), (buse - 1u) & 1u, p.status, p.wait_ns, m.abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BG_TILE_N;
        for (uint32_t kb = kb0; kb < kb1; ++kb) {
            if (!bg_wait(smem_u32(&m.full[pipe.stage]), pipe.use & 1u, p.status, p.wait_ns, m.abort_flag)) break;
            tc_fence_after();
            const uint32_t a_addr = m.tiles + pipe.stage * BG_STAGE_BYTES;
            const uint64_t a_desc = umma_desc_sw128(a_addr), b_desc = umma_desc_sw128(a_addr + BG_A_BYTES);
#pragma unroll
            for (uint32_t k = 0; k < BG_TILE_K / 16; ++k)   // 16 bf16 = 32 bytes further along the swizzled row
                umma_f16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb != kb0 || k != 0u) ? 1u : 0u);
            umma_commit(smem_u32(&m.empty[pipe.stage]));   // the stage may be refilled when these MMAs are done
            if (++pipe.stage == BG_STAGES) {
                pipe.stage = 0;
                ++pipe.use;
            }
        }
        umma_commit(smem_u32(&m.acc_full[buf]));
    }
}

// Epilogue warp (one of four): reads TMEM lanes 32 * quarter .. + 31 = rows of the tile, adds the hi and lo halves,
// applies the RMSNorm factor and stores the partial tile.
__device__ __forceinline__ void bg_epilogue(const BgView& p, const BgSmem& m, BgPipe& pipe, uint32_t tmem_base,
                                            uint32_t quarter, uint32_t lane) {
    float inv = 1.0f;   // lane b: the RMSNorm factor of sequence b
    if (p.ssq != nullptr && lane < p.B) {
        float ss = 0.f;
        for (uint32_t c = 0; c < p.ssq_n; ++c) ss += p.ssq[lane * BV_MAX_CHUNKS + c];
        inv = rsqrtf(ss / (float)p.K + p.eps);
    }
    const uint32_t ntiles = (p.R + BG_TILE_M - 1) / BG_TILE_M;
    BgIter iter(p, ntiles);
    BgSeg sg;
    for (; iter.next(sg); ++pipe.it) {
        const uint32_t t = sg.t;
        const uint32_t buf = pipe.it & 1u, buse = pipe.it >> 1;
        if (!bg_wait(smem_u32(&m.acc_full[buf]), buse & 1u, p.status, p.wait_ns, m.abort_flag)) break;
        tc_fence_after();
        uint32_t hi[32], lo[32];
        const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + buf * BG_TILE_N;
        tmem_ld32(taddr, hi);
        tmem_ld32(taddr + 32u, lo);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&m.acc_empty[buf]));
        const uint32_t row = t * BG_TILE_M + quarter * 32u + lane;
        // tile schedule: [slot][b][R rows]; stream schedule: [slot][b][128 rows of the tile]
        float* dst = p.stream ? p.out + (size_t)sg.slot * BG_MAX_BATCH * BG_TILE_M + quarter * 32u + lane
                              : p.out + (size_t)sg.slot * BG_MAX_BATCH * p.R + row;
        const size_t bstride = p.stream ? (size_t)BG_TILE_M : (size_t)p.R;
#pragma unroll
        for (uint32_t b = 0; b < 32; ++b) {
            const float sc = __shfl_sync(0xffffffffu, inv, b);   // all lanes take part, also those past the last row
            if (row < p.R && b < p.B) dst[(size_t)b * bstride] = (__uint_as_float(hi[b]) + __uint_as_float(lo[b])) * sc;
        }
    }
}

__global__ void __launch_bounds__(BG_THREADS, 1) kl_bgemm_kernel(const __grid_constant__ BgemmParams p) {
    extern __shared__ uint8_t bg_smem_raw[];
    const BgSmem m = bg_carve(bg_smem_raw);
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) bg_init_barriers(m);
    if (warp == 1) {
        tmem_alloc(smem_u32(m.tmem_base_s), BG_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *m.tmem_base_s;

    griddep_launch();
    bool skip = false;
    if (!(warp == 0 && lane == 0)) {
        griddep_wait();
        skip = *p.status != 0;   // an earlier kernel of this step flagged an error: the step is a no-op
    }
    BgPipe pipe = {0u, 0u, 0u};
    if (warp == 0 && lane == 0) {
        // The weight tiles of the first ring round are requested before the predecessor kernel has finished; their
        // input tiles follow once it has.
        const bool ok = bg_produce(p, &p.map_w, &p.map_wl, &p.map_x, m, pipe, [&]() {
            griddep_wait();
            return *p.status == 0;
        });
        if (!ok) bg_drain(m, pipe, p.wait_ns);
    } else if (!skip && warp == 1 && lane == 0) {
        bg_mma(p, m, pipe, tmem_base);
    } else if (!skip && warp >= 2) {
        bg_epilogue(p, m, pipe, tmem_base, warp & 3u, lane);
    }
    // ---- common exit: nobody may still be using TMEM when it is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BG_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------ vector kernels

// Row b of the N operand of a projection: xop[b][k] = hi half, xop[32 + b][k] = lo half (bf16) of the fp32 value.
// Every projection input width has an operand buffer of its own; rows of sequences beyond the batch keep whatever
// finite values they last held (the MMA columns they feed are never stored).
__device__ __forceinline__ void put_operand2(__nv_bfloat16* xop, uint32_t K, uint32_t b, uint32_t k, float v0, float v1) {
    const uint32_t hi = pack_bf16(v0, v1);
    const uint32_t lo = pack_bf16(v0 - bf_lo(hi), v1 - bf_hi(hi));
    *reinterpret_cast<uint32_t*>(xop + (size_t)b * K + k) = hi;
    *reinterpret_cast<uint32_t*>(xop + (size_t)(32 + b) * K + k) = lo;
}

// SwiGLU of two neighbouring features from their (gate, up) sums, written as the next projection's operand.
__device__ __forceinline__ void b_swiglu_store(const float (&gu)[4], __nv_bfloat16* xop, uint32_t K, uint32_t b, uint32_t k) {
    const float v0 = gu[0] / (1.0f + __expf(-gu[0])) * gu[1];
    const float v1 = gu[2] / (1.0f + __expf(-gu[2])) * gu[3];
    put_operand2(xop, K, b, k, v0, v1);
}

// Barrier among the NT threads that work on one item together: the whole block of a vector kernel (barrier 0), or a
// group of warps of the looped kernel (a named barrier of its own).
template <int BAR, int NT>
__device__ __forceinline__ void group_bar() {
    asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// Vector work between two projections, one item = (sequence b, chunk c of BV_CHUNK elements), 256 threads x 2 elements.
//   swiglu = 0:  v[k] = res[b][k] + sum_s part[s][b][k];  xout[b][k] = v[k];  operand = gain[k] * v[k] (the RMSNorm
//                factor is applied behind the next contraction);  ssq[b][chunk] = sum of v[k]^2 over the chunk.
//   swiglu = 1:  v[f] = silu(sum_s part[s][b][2f]) * (sum_s part[s][b][2f+1]);  operand = v.
// The sums over the splits run in split order and the sum of squares in a fixed tree: reproducible.
// red: 8 floats of shared memory owned by the group.
template <int BAR>
__device__ __forceinline__ void b_finish_item(const BgPartials& part, const float* res, float* xout, const __nv_bfloat16* gain,
                                              int swiglu, uint32_t K, __nv_bfloat16* xop, float* ssq, uint32_t b, uint32_t c,
                                              uint32_t tid, float* red) {
    const uint32_t k = c * BV_CHUNK + 2 * tid;
    float v0 = 0.f, v1 = 0.f;
    if (k < K) {   // K is even
        if (swiglu) {
            float gu[4];   // gate f, up f, gate f + 1, up f + 1
            bg_sum_partials<4>(part, b, 2 * k, gu);
            b_swiglu_store(gu, xop, K, b, k);
        } else {
            const float2 r = *reinterpret_cast<const float2*>(res + (size_t)b * K + k);
            float a[2];
            if (part.part != nullptr) bg_sum_partials<2>(part, b, k, a);
            else a[0] = a[1] = 0.f;
            v0 = r.x + a[0];
            v1 = r.y + a[1];
            *reinterpret_cast<float2*>(xout + (size_t)b * K + k) = make_float2(v0, v1);
            const uint32_t gg = *reinterpret_cast<const uint32_t*>(gain + k);
            put_operand2(xop, K, b, k, v0 * bf_lo(gg), v1 * bf_hi(gg));
        }
    }
    if (swiglu) return;
    float ss = v0 * v0 + v1 * v1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    group_bar<BAR, 256>();
    if (tid == 0) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        ssq[b * BV_MAX_CHUNKS + c] = tot;
    }
}

// grid (batch, ceil(K / BV_CHUNK)), 256 threads
__global__ void __launch_bounds__(256) kl_b_finish_kernel(const BgPartials part, const float* res, float* xout,
                                                          const __nv_bfloat16* gain, int swiglu, uint32_t K, __nv_bfloat16* xop,
                                                          float* ssq, const int32_t* status) {
    __shared__ float red[8];
    griddep_launch();
    griddep_wait();
    if (*status != 0) return;
    b_finish_item<0>(part, res, xout, gain, swiglu, K, xop, ssq, blockIdx.x, blockIdx.y, threadIdx.x, red);
}

// Token embedding of every sequence of the batch, the check of the whole batch, and the step's rotary table:
// x[b] = E[token_b]; cs[b][i] = (cos, sin)(position_b * inv_freq[i]).  Grid (batch), 256 threads.
template <int NT>
__device__ __forceinline__ void b_embed_item(const int32_t* tokens, const int32_t* positions, const __nv_bfloat16* embed, float* x,
                                             uint32_t H, uint32_t V, uint32_t max_ctx, const double* inv_freq, float* cs,
                                             uint32_t half, int32_t* status, uint32_t b, uint32_t tid) {
    int32_t tok = tokens[b];
    const int32_t pos = positions[b];
    if (tid == 0 && (tok < 0 || tok >= (int32_t)V || pos < 0 || pos >= (int32_t)max_ctx)) atomicCAS(status, 0, ERR_OUT_OF_RANGE);
    if (tok < 0 || tok >= (int32_t)V) tok = 0;
    for (uint32_t i = tid; i < half; i += NT) {
        double sn, c;
        sincos((double)pos * inv_freq[i], &sn, &c);
        cs[(size_t)b * 2 * half + 2 * i] = (float)c;
        cs[(size_t)b * 2 * half + 2 * i + 1] = (float)sn;
    }
    const __nv_bfloat16* row = embed + (size_t)tok * H;
    for (uint32_t i = tid; i < H; i += NT) x[(size_t)b * H + i] = __bfloat162float(row[i]);
}

__global__ void __launch_bounds__(256) kl_b_embed_kernel(const int32_t* tokens, const int32_t* positions, const __nv_bfloat16* embed,
                                                         float* x, uint32_t H, uint32_t V, uint32_t max_ctx, const double* inv_freq,
                                                         float* cs, uint32_t half, int32_t* status) {
    griddep_launch();
    griddep_wait();
    b_embed_item<256>(tokens, positions, embed, x, H, V, max_ctx, inv_freq, cs, half, status, blockIdx.x, threadIdx.x);
}

struct BAttnView {
    __nv_bfloat16* kv;
    const int32_t* positions;
    const float* cs;          // [32][hd / 2][2] (cos, sin) of the step's positions
    BgPartials qkv;           // partial results of the QKV projection
    const __nv_bfloat16* bias;   // biases of this layer's q, k, v projections [QD + 2 KVD], or null
    float* q;                 // [32][QD] rotated, pre-scaled queries
    float* part_o;            // [B * nkv + NW][G][hd] partial results, slot = pair + warp
    float* part_ml;           // [B * nkv + NW][G][2]
    __nv_bfloat16* xop;       // operand of the O projection [64][QD]
    uint32_t QD, KVD, nq, nkv, G, hd, B, max_ctx, layer, NW;   // NW: warps of the attention grid
    int32_t* status;
    uint64_t wait_ns;
};
struct BAttnParams : BAttnView {
    CUtensorMap kv_map;       // the whole KV cache as a 4-D tensor: 64 columns, rows, column halves, K | V (one copy per chunk)
};

// RoPE and cache append; grid (batch, n_q_heads + 2 * n_kv_heads), one head of one sequence per block of 128
// threads: sums the splits of the QKV projection, rotates a q head (and scales it by log2(e) / sqrt(hd) for the base-2
// softmax) or a k head at the sequence's position, rounds k and v to bf16 and writes them into row `position` of the
// sequence's cache slabs.  The attention kernel that follows reads that row from the cache like any other.
template <int NT>   // threads that share the item
__device__ __forceinline__ void b_rope_item(const BAttnView& p, uint32_t b, uint32_t head, uint32_t tid) {
    const uint32_t hd = p.hd, half = hd >> 1;
    const int32_t pos = p.positions[b];
    const float* cs = p.cs + (size_t)b * hd;
    auto val = [&](uint32_t r) {   // row r of [q | k | v]: sum of the partial results, plus the projection's bias if any
        float v[1];
        bg_sum_partials<1>(p.qkv, b, r, v);
        return p.bias ? v[0] + __bfloat162float(p.bias[r]) : v[0];
    };
    const size_t slab = (size_t)p.max_ctx * hd;
    if (head < p.nq) {
        const float qscale = 1.4426950408889634f * rsqrtf((float)hd);
        for (uint32_t i = tid; i < half; i += NT) {
            const float a = val(head * hd + i), bb = val(head * hd + i + half), c = cs[2 * i], sn = cs[2 * i + 1];
            p.q[(size_t)b * p.QD + head * hd + i] = (a * c - bb * sn) * qscale;
            p.q[(size_t)b * p.QD + head * hd + i + half] = (bb * c + a * sn) * qscale;
        }
    } else if (head < p.nq + p.nkv) {
        const uint32_t g = head - p.nq;
        __nv_bfloat16* row = p.kv + ((((size_t)p.layer * 2 + 0) * p.B + b) * p.nkv + g) * slab + (size_t)pos * hd;
        for (uint32_t i = tid; i < half; i += NT) {
            const float a = val(p.QD + g * hd + i), bb = val(p.QD + g * hd + i + half), c = cs[2 * i], sn = cs[2 * i + 1];
            row[i] = __float2bfloat16_rn(a * c - bb * sn);
            row[i + half] = __float2bfloat16_rn(bb * c + a * sn);
        }
    } else {
        const uint32_t g = head - p.nq - p.nkv;
        __nv_bfloat16* row = p.kv + ((((size_t)p.layer * 2 + 1) * p.B + b) * p.nkv + g) * slab + (size_t)pos * hd;
        for (uint32_t d = tid; d < hd; d += NT) row[d] = __float2bfloat16_rn(val(p.QD + p.KVD + g * hd + d));
    }
}

__global__ void __launch_bounds__(128) kl_b_rope_kernel(const BAttnParams p) {
    griddep_launch();
    griddep_wait();
    if (*p.status != 0) return;
    b_rope_item<128>(p, blockIdx.x, blockIdx.y, threadIdx.x);
}

constexpr int BA_WARPS = 11;     // independent warps per CTA; one persistent CTA per SM (the looped kernel's twelfth warp streams weights)
constexpr int BA_THREADS = BA_WARPS * 32;
constexpr int BA_SLOTS = 2;      // ring slots per warp
constexpr int BA_SLOT_BYTES = 8192;   // K rows | V rows of 16 (head size 128) or 32 (head size 64) cached positions

// Chunks of cached positions a sequence at position `pos` holds after this step's append (pb positions per chunk).
__device__ __forceinline__ uint32_t ba_chunks(int32_t pos, uint32_t pb) { return ((uint32_t)pos + 1u + pb - 1u) / pb; }

// First chunk of warp w when W chunks are dealt in contiguous, equally long ranges to NW warps.
__device__ __forceinline__ uint32_t ba_range_lo(uint32_t w, uint32_t W, uint32_t NW) { return (uint32_t)(((uint64_t)w * W) / NW); }

// Warps that share the W chunks of a step: all NW of the grid when there is enough to stream, fewer for a small batch or
// short contexts -- at least BA_MIN_CHUNKS chunks per working warp, so that a (sequence, kv head) pair is not cut into
// more segments than the merge can add up cheaply.  Every working warp gets at least one chunk.
constexpr uint32_t BA_MIN_CHUNKS = 8;
__device__ __forceinline__ uint32_t ba_workers(uint32_t W, uint32_t NW) { return max(1u, min(NW, W / BA_MIN_CHUNKS)); }

// Walks the chunk list of the step: (sequence b, kv head g, chunk c of the sequence's nch chunks), in that order.
struct BaCursor {
    uint32_t b, g, c, nch;
};

// Attention of a batch as ONE balanced stream.  The chunks (16 or 32 cached positions of one kv head of one sequence:
// an 8 KB K|V tile pair) of all (sequence, kv head) pairs form one list; every warp of the persistent grid takes a
// contiguous range of W / NW chunks of it, streams them through a two-slot TMA ring of its own (loads run two chunks
// ahead, across pair boundaries) and runs the mma.sync tiles of kl_attention_tc.cuh on them.  Whenever its range
// leaves a pair the warp writes its flash-decoding partial result for that pair (O^T unnormalised, running maximum,
// sum) to slot (pair + warp) -- unique, because along the list either the pair or the warp advances from one segment
// to the next.  kl_b_attn_merge_kernel combines the segments of every pair.  No warp waits for another one, every
// warp streams the same number of bytes (+- one chunk), and a sequence's length only decides how many warps share it.
// `warp` = index of the calling warp among the BA_WARPS workers of its CTA; `ring` = shared-memory address of its
// BA_SLOTS slots (1024-byte aligned); `full` = its BA_SLOTS barriers (initialised by the caller); `uses` = chunks this
// warp has taken through its slots so far (the barrier phases go on from there: 0 in a kernel of its own, carried
// from layer to layer in the looped kernel).
template <int HD, bool PACK>
__device__ __forceinline__ void b_attn_stream(const BAttnView& p, const CUtensorMap* kv_map, uint32_t warp, uint32_t lane, uint32_t ring,
                                              uint64_t* full, volatile int* abort_flag, uint32_t& uses) {
    const uint32_t G = p.G;
    constexpr uint32_t pb = BA_SLOT_BYTES / (4u * HD);
    constexpr uint32_t box_bytes = pb * 128u;
    // lane b keeps the chunk count of sequence b; W = chunks of the whole step
    const uint32_t my_nch = lane < p.B ? ba_chunks(p.positions[lane], pb) : 0u;
    uint32_t W = my_nch;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) W += __shfl_xor_sync(0xffffffffu, W, o);
    W *= p.nkv;
    // worker w = warp (w / CTAs) of CTA (w % CTAs): when fewer warps than the grid has are at work, they spread over all SMs
    const uint32_t NW = ba_workers(W, p.NW), gw = warp * gridDim.x + blockIdx.x;
    if (gw >= NW) return;
    const uint32_t lo = ba_range_lo(gw, W, NW), hi = ba_range_lo(gw + 1, W, NW);

    // cursor at chunk `lo`
    BaCursor cur = {0u, 0u, 0u, __shfl_sync(0xffffffffu, my_nch, 0)};
    {
        uint32_t skip = lo;
        while (skip >= cur.nch * p.nkv) {   // whole sequences before the range (sequences have at least one chunk)
            skip -= cur.nch * p.nkv;
            ++cur.b;
            cur.nch = __shfl_sync(0xffffffffu, my_nch, cur.b & 31u);
        }
        cur.g = skip / cur.nch;
        cur.c = skip % cur.nch;
    }
    auto advance = [&](BaCursor& x) {   // warp-uniform
        if (++x.c == x.nch) {
            x.c = 0;
            if (++x.g == p.nkv) {
                x.g = 0;
                ++x.b;
                x.nch = __shfl_sync(0xffffffffu, my_nch, x.b & 31u);
            }
        }
    };
    const uint32_t vdelta = p.B * p.nkv * p.max_ctx;
    const uint64_t pol = l2_policy_evict_first();
    const uint32_t use0 = uses;   // chunk k of the range is this warp's chunk number use0 + k - lo
    auto issue = [&](const BaCursor& x, uint32_t slot) {   // lane 0: the chunk under cursor x into this warp's slot
        const uint32_t n = (uint32_t)p.positions[x.b] + 1u;
        const AttnWindow w = attn_window(0u, n, pb, x.c);
        const uint32_t row0 = p.layer * 2u * vdelta + (x.b * p.nkv + x.g) * p.max_ctx + w.w0;
        const uint32_t bar = smem_u32(&full[slot]);
        const uint32_t dst = ring + slot * BA_SLOT_BYTES;
        mbar_arrive_expect_tx(bar, (uint32_t)BA_SLOT_BYTES);
        // one copy: the K and the V rows of the chunk, every 64-column half a box of its own (the outer dimensions of the map)
        tma_tensor_4d_g2s(dst, kv_map, 0, (int32_t)row0, 0, 0, bar, pol);
    };

    // the first chunks of the range go out before anything else
    BaCursor nxt = cur;   // cursor of the next chunk to request
    uint32_t issued = 0;
    for (; issued < (uint32_t)BA_SLOTS && lo + issued < hi; ++issued) {
        if (lane == 0) issue(nxt, (use0 + issued) % BA_SLOTS);
        advance(nxt);
    }

    constexpr int NKB = HD / 16, NMT = HD / 16;
    const uint32_t gq = lane >> 2, t = lane & 3u;
    AttnTcState<HD> st;
    auto begin_pair = [&](const BaCursor& x) {   // Q fragments of the pair's heads, empty accumulators
        const float* q = p.q + (size_t)x.b * p.QD + (size_t)x.g * G * HD;
#pragma unroll
        for (int kb = 0; kb < NKB; ++kb) {
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const uint32_t k = kb * 16 + hf * 8 + 2 * t;
                const uint32_t head = PACK ? (gq & 3u) : gq;   // PACK: column gq = hi (gq < 4) or lo half of head gq % 4
                float2 xx = make_float2(0.f, 0.f);
                if (head < G) xx = *reinterpret_cast<const float2*>(q + head * HD + k);
                const uint32_t qhi = pack_bf16(xx.x, xx.y);
                const uint32_t qlo = pack_bf16(xx.x - bf_lo(qhi), xx.y - bf_hi(qhi));
                st.qh[kb][hf] = (PACK && gq >= 4u) ? qlo : qhi;
                st.ql[kb][hf] = qlo;
            }
        }
#pragma unroll
        for (int nn = 0; nn < NMT; ++nn) st.o[nn][0] = st.o[nn][1] = st.o[nn][2] = st.o[nn][3] = 0.f;
        st.m[0] = st.m[1] = -INFINITY;
        st.l[0] = st.l[1] = 0.f;
    };
    auto end_pair = [&](const BaCursor& x) {   // this warp's partial result of the pair to slot (pair + warp)
        float l0 = st.l[0], l1 = st.l[1];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {   // the lanes that share the heads (same lane % 4) hold parts of the row sums
            l0 += __shfl_xor_sync(0xffffffffu, l0, o);
            l1 += __shfl_xor_sync(0xffffffffu, l1, o);
        }
        if (PACK) {   // columns 0..3 hold the hi parts of O^T, columns 4..7 the lo parts: lanes t and t ^ 2 of a quad
#pragma unroll
            for (int nn = 0; nn < NMT; ++nn)
#pragma unroll
                for (int j = 0; j < 4; ++j) st.o[nn][j] += __shfl_xor_sync(0xffffffffu, st.o[nn][j], 2);
        }
        const size_t slot = (size_t)(x.b * p.nkv + x.g) + gw;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const uint32_t h = 2 * t + hh;
            if (h < G && (!PACK || t < 2u)) {
                float* dst = p.part_o + (slot * G + h) * HD;
#pragma unroll
                for (int nn = 0; nn < NMT; ++nn) {
                    dst[nn * 16 + gq] = st.o[nn][hh];
                    dst[nn * 16 + gq + 8] = st.o[nn][2 + hh];
                }
                if (gq == 0) *reinterpret_cast<float2*>(p.part_ml + (slot * G + h) * 2) = make_float2(st.m[hh], hh ? l1 : l0);
            }
        }
    };

    begin_pair(cur);
    uint32_t k = lo;
    for (; k < hi; ++k) {
        const uint32_t slot = (use0 + k - lo) % BA_SLOTS, phase = ((use0 + k - lo) / BA_SLOTS) & 1u;
        if (!bg_wait(smem_u32(&full[slot]), phase, p.status, p.wait_ns, abort_flag)) break;
        const uint32_t kbase = ring + slot * BA_SLOT_BYTES;
        const AttnWindow w = attn_window(0u, (uint32_t)p.positions[cur.b] + 1u, pb, cur.c);
#pragma unroll
        for (uint32_t r0 = 0; r0 < pb; r0 += 16)
            if (r0 + 16 > w.lo && r0 < w.hi) attn_tc_tile<HD, PACK>(st, kbase, kbase + BA_SLOT_BYTES / 2, box_bytes, r0, w.lo, w.hi, lane);
        __syncwarp();
        if (lo + issued < hi) {   // refill the slot just read
            if (lane == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the slot was read through the generic proxy
                issue(nxt, slot);
            }
            advance(nxt);
            ++issued;
        }
        const BaCursor done = cur;
        advance(cur);
        if (k + 1 == hi || cur.c == 0) {   // the pair ends here for this warp
            end_pair(done);
            if (k + 1 < hi) begin_pair(cur);
        }
    }
    // after a time-out copies may still be in flight: wait (bounded) for every chunk requested but not consumed
    if (k < hi && lane == 0) {
        const uint64_t t0 = globaltimer_ns();
        for (uint32_t c = use0 + k - lo; c < use0 + issued; ++c)
            while (!mbar_try_wait(smem_u32(&full[c % BA_SLOTS]), (c / BA_SLOTS) & 1u))
                if (globaltimer_ns() - t0 > p.wait_ns) break;
    }
    uses = use0 + issued;
}

// Picks the instantiation for the head size and the group size.
// kv_map: the cache's tensor map, in the kernel's parameter space.
__device__ __forceinline__ void b_attn_dispatch(const BAttnView& p, const CUtensorMap* kv_map, uint32_t warp, uint32_t lane,
                                                uint32_t ring, uint64_t* full, volatile int* abort_flag, uint32_t& uses) {
    if (p.hd == 128) {
        if (p.G <= 4) b_attn_stream<128, true>(p, kv_map, warp, lane, ring, full, abort_flag, uses);
        else b_attn_stream<128, false>(p, kv_map, warp, lane, ring, full, abort_flag, uses);
    } else {
        if (p.G <= 4) b_attn_stream<64, true>(p, kv_map, warp, lane, ring, full, abort_flag, uses);
        else b_attn_stream<64, false>(p, kv_map, warp, lane, ring, full, abort_flag, uses);
    }
}

__global__ void __launch_bounds__(BA_THREADS, 1) kl_b_attn_kernel(const __grid_constant__ BAttnParams p) {
    extern __shared__ uint8_t ba_smem_raw[];
    griddep_launch();
    griddep_wait();
    if (*p.status != 0) return;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t raw = smem_u32(ba_smem_raw);
    const uint32_t ring = ((raw + 1023u) & ~1023u) + warp * BA_SLOTS * BA_SLOT_BYTES;   // this warp's slots
    uint8_t* after = ba_smem_raw + (((raw + 1023u) & ~1023u) - raw) + (size_t)BA_WARPS * BA_SLOTS * BA_SLOT_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(after) + warp * BA_SLOTS;        // [BA_WARPS][BA_SLOTS]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(after + BA_WARPS * BA_SLOTS * 8);
    if (tid == 0) *abort_flag = 0;
    if (lane == 0) {
        for (int i = 0; i < BA_SLOTS; ++i) mbar_init(smem_u32(&full[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    uint32_t uses = 0;
    b_attn_dispatch(p, &p.kv_map, warp, lane, ring, full, abort_flag, uses);
}

// Combines the segments of every (sequence, kv head) pair and writes the attention output straight into the operand
// of the O projection (bf16 hi and lo halves).  The pair's chunks [first, first + nch) were processed by the warps
// whose ranges meet them; warp w left its part in slot (pair + w).  Grid (query heads, batch), hd / 2 threads x 2
// outputs: the threads first turn the segments' (maximum, sum) pairs into one weight per segment (in shared memory,
// segments beyond BA_MERGE_SEGS in further rounds), then every thread adds up its two outputs over the segments --
// independent loads, the additions in segment order.
constexpr int BA_MERGE_SEGS = 64;
// Shared memory of one merge item (a group of hd / 2 <= 64 threads).
struct BaMergeSmem {
    uint32_t seg[2];
    float wgt[BA_MERGE_SEGS];
    float red[4];
};
// One item = (query head hq, sequence b), NT = hd / 2 threads (32 or 64), BAR = the group's barrier.
template <int BAR, int NT>
__device__ __forceinline__ void b_merge_item(const BAttnView& p, uint32_t hq, uint32_t b, uint32_t tid, BaMergeSmem& sm) {
    const uint32_t G = p.G, hd = p.hd, g = hq / G, h = hq % G;
    if (tid < 32) {   // lane bb: chunks of sequence bb; W = all chunks, first = chunks before this pair
        const uint32_t pb = BA_SLOT_BYTES / (4u * hd);
        const uint32_t n = tid < p.B ? ba_chunks(p.positions[tid], pb) * p.nkv : 0u;
        uint32_t W = n, first = tid < b ? n : 0u;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            W += __shfl_xor_sync(0xffffffffu, W, o);
            first += __shfl_xor_sync(0xffffffffu, first, o);
        }
        if (tid == 0) {
            const uint32_t nch = ba_chunks(p.positions[b], pb), NW = ba_workers(W, p.NW);
            first += g * nch;
            // the warp whose range holds chunk x: floor(((x + 1) * NW - 1) / W)  (every range holds at least one chunk)
            sm.seg[0] = (uint32_t)((((uint64_t)first + 1u) * NW - 1u) / W);
            sm.seg[1] = (uint32_t)((((uint64_t)first + nch) * NW - 1u) / W);
        }
    }
    group_bar<BAR, NT>();
    const uint32_t w_first = sm.seg[0], nseg = sm.seg[1] - sm.seg[0] + 1u;
    const size_t pair = (size_t)b * p.nkv + g;
    const float* ml = p.part_ml + ((pair + w_first) * G + h) * 2;   // segment s: ml[s * G * 2], o[s * G * hd]
    const float* po = p.part_o + ((pair + w_first) * G + h) * hd;
    // running maximum over all segments
    float M = -INFINITY;
    for (uint32_t s = tid; s < nseg; s += NT) M = fmaxf(M, ml[(size_t)s * G * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    if ((tid & 31) == 0) sm.red[tid >> 5] = M;
    group_bar<BAR, NT>();
    M = fmaxf(sm.red[0], NT > 32 ? sm.red[1] : -INFINITY);
    float L = 0.f, A0 = 0.f, A1 = 0.f;
    const uint32_t d = 2 * tid;   // hd is even; NT = hd / 2
    for (uint32_t s0 = 0; s0 < nseg; s0 += BA_MERGE_SEGS) {
        const uint32_t ns = min((uint32_t)BA_MERGE_SEGS, nseg - s0);
        group_bar<BAR, NT>();   // the previous round's weights have been used
        for (uint32_t s = tid; s < ns; s += NT) sm.wgt[s] = rescale(ml[(size_t)(s0 + s) * G * 2], M);
        group_bar<BAR, NT>();
#pragma unroll 4
        for (uint32_t s = 0; s < ns; ++s) {   // every thread also sums the segments' row sums itself, in segment order
            const float c = sm.wgt[s];
            const float2 o = *reinterpret_cast<const float2*>(po + (size_t)(s0 + s) * G * hd + d);
            L += ml[(size_t)(s0 + s) * G * 2 + 1] * c;
            A0 += o.x * c;
            A1 += o.y * c;
        }
    }
    if (d < hd) put_operand2(p.xop, p.QD, b, hq * hd + d, A0 / L, A1 / L);
}

// grid (query heads, batch), hd / 2 threads
__global__ void __launch_bounds__(64) kl_b_attn_merge_kernel(const BAttnParams p) {
    __shared__ BaMergeSmem sm;
    griddep_launch();
    griddep_wait();
    if (*p.status != 0) return;
    if (p.hd == 128) b_merge_item<0, 64>(p, blockIdx.x, blockIdx.y, threadIdx.x, sm);
    else b_merge_item<0, 32>(p, blockIdx.x, blockIdx.y, threadIdx.x, sm);
}

}  // namespace kl
